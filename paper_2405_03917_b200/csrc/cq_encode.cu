// Tuned encode kernels (placeholder until the tuned path lands).
#include "cq_common.cuh"
namespace cq {
bool encode_tuned_supported(const Shape&) { return false; }
cudaError_t launch_encode_tuned(const __half*, const float*, const int32_t*, const Shape&, int64_t, int64_t, uint8_t*,
                                cudaStream_t)
{
    return cudaErrorNotSupported;
}
}  // namespace cq
