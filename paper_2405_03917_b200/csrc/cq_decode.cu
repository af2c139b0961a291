// Tuned decode-attention kernels (placeholder until the tuned path lands).
#include "cq_common.cuh"
namespace cq {
bool decode_tuned_supported(const Shape&) { return false; }
int decode_tuned_parts(const Shape&) { return 1; }
cudaError_t launch_decode_tuned(const __half*, const uint8_t*, const uint8_t*, const float*, const float*,
                                const int32_t*, float, const Shape&, float*, float*, cudaStream_t)
{
    return cudaErrorNotSupported;
}
}  // namespace cq
