// extern "C" entry points of the CQ library: host-side validation and dispatch only.
#include <mutex>

#include "cq_common.cuh"

using namespace cq;

namespace cq {

namespace {
constexpr int kDeviceSlots = 64;
std::mutex g_device_mutex;
int g_sm_count[kDeviceSlots] = {};                   // 0: not queried yet
int g_smem_set[kDeviceSlots][96] = {};               // per device and call site: dynamic shared memory size already set
}  // namespace

int device_sm_count()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kDeviceSlots) {
        cudaGetLastError();                          // no usable device (size queries on a machine without a GPU): B200's count
        return 148;
    }
    std::lock_guard<std::mutex> lock(g_device_mutex);
    if (g_sm_count[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = 148;
        }
        g_sm_count[dev] = n;
    }
    return g_sm_count[dev];
}

cudaError_t ensure_dynamic_smem(const void* func, int bytes, int slot)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kDeviceSlots || slot < 0 || slot >= 96)
        return cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    std::lock_guard<std::mutex> lock(g_device_mutex);
    if (g_smem_set[dev][slot] >= bytes && bytes > 0) return cudaSuccess;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) g_smem_set[dev][slot] = bytes;
    return e;
}

}  // namespace cq

namespace {

constexpr int kMaxHeadDim = 256;
constexpr int64_t kSmallEncodeVectors = 128;         // appends up to this many vectors per head may take the few-vector kernel
constexpr int64_t kGenericMaxTableEntries = 24576;   // (G * 2^b) floats x 2 tables must fit shared memory

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates the quantiser shape and fills `sh`; n_q_heads == n_kv_heads for encode-side calls.
int make_shape(int64_t n_seq, int64_t max_tokens, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
               Shape* sh)
{
    if (n_seq <= 0 || max_tokens <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 || c <= 0)
        return CQ_ERR_SHAPE;
    if (head_dim % c != 0 || n_q_heads % n_kv_heads != 0) return CQ_ERR_SHAPE;
    // codes wider than a byte keep their upper bits in a separate word of the block; only widths
    // whose upper part never straddles a byte are laid out
    if (b < 1 || (b > 8 && b != 9 && b != 10 && b != 12 && b != 16) || head_dim > kMaxHeadDim) return CQ_ERR_UNSUPPORTED;
    if (n_seq * (int64_t)n_q_heads > (int64_t)1 << 24) return CQ_ERR_UNSUPPORTED;
    sh->n_seq = n_seq;
    sh->max_tokens = max_tokens;
    sh->n_blocks = (max_tokens + kTokenBlock - 1) / kTokenBlock;
    sh->n_q_heads = n_q_heads;
    sh->n_kv_heads = n_kv_heads;
    sh->head_dim = head_dim;
    sh->c = c;
    sh->b = b;
    sh->G = head_dim / c;
    sh->K = 1 << b;
    sh->R = n_q_heads / n_kv_heads;
    sh->hb = high_bits(b);
    sh->block_bytes = block_bytes_for(sh->G, b);
    return CQ_OK;
}

// Partial slots per (sequence, query head) that the workspace must hold for any variant.
int max_parts(const Shape& sh)
{
    int p = decode_generic_splits(sh);
    if (decode_tuned_supported(sh)) {
        const int t = decode_tuned_parts(sh);
        if (t > p) p = t;
    }
    return p;
}

size_t partial_bytes(const Shape& sh)
{
    return (size_t)sh.n_seq * sh.n_q_heads * max_parts(sh) * partial_stride(sh.head_dim) * sizeof(float);
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

extern "C" {

int cq_layout_version(void) { return 1; }

const char* cq_status_string(int status)
{
    switch (status) {
        case CQ_OK: return "CQ_OK";
        case CQ_ERR_NULL: return "CQ_ERR_NULL: a required pointer is NULL";
        case CQ_ERR_SHAPE: return "CQ_ERR_SHAPE: invalid dimensions or token range";
        case CQ_ERR_UNSUPPORTED: return "CQ_ERR_UNSUPPORTED: shape outside what the library was built for";
        case CQ_ERR_ALIGN: return "CQ_ERR_ALIGN: pointer not 16-byte aligned";
        case CQ_ERR_WORKSPACE: return "CQ_ERR_WORKSPACE: workspace too small";
        case CQ_ERR_CUDA: return "CQ_ERR_CUDA: CUDA runtime error";
        default: return "unknown cq_status";
    }
}

size_t cq_codes_bytes(int64_t n_seq, int64_t max_tokens, int n_heads, int head_dim, int c, int b)
{
    Shape sh;
    if (make_shape(n_seq, max_tokens, n_heads, n_heads, head_dim, c, b, &sh) != CQ_OK) return 0;
    return round_up((size_t)sh.n_seq * n_heads * sh.n_blocks * sh.block_bytes, 16);
}

int cq_encode_variant(const void* x_fp16, const float* codebooks, const int32_t* seq_offsets, int64_t n_seq,
                      int64_t n_tokens, int64_t token_offset, int64_t max_tokens, int n_heads, int head_dim, int c,
                      int b, void* codes_out, int variant, void* stream)
{
    if (!x_fp16 || !codebooks || !codes_out) return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_heads, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (n_tokens < 0 || token_offset < 0) return CQ_ERR_SHAPE;
    if (!seq_offsets && token_offset + n_tokens > max_tokens) return CQ_ERR_SHAPE;
    if (!aligned16(x_fp16) || !aligned16(codebooks) || !aligned16(codes_out)) return CQ_ERR_ALIGN;
    if (variant < 0 || variant > 4) return CQ_ERR_SHAPE;
    if (n_tokens == 0) return CQ_OK;
    const bool tuned_ok = encode_tuned_supported(sh);
    if (variant == 2 && !tuned_ok) return CQ_ERR_UNSUPPORTED;
    if (variant == 4 && !encode_tc_supported(sh)) return CQ_ERR_UNSUPPORTED;
    const bool small_ok = encode_small_supported(sh);
    if (variant == 3 && !small_ok) return CQ_ERR_UNSUPPORTED;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // An append (a few vectors per head) is latency-bound.  Shapes without a tuned kernel take the
    // few-vector kernel for it (13 us against 300 us of the generic kernel for 64 vectors x 8 heads of
    // CQ-8c8b); the tuned kernel's single-tile form is still faster where it exists (9 us).
    if (variant == 3 || (variant == 0 && !tuned_ok && small_ok && n_seq * n_tokens <= kSmallEncodeVectors)) {
        cudaError_t es = launch_encode_small(static_cast<const __half*>(x_fp16), codebooks, seq_offsets, sh, n_tokens,
                                             token_offset, static_cast<uint8_t*>(codes_out), cs);
        return es == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
    }
    if (variant == 4) {
        cudaError_t et = launch_encode_tc(static_cast<const __half*>(x_fp16), codebooks, seq_offsets, sh, n_tokens, token_offset,
                                          static_cast<uint8_t*>(codes_out), cs, nullptr, nullptr, nullptr);
        return et == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
    }
    const bool use_tuned = variant == 2 || (variant == 0 && tuned_ok);
    cudaError_t e = use_tuned
                        ? launch_encode_tuned(static_cast<const __half*>(x_fp16), codebooks, seq_offsets, sh, n_tokens,
                                              token_offset, static_cast<uint8_t*>(codes_out), cs, nullptr, nullptr, nullptr,
                                              variant == 0)
                        : launch_encode_generic(static_cast<const __half*>(x_fp16), codebooks, seq_offsets, sh,
                                                n_tokens, token_offset, static_cast<uint8_t*>(codes_out), cs);
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_encode(const void* x_fp16, const float* codebooks, const int32_t* seq_offsets, int64_t n_seq, int64_t n_tokens,
              int64_t token_offset, int64_t max_tokens, int n_heads, int head_dim, int c, int b, void* codes_out,
              void* stream)
{
    return cq_encode_variant(x_fp16, codebooks, seq_offsets, n_seq, n_tokens, token_offset, max_tokens, n_heads,
                             head_dim, c, b, codes_out, 0, stream);
}

int cq_encode_kv(const void* k_fp16, const void* v_fp16, const float* k_cb, const float* v_cb,
                 const int32_t* seq_offsets, int64_t n_seq, int64_t n_tokens, int64_t token_offset, int64_t max_tokens,
                 int n_heads, int head_dim, int c, int b, void* k_codes_out, void* v_codes_out, void* stream)
{
    if (!k_fp16 || !v_fp16 || !k_cb || !v_cb || !k_codes_out || !v_codes_out) return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_heads, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (n_tokens < 0 || token_offset < 0) return CQ_ERR_SHAPE;
    if (!seq_offsets && token_offset + n_tokens > max_tokens) return CQ_ERR_SHAPE;
    if (!aligned16(k_fp16) || !aligned16(v_fp16) || !aligned16(k_cb) || !aligned16(v_cb) || !aligned16(k_codes_out) ||
        !aligned16(v_codes_out))
        return CQ_ERR_ALIGN;
    if (k_codes_out == v_codes_out) return CQ_ERR_SHAPE;
    if (n_tokens == 0) return CQ_OK;
    if (encode_tuned_supported(sh)) {       // one launch for both tensors
        cudaError_t e = launch_encode_tuned(static_cast<const __half*>(k_fp16), k_cb, seq_offsets, sh, n_tokens, token_offset,
                                            static_cast<uint8_t*>(k_codes_out), static_cast<cudaStream_t>(stream),
                                            static_cast<const __half*>(v_fp16), v_cb, static_cast<uint8_t*>(v_codes_out));
        return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
    }
    st = cq_encode(k_fp16, k_cb, seq_offsets, n_seq, n_tokens, token_offset, max_tokens, n_heads, head_dim, c, b,
                   k_codes_out, stream);
    if (st != CQ_OK) return st;
    return cq_encode(v_fp16, v_cb, seq_offsets, n_seq, n_tokens, token_offset, max_tokens, n_heads, head_dim, c, b,
                     v_codes_out, stream);
}

int cq_codes_to_rowmajor(const void* codes, int64_t n_seq, int64_t max_tokens, int n_heads, int head_dim, int c,
                         int b, void* rowmajor_out, void* stream)
{
    if (!codes || !rowmajor_out) return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_heads, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (!aligned16(codes)) return CQ_ERR_ALIGN;
    cudaError_t e = launch_to_rowmajor(static_cast<const uint8_t*>(codes), sh, static_cast<uint8_t*>(rowmajor_out),
                                       static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_codes_from_rowmajor(const void* rowmajor, int64_t n_seq, int64_t max_tokens, int n_heads, int head_dim, int c,
                           int b, void* codes_out, void* stream)
{
    if (!rowmajor || !codes_out) return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_heads, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (!aligned16(codes_out)) return CQ_ERR_ALIGN;
    cudaError_t e = launch_from_rowmajor(static_cast<const uint8_t*>(rowmajor), sh, static_cast<uint8_t*>(codes_out),
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

size_t cq_decode_attn_workspace_bytes(int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                                      int64_t max_tokens)
{
    Shape sh;
    if (make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh) != CQ_OK) return 0;
    return round_up(partial_bytes(sh), 256);
}

int cq_decode_attn_variant(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb,
                           const float* v_cb, const int32_t* seq_lens, float scale, int n_seq, int n_q_heads,
                           int n_kv_heads, int head_dim, int c, int b, int64_t max_tokens, float* out, void* workspace,
                           size_t workspace_bytes, int variant, void* stream)
{
    if (!q_fp16 || !k_codes || !v_codes || !k_cb || !v_cb || !seq_lens || !out || !workspace) return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (variant < 0 || variant > 3) return CQ_ERR_SHAPE;
    if (!aligned16(k_codes) || !aligned16(v_codes) || !aligned16(workspace) || !aligned16(k_cb) || !aligned16(v_cb) ||
        (reinterpret_cast<uintptr_t>(q_fp16) & 1u) || (reinterpret_cast<uintptr_t>(out) & 3u))
        return CQ_ERR_ALIGN;
    if (workspace_bytes < round_up(partial_bytes(sh), 256)) return CQ_ERR_WORKSPACE;
    const bool tuned_ok = decode_tuned_supported(sh);
    if ((variant == 2 || variant == 3) && !tuned_ok) return CQ_ERR_UNSUPPORTED;
    const bool use_tuned = variant == 2 || variant == 3 || (variant == 0 && tuned_ok);
    if (!use_tuned && (int64_t)sh.G * sh.K > kGenericMaxTableEntries) return CQ_ERR_UNSUPPORTED;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const __half* q = static_cast<const __half*>(q_fp16);
    const uint8_t* kc = static_cast<const uint8_t*>(k_codes);
    const uint8_t* vc = static_cast<const uint8_t*>(v_codes);
    float* partials = static_cast<float*>(workspace);
    cudaError_t e = use_tuned ? launch_decode_tuned(q, kc, vc, k_cb, v_cb, seq_lens, scale, sh, out, partials, cs, variant == 3)
                              : launch_decode_generic(q, kc, vc, k_cb, v_cb, seq_lens, scale, sh, out, partials, cs);
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_decode_attn(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb, const float* v_cb,
                   const int32_t* seq_lens, float scale, int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c,
                   int b, int64_t max_tokens, float* out, void* workspace, size_t workspace_bytes, void* stream)
{
    return cq_decode_attn_variant(q_fp16, k_codes, v_codes, k_cb, v_cb, seq_lens, scale, n_seq, n_q_heads, n_kv_heads,
                                  head_dim, c, b, max_tokens, out, workspace, workspace_bytes, 0, stream);
}

int cq_decode_attn_rope_variant(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb,
                                const float* v_cb, const int32_t* seq_lens, const float* rope_cos, const float* rope_sin,
                                int pairing, float scale, int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c,
                                int b, int64_t max_tokens, float* out, void* workspace, size_t workspace_bytes, int variant,
                                void* stream)
{
    if (!q_fp16 || !k_codes || !v_codes || !k_cb || !v_cb || !seq_lens || !rope_cos || !rope_sin || !out || !workspace)
        return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (pairing != CQ_ROPE_HALF && pairing != CQ_ROPE_INTERLEAVED) return CQ_ERR_SHAPE;
    if (head_dim % 2 != 0) return CQ_ERR_SHAPE;
    // a pair must lie in whole groups: (i, i + D/2) needs an even number of groups, (2i, 2i+1) an even c
    if (pairing == CQ_ROPE_HALF ? sh.G % 2 != 0 : c % 2 != 0) return CQ_ERR_UNSUPPORTED;
    if (!aligned16(k_codes) || !aligned16(v_codes) || !aligned16(workspace) || !aligned16(k_cb) || !aligned16(v_cb) ||
        (reinterpret_cast<uintptr_t>(q_fp16) & 1u) || (reinterpret_cast<uintptr_t>(out) & 3u) ||
        (reinterpret_cast<uintptr_t>(rope_cos) & 3u) || (reinterpret_cast<uintptr_t>(rope_sin) & 3u))
        return CQ_ERR_ALIGN;
    if (workspace_bytes < round_up(partial_bytes(sh), 256)) return CQ_ERR_WORKSPACE;
    if (variant < 0 || variant > 2) return CQ_ERR_SHAPE;
    const bool tuned_ok = decode_rope_tuned_supported(sh, pairing) &&
                          ((reinterpret_cast<uintptr_t>(rope_cos) | reinterpret_cast<uintptr_t>(rope_sin)) & 7u) == 0;
    if (variant == 2 && !tuned_ok) return CQ_ERR_UNSUPPORTED;
    if (variant == 2 || (variant == 0 && tuned_ok)) {
        cudaError_t et = launch_decode_rope_tuned(static_cast<const __half*>(q_fp16), static_cast<const uint8_t*>(k_codes),
                                                  static_cast<const uint8_t*>(v_codes), k_cb, v_cb, seq_lens, rope_cos, rope_sin,
                                                  scale, sh, out, static_cast<float*>(workspace),
                                                  static_cast<cudaStream_t>(stream));
        return et == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
    }
    if ((int64_t)sh.G * sh.K > 2 * kGenericMaxTableEntries) return CQ_ERR_UNSUPPORTED;     // one table (the bins) only
    cudaError_t e = launch_decode_rope(static_cast<const __half*>(q_fp16), static_cast<const uint8_t*>(k_codes),
                                       static_cast<const uint8_t*>(v_codes), k_cb, v_cb, seq_lens, rope_cos, rope_sin,
                                       pairing, scale, sh, out, static_cast<float*>(workspace),
                                       static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_decode_attn_rope(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb,
                        const float* v_cb, const int32_t* seq_lens, const float* rope_cos, const float* rope_sin,
                        int pairing, float scale, int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                        int64_t max_tokens, float* out, void* workspace, size_t workspace_bytes, void* stream)
{
    return cq_decode_attn_rope_variant(q_fp16, k_codes, v_codes, k_cb, v_cb, seq_lens, rope_cos, rope_sin, pairing, scale, n_seq,
                                       n_q_heads, n_kv_heads, head_dim, c, b, max_tokens, out, workspace, workspace_bytes, 0,
                                       stream);
}

int cq_prefill_attn_variant(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb,
                            const float* v_cb, const int32_t* seq_lens, float scale, int n_seq, int n_q_tokens,
                            int n_q_heads, int n_kv_heads, int head_dim, int c, int b, int64_t max_tokens, float* out,
                            int variant, void* stream)
{
    if (!q_fp16 || !k_codes || !v_codes || !k_cb || !v_cb || !seq_lens || !out) return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (n_q_tokens <= 0 || n_q_tokens > max_tokens) return CQ_ERR_SHAPE;
    if (variant < 0 || variant > 2) return CQ_ERR_SHAPE;
    if ((int64_t)n_seq * n_q_tokens * n_q_heads > (int64_t)1 << 30) return CQ_ERR_UNSUPPORTED;
    if (!aligned16(k_codes) || !aligned16(v_codes) || !aligned16(k_cb) || !aligned16(v_cb) || !aligned16(q_fp16) ||
        !aligned16(out))
        return CQ_ERR_ALIGN;
    const bool mma_ok = prefill_mma_supported(sh);
    if (variant == 2 && !mma_ok) return CQ_ERR_UNSUPPORTED;
    cudaError_t e = launch_prefill(static_cast<const __half*>(q_fp16), static_cast<const uint8_t*>(k_codes),
                                   static_cast<const uint8_t*>(v_codes), k_cb, v_cb, seq_lens, scale, sh, n_q_tokens, out,
                                   variant == 1, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_prefill_attn(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb, const float* v_cb,
                    const int32_t* seq_lens, float scale, int n_seq, int n_q_tokens, int n_q_heads, int n_kv_heads,
                    int head_dim, int c, int b, int64_t max_tokens, float* out, void* stream)
{
    return cq_prefill_attn_variant(q_fp16, k_codes, v_codes, k_cb, v_cb, seq_lens, scale, n_seq, n_q_tokens, n_q_heads,
                                   n_kv_heads, head_dim, c, b, max_tokens, out, 0, stream);
}

// ---------------------------------------------------------------------------------------------
// cq_decode_attn_static: the split-K partials live in this array instead of a caller workspace.
// In host code the name `g_static_workspace` is only a handle for the runtime, not a device
// address; the address a kernel can use comes from cudaGetSymbolAddress, looked up once per
// device and remembered here.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_workspace[CQ_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};          // device address of g_static_workspace, per device ordinal

// Device address of the array on the current device; nullptr (and *err set) when the look-up fails.
void* static_workspace(cudaError_t* err)
{
    int dev = -1;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= kMaxDevices) { *err = cudaErrorInvalidDevice; return nullptr; }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        *err = cudaGetSymbolAddress(&p, g_static_workspace);
        if (*err != cudaSuccess) return nullptr;
        g_static_ptr[dev] = p;
    }
    return g_static_ptr[dev];
}
}  // namespace

int cq_decode_attn_static(const void* q_fp16, const void* k_codes, const void* v_codes, const float* k_cb,
                          const float* v_cb, const int32_t* seq_lens, float scale, int n_seq, int n_q_heads,
                          int n_kv_heads, int head_dim, int c, int b, int64_t max_tokens, float* out, void* stream)
{
    if (!q_fp16 || !k_codes || !v_codes || !k_cb || !v_cb || !seq_lens || !out) return CQ_ERR_NULL;
    const size_t need = cq_decode_attn_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens);
    if (need == 0) {
        Shape sh;
        return make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh);
    }
    if (need > (size_t)CQ_STATIC_WORKSPACE_BYTES) return CQ_ERR_WORKSPACE;     // too large for the built-in array
    cudaError_t err = cudaSuccess;
    void* ws = static_workspace(&err);
    if (!ws) return CQ_ERR_CUDA;
    return cq_decode_attn(q_fp16, k_codes, v_codes, k_cb, v_cb, seq_lens, scale, n_seq, n_q_heads, n_kv_heads,
                          head_dim, c, b, max_tokens, out, ws, (size_t)CQ_STATIC_WORKSPACE_BYTES, stream);
}

// ---------------------------------------------------------------------------------------------
// Centroid learning (Section 3.2.1): k-means++ initialisation and k-means iterations.
// ---------------------------------------------------------------------------------------------
namespace {
int learn_shape(int64_t n_vec, int n_heads, int head_dim, int c, int b, Shape* sh)
{
    if (n_vec <= 0) return CQ_ERR_SHAPE;
    const int st = make_shape(1, n_vec, n_heads, n_heads, head_dim, c, b, sh);
    if (st != CQ_OK) return st;
    // the update step keeps sums, counts and the old centroids of one problem in shared memory
    if ((size_t)(2 * sh->K * sh->c + sh->K) * sizeof(float) > (size_t)200 * 1024) return CQ_ERR_UNSUPPORTED;
    return CQ_OK;
}
}  // namespace

size_t cq_learn_workspace_bytes(int64_t n_vec, int n_heads, int head_dim, int c, int b)
{
    Shape sh;
    if (learn_shape(n_vec, n_heads, head_dim, c, b, &sh) != CQ_OK) return 0;
    return learn_workspace_bytes(sh, n_vec);
}

int cq_kmeanspp_init(const void* x_fp16, const float* weights, const double* uniforms, int64_t n_vec, int n_heads,
                     int head_dim, int c, int b, float* codebooks_out, void* workspace, size_t workspace_bytes,
                     void* stream)
{
    if (!x_fp16 || !uniforms || !codebooks_out || !workspace) return CQ_ERR_NULL;
    Shape sh;
    int st = learn_shape(n_vec, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (!aligned16(x_fp16) || !aligned16(codebooks_out) || !aligned16(workspace)) return CQ_ERR_ALIGN;
    if (workspace_bytes < learn_workspace_bytes(sh, n_vec)) return CQ_ERR_WORKSPACE;
    cudaError_t e = launch_kmeanspp_init(static_cast<const __half*>(x_fp16), weights, uniforms, sh, n_vec, codebooks_out,
                                         workspace, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_lloyd_step(const void* x_fp16, const float* weights, const float* codebooks_in, int64_t n_vec, int n_heads,
                  int head_dim, int c, int b, float* codebooks_out, double* objective_out, void* workspace,
                  size_t workspace_bytes, void* stream)
{
    if (!x_fp16 || !codebooks_in || !codebooks_out || !workspace) return CQ_ERR_NULL;
    if (codebooks_in == codebooks_out) return CQ_ERR_SHAPE;
    Shape sh;
    int st = learn_shape(n_vec, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (!aligned16(x_fp16) || !aligned16(codebooks_in) || !aligned16(codebooks_out) || !aligned16(workspace))
        return CQ_ERR_ALIGN;
    if (workspace_bytes < learn_workspace_bytes(sh, n_vec)) return CQ_ERR_WORKSPACE;
    cudaError_t e = launch_lloyd_step(static_cast<const __half*>(x_fp16), weights, codebooks_in, sh, n_vec, codebooks_out,
                                      objective_out, workspace, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

int cq_learn_centroids(const void* x_fp16, const float* weights, const double* uniforms, int64_t n_vec, int n_heads,
                       int head_dim, int c, int b, int n_iters, float* codebooks_out, double* objective_out,
                       void* workspace, size_t workspace_bytes, void* stream)
{
    if (!x_fp16 || !uniforms || !codebooks_out || !workspace) return CQ_ERR_NULL;
    if (n_iters < 0) return CQ_ERR_SHAPE;
    Shape sh;
    int st = learn_shape(n_vec, n_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (!aligned16(x_fp16) || !aligned16(codebooks_out) || !aligned16(workspace)) return CQ_ERR_ALIGN;
    if (workspace_bytes < learn_workspace_bytes(sh, n_vec)) return CQ_ERR_WORKSPACE;
    cudaError_t e = launch_learn(static_cast<const __half*>(x_fp16), weights, uniforms, sh, n_vec, n_iters, codebooks_out,
                                 objective_out, workspace, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}

// Staging area of cq_decode_step_host inside the caller's workspace (all 256-byte aligned):
//   [q fp16][k_new fp16][v_new fp16][seq_lens int32][seq_lens+1 int32][out fp32][attention workspace]
size_t cq_decode_step_workspace_bytes(int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                                      int64_t max_tokens)
{
    const size_t attn = cq_decode_attn_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens);
    if (attn == 0) return 0;
    return attn + round_up((size_t)n_seq * 4, 256);          // the lengths after the append, where they are needed
}

int cq_decode_step_launches(int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b, int64_t max_tokens)
{
    Shape sh;
    if (make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh) != CQ_OK) return 0;
    if (decode_tuned_supported(sh) && decode_fused_append_supported(sh))
        return decode_step_fused_launches(sh);                   // attention (with the append inside) [+ merge]
    return 4;                                                      // lengths plus one, append, attention, merge
}

int cq_decode_step(const void* q_fp16, const void* k_new_fp16, const void* v_new_fp16, const int32_t* seq_lens,
                   void* k_codes, void* v_codes, const float* k_cb, const float* v_cb, float scale, int n_seq,
                   int n_q_heads, int n_kv_heads, int head_dim, int c, int b, int64_t max_tokens, float* out,
                   void* workspace, size_t workspace_bytes, void* stream)
{
    if (!q_fp16 || !k_new_fp16 || !v_new_fp16 || !seq_lens || !k_codes || !v_codes || !k_cb || !v_cb || !out || !workspace)
        return CQ_ERR_NULL;
    Shape sh;
    int st = make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh);
    if (st != CQ_OK) return st;
    if (!aligned16(k_codes) || !aligned16(v_codes) || !aligned16(workspace) || !aligned16(k_cb) || !aligned16(v_cb) ||
        !aligned16(k_new_fp16) || !aligned16(v_new_fp16) || (reinterpret_cast<uintptr_t>(q_fp16) & 1u) ||
        (reinterpret_cast<uintptr_t>(out) & 3u))
        return CQ_ERR_ALIGN;
    if (k_codes == v_codes) return CQ_ERR_SHAPE;
    const size_t attn_bytes = round_up(partial_bytes(sh), 256);
    if (workspace_bytes < attn_bytes + round_up((size_t)n_seq * 4, 256)) return CQ_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (decode_tuned_supported(sh) && decode_fused_append_supported(sh)) {
        AppendArgs app;
        app.k_new = static_cast<const __half*>(k_new_fp16);
        app.v_new = static_cast<const __half*>(v_new_fp16);
        app.kc_w = static_cast<uint8_t*>(k_codes);
        app.vc_w = static_cast<uint8_t*>(v_codes);
        cudaError_t e = launch_decode_step_fused(static_cast<const __half*>(q_fp16), app.kc_w, app.vc_w, k_cb, v_cb, seq_lens,
                                                 scale, sh, out, static_cast<float*>(workspace), app, cs);
        return e == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
    }
    // every other shape: the append is a launch of its own, the attention reads the lengths plus one
    int32_t* sl1 = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + attn_bytes);
    if (launch_add_one(seq_lens, sl1, n_seq, cs) != cudaSuccess) return CQ_ERR_CUDA;
    st = cq_encode_kv(k_new_fp16, v_new_fp16, k_cb, v_cb, seq_lens, n_seq, 1, 0, max_tokens, n_kv_heads, head_dim, c, b,
                      k_codes, v_codes, stream);
    if (st != CQ_OK) return st;
    return cq_decode_attn(q_fp16, k_codes, v_codes, k_cb, v_cb, sl1, scale, n_seq, n_q_heads, n_kv_heads, head_dim, c, b,
                          max_tokens, out, workspace, attn_bytes, stream);
}

size_t cq_decode_step_host_workspace_bytes(int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                                           int64_t max_tokens)
{
    const size_t attn = cq_decode_attn_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens);
    if (attn == 0) return 0;
    const size_t q = round_up((size_t)n_seq * n_q_heads * head_dim * 2, 256);
    const size_t kv = round_up((size_t)n_seq * n_kv_heads * head_dim * 2, 256);
    const size_t sl = round_up((size_t)n_seq * 4, 256);
    const size_t o = round_up((size_t)n_seq * n_q_heads * head_dim * 4, 256);
    return q + 2 * kv + 2 * sl + o + attn;
}

int cq_decode_step_host(const void* q_host, const void* k_new_host, const void* v_new_host,
                        const int32_t* seq_lens_host, void* k_codes, void* v_codes, const float* k_cb,
                        const float* v_cb, float scale, int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c,
                        int b, int64_t max_tokens, float* out_host, void* workspace, size_t workspace_bytes,
                        void* stream)
{
    if (!q_host || !k_new_host || !v_new_host || !seq_lens_host || !k_codes || !v_codes || !k_cb || !v_cb ||
        !out_host || !workspace)
        return CQ_ERR_NULL;
    const size_t need = cq_decode_step_host_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens);
    if (need == 0) {
        Shape sh;
        return make_shape(n_seq, max_tokens, n_q_heads, n_kv_heads, head_dim, c, b, &sh);
    }
    if (workspace_bytes < need) return CQ_ERR_WORKSPACE;
    if (!aligned16(workspace)) return CQ_ERR_ALIGN;
    for (int s = 0; s < n_seq; ++s)
        if (seq_lens_host[s] < 0 || seq_lens_host[s] >= max_tokens) return CQ_ERR_SHAPE;

    const size_t qb = (size_t)n_seq * n_q_heads * head_dim * 2;
    const size_t kvb = (size_t)n_seq * n_kv_heads * head_dim * 2;
    const size_t slb = (size_t)n_seq * 4;
    const size_t ob = (size_t)n_seq * n_q_heads * head_dim * 4;
    char* w = static_cast<char*>(workspace);
    char* d_q = w;                 w += round_up(qb, 256);
    char* d_k = w;                 w += round_up(kvb, 256);
    char* d_v = w;                 w += round_up(kvb, 256);
    int32_t* d_sl = reinterpret_cast<int32_t*>(w);   w += round_up(slb, 256);
    float* d_out = reinterpret_cast<float*>(w);      w += round_up(ob, 256);
    void* step_ws = w;              // attention partials, and the lengths plus one for the shapes that need them
    const size_t step_bytes = workspace_bytes - (size_t)(w - static_cast<char*>(workspace));

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // Few, large copies: query, key and value travel in one copy when the caller keeps them back to back
    // in host memory (the staging areas are then packed the same way).
    const bool packed = static_cast<const char*>(k_new_host) == static_cast<const char*>(q_host) + qb &&
                        static_cast<const char*>(v_new_host) == static_cast<const char*>(k_new_host) + kvb &&
                        qb % 16 == 0 && kvb % 16 == 0;
    if (packed) {
        d_k = d_q + qb;
        d_v = d_k + kvb;            // (fits: the three areas were sized with their paddings)
        if (cudaMemcpyAsync(d_q, q_host, qb + 2 * kvb, cudaMemcpyHostToDevice, cs) != cudaSuccess) return CQ_ERR_CUDA;
    } else {
        if (cudaMemcpyAsync(d_q, q_host, qb, cudaMemcpyHostToDevice, cs) != cudaSuccess) return CQ_ERR_CUDA;
        if (cudaMemcpyAsync(d_k, k_new_host, kvb, cudaMemcpyHostToDevice, cs) != cudaSuccess) return CQ_ERR_CUDA;
        if (cudaMemcpyAsync(d_v, v_new_host, kvb, cudaMemcpyHostToDevice, cs) != cudaSuccess) return CQ_ERR_CUDA;
    }
    if (cudaMemcpyAsync(d_sl, seq_lens_host, slb, cudaMemcpyHostToDevice, cs) != cudaSuccess) return CQ_ERR_CUDA;
    // The new token is appended at position seq_lens[s]; the attention then reads seq_lens[s] + 1 tokens.
    const int st = cq_decode_step(d_q, d_k, d_v, d_sl, k_codes, v_codes, k_cb, v_cb, scale, n_seq, n_q_heads, n_kv_heads,
                                  head_dim, c, b, max_tokens, d_out, step_ws, step_bytes, stream);
    if (st != CQ_OK) return st;
    if (cudaMemcpyAsync(out_host, d_out, ob, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return CQ_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return CQ_ERR_CUDA;
    return CQ_OK;
}

}  // extern "C"
