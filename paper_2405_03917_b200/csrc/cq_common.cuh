// Shared declarations of the CQ library's translation units (device code is sm_100a only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cq.h"

namespace cq {

constexpr int kTokenBlock = CQ_TOKEN_BLOCK;   // tokens per code block of the library layout
constexpr float kLog2e = 1.4426950408889634f;

// Shape of one call, filled by the API layer after validation.
struct Shape {
    int64_t n_seq;
    int64_t max_tokens;
    int64_t n_blocks;     // ceil(max_tokens / 16): code blocks per (sequence, head)
    int n_q_heads;
    int n_kv_heads;
    int head_dim;
    int c;
    int b;
    int G;                // head_dim / c
    int K;                // 2^b
    int R;                // n_q_heads / n_kv_heads
    int hb;               // code bits above the low byte: 0 for b <= 8, else b - 8 (1, 2, 4 or 8)
    int block_bytes;      // bytes of one 16-token block of one head: G * (16 + 2 * hb)
};

// Bits of a code above its low byte, and the bytes of a block, for b bits per code.
__host__ __device__ inline int high_bits(int b) { return b > 8 ? b - 8 : 0; }
__host__ __device__ inline int block_bytes_for(int G, int b) { return G * (kTokenBlock + 2 * high_bits(b)); }

// Layout of a block (16 tokens of one head): first the G low words (16 bytes: the low byte of the
// code of each token), then, for b > 8, the G high words (2 * hb bytes: the remaining hb bits of
// token k at bits [k * hb, (k + 1) * hb), little endian).
// Byte offset of the low word of (sequence s, head h, block blk, group g).
__host__ __device__ inline int64_t code_word_offset(const Shape& sh, int n_heads, int64_t s, int h, int64_t blk, int g)
{
    return ((s * n_heads + h) * sh.n_blocks + blk) * (int64_t)sh.block_bytes + (int64_t)g * kTokenBlock;
}
// Byte offset of the high word of the same (block, group); only for b > 8.
__host__ __device__ inline int64_t code_high_offset(const Shape& sh, int n_heads, int64_t s, int h, int64_t blk, int g)
{
    return ((s * n_heads + h) * sh.n_blocks + blk) * (int64_t)sh.block_bytes + (int64_t)sh.G * kTokenBlock +
           (int64_t)g * 2 * sh.hb;
}
#ifdef __CUDACC__
// Code of token k (0..15) of group g in the block that starts at `block`.
__device__ inline int read_code(const uint8_t* __restrict__ block, const Shape& sh, int g, int k)
{
    int code = block[g * kTokenBlock + k];
    if (sh.hb) {
        const int bit = k * sh.hb;
        const int hi = (block[sh.G * kTokenBlock + g * 2 * sh.hb + (bit >> 3)] >> (bit & 7)) & ((1 << sh.hb) - 1);
        code |= hi << 8;
    }
    return code;
}
#endif

// A split-K partial: running max (log2 domain), normaliser, head_dim accumulators.
__host__ __device__ inline int partial_stride(int head_dim) { return head_dim + 2; }

// ---- host helpers (cq_api.cu) ----
// SM count of the current device (queried once per device and process).
int device_sm_count();
// cudaFuncAttributeMaxDynamicSharedMemorySize for `func`, set once per device and (func, bytes);
// `slot` is a small integer unique to the call site (0 <= slot < 64).
cudaError_t ensure_dynamic_smem(const void* func, int bytes, int slot);

// Launch plan of one tuned decode call: context chunk per CTA, partial slots per (sequence, query
// head), and the first item of the tail (-1: none).
struct DecodePlan {
    int chunk;
    int n_parts;
    int tail_first;
    unsigned grid;
};

// The token that a decode step appends before it attends (all null: none).  k_new, v_new: fp16
// (n_seq, n_kv_heads, head_dim); kc_w, vc_w: the caches, which take the token's codes at position seq_lens[s].
struct AppendArgs {
    const __half* k_new = nullptr;
    const __half* v_new = nullptr;
    uint8_t* kc_w = nullptr;
    uint8_t* vc_w = nullptr;
};

// ---- launchers implemented in the .cu files (return cudaGetLastError()) ----
cudaError_t launch_encode_generic(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                  int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st);
bool encode_small_supported(const Shape& sh);       // few-vector kernel: the group's codebook fits 48 KiB
cudaError_t launch_encode_small(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st);
// tcgen05 / tensor-memory encode kernel (head_dim 128, b = 8, c in {2, 4, 8}); same arguments as launch_encode_tuned
bool encode_tc_supported(const Shape& sh);
cudaError_t launch_encode_tc(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh, int64_t n_tokens,
                             int64_t token_offset, uint8_t* codes, cudaStream_t st, const __half* x2, const float* cb2,
                             uint8_t* codes2);
bool encode_tuned_supported(const Shape& sh);
// (x2, cb2, codes2): an optional second tensor of the same shape, encoded by the same launch.
// allow_tc: bulk inputs of byte codes go to the tensor-memory kernel (false: always the mma.sync kernels).
cudaError_t launch_encode_tuned(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st,
                                const __half* x2 = nullptr, const float* cb2 = nullptr, uint8_t* codes2 = nullptr,
                                bool allow_tc = true);

cudaError_t launch_to_rowmajor(const uint8_t* codes, const Shape& sh, uint8_t* rowmajor, cudaStream_t st);
cudaError_t launch_from_rowmajor(const uint8_t* rowmajor, const Shape& sh, uint8_t* codes, cudaStream_t st);

// Number of context splits each decode variant uses for this shape (host-side policy).
int decode_generic_splits(const Shape& sh);
cudaError_t launch_decode_generic(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                  const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                  float* out, float* partials, cudaStream_t st);
// Attention over codes of pre-RoPE keys (generic kernel; uses decode_generic_splits partial slots).
cudaError_t launch_decode_rope(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                               const float* vcb, const int32_t* seq_lens, const float* rope_cos, const float* rope_sin,
                               int pairing, float scale, const Shape& sh, float* out, float* partials, cudaStream_t st);
// Pre-RoPE key codes on the tuned kernel (cq_decode_rope.cu): head_dim 128, b = 8, c in {4, 8}, pairing (i, i + 64);
// the cos / sin tables must be 8-byte aligned.
bool decode_rope_tuned_supported(const Shape& sh, int pairing);
cudaError_t launch_decode_rope_tuned(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                     const float* vcb, const int32_t* seq_lens, const float* rope_cos, const float* rope_sin,
                                     float scale, const Shape& sh, float* out, float* partials, cudaStream_t st);
bool decode_tuned_supported(const Shape& sh);
int decode_tuned_parts(const Shape& sh);      // partial slots per (sequence, query head)
// per_head_tables: keep to decode_tuned_kernel (one table word per query head) also where the kernel
// with shared table words (cq_decode_pair.cu) would be picked.
cudaError_t launch_decode_tuned(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                float* out, float* partials, cudaStream_t st, bool per_head_tables = false,
                                const AppendArgs& app = AppendArgs());
// True when launch_decode_tuned would take a kernel that can append a token inside the attention launch.
bool decode_fused_append_supported(const Shape& sh);
int decode_step_fused_launches(const Shape& sh);      // 1: the attention kernel also writes the output; 2: plus the merge
// One decode step: the token (app) is encoded and appended at position seq_lens[s] and the attention covers
// seq_lens[s] + 1 tokens, in one attention launch (plus the merge).  Only where decode_fused_append_supported.
cudaError_t launch_decode_step_fused(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                     const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                     float* out, float* partials, const AppendArgs& app, cudaStream_t st);

// CQ-8c8b with a multiple of four query heads per KV head: two query heads per table word (cq_decode_pair.cu).
bool decode_pair_supported(const Shape& sh);
DecodePlan decode_pair_plan(const Shape& sh);
cudaError_t launch_decode_pair(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                               const int32_t* seq_lens, float scale, const Shape& sh, const DecodePlan& pl,
                               float* partials, cudaStream_t st, const AppendArgs& app = AppendArgs(), float* out = nullptr);
// (out: where the attention output goes; with one part per item (pl.n_parts == 1) the kernel writes it itself and
// no merge is needed, otherwise out is left alone and the caller merges the partials)

// Causal attention of the n_q newest cached tokens of every sequence (cq_prefill.cu); `generic` forces the plain kernel.
bool prefill_mma_supported(const Shape& sh);
cudaError_t launch_prefill(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                           const int32_t* seq_lens, float scale, const Shape& sh, int n_q, float* out, bool generic,
                           cudaStream_t st);

// dst[i] = src[i] + 1 for i < n (context length after one appended token).
cudaError_t launch_add_one(const int32_t* src, int32_t* dst, int n, cudaStream_t st);

// Centroid learning (cq_learn.cu): the vectors are [n_vec][n_heads][head_dim], weights [n_vec][n_heads][G] or null.
size_t learn_workspace_bytes(const Shape& sh, int64_t n_vec);
cudaError_t launch_kmeanspp_init(const __half* x, const float* weights, const double* uniforms, const Shape& sh,
                                 int64_t n_vec, float* codebooks, void* workspace, cudaStream_t st);
cudaError_t launch_lloyd_step(const __half* x, const float* weights, const float* cb_in, const Shape& sh, int64_t n_vec,
                              float* cb_out, double* objective, void* workspace, cudaStream_t st);
cudaError_t launch_learn(const __half* x, const float* weights, const double* uniforms, const Shape& sh, int64_t n_vec,
                         int n_iters, float* codebooks, double* objective, void* workspace, cudaStream_t st);

// Merge of split-K partials into out (shared by both decode variants).
cudaError_t launch_merge(const float* partials, int n_parts, const Shape& sh, float* out, cudaStream_t st);

}  // namespace cq
