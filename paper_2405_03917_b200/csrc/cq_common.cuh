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
};

// Byte offset of the 16-byte code word of (sequence s, head h, block blk, group g).
__host__ __device__ inline int64_t code_word_offset(const Shape& sh, int n_heads, int64_t s, int h, int64_t blk, int g)
{
    return (((s * n_heads + h) * sh.n_blocks + blk) * sh.G + g) * (int64_t)kTokenBlock;
}

// A split-K partial: running max (log2 domain), normaliser, head_dim accumulators.
__host__ __device__ inline int partial_stride(int head_dim) { return head_dim + 2; }

// ---- launchers implemented in the .cu files (return cudaGetLastError()) ----
cudaError_t launch_encode_generic(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                  int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st);
bool encode_tuned_supported(const Shape& sh);
cudaError_t launch_encode_tuned(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st);

cudaError_t launch_to_rowmajor(const uint8_t* codes, const Shape& sh, uint8_t* rowmajor, cudaStream_t st);
cudaError_t launch_from_rowmajor(const uint8_t* rowmajor, const Shape& sh, uint8_t* codes, cudaStream_t st);

// Number of context splits each decode variant uses for this shape (host-side policy).
int decode_generic_splits(const Shape& sh);
cudaError_t launch_decode_generic(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                  const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                  float* out, float* partials, cudaStream_t st);
bool decode_tuned_supported(const Shape& sh);
int decode_tuned_parts(const Shape& sh);      // partial slots per (sequence, query head)
cudaError_t launch_decode_tuned(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                float* out, float* partials, cudaStream_t st);

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
