/*
 * cq.h -- C ABI of the Coupled Quantization (CQ) KV-cache library for NVIDIA B200 (sm_100a).
 *
 * CQ (arXiv 2405.03917, Section 3.2) splits the head_dim channels of every key
 * or value vector into G = head_dim / c groups of c contiguous channels and
 * stores, per group, the b-bit index of the nearest of 2^b group-specific
 * centroids ("CQ-<c>c<b>b").  This library holds the two data-parallel steps
 * that touch every cached token:
 *
 *   cq_encode       vectors -> codes           (Section 3.2; the map CQ(.) of Eq. 5)
 *   cq_decode_attn  single-query attention that reads only the codes
 *                   (Eq. 1 with K and V replaced by their CQ reconstructions)
 *
 * and, around them: cq_encode_kv (key and value of the same tokens in one launch),
 * cq_decode_attn_rope (key codes taken before the rotary embedding, Section 3.2),
 * cq_prefill_attn (causal attention of a run of new tokens over the coded cache),
 * cq_decode_attn_static (no caller workspace), cq_decode_step_host (one decode
 * step from host buffers) and the centroid learning of Section 3.2.1
 * (cq_kmeanspp_init, cq_lloyd_step, cq_learn_centroids).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.  The
 *     caller owns all buffers, including the workspace; the library allocates
 *     nothing and keeps no state between calls (cq_decode_attn_static, below, is
 *     the one exception: it remembers the address of its built-in array).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     enqueue work and return; they never synchronise, except cq_decode_step_host.
 *   - Every function that returns int returns a cq_status: arguments are checked
 *     on the host before anything is launched, a failed check launches nothing,
 *     and a CUDA launch error is reported as CQ_ERR_CUDA.  Nothing aborts or traps.
 *   - Supported shapes: c divides head_dim, head_dim <= 256, n_q_heads a multiple
 *     of n_kv_heads, and b bits per code with 1 <= b <= 8 (one byte per code) or
 *     b = 9, 10, 12 or 16 (the low byte as for b <= 8 plus b - 8 packed upper bits,
 *     see the layout below; CQ-8c10b of the paper's Section 4 is the case b = 10:
 *     1.25 bytes per code).  Decode attention needs (head_dim / c) * 2^b <= 24576
 *     table entries (CQ_ERR_UNSUPPORTED otherwise).  Tuned kernels
 *     exist for head_dim 128: encode for c = 2, 4, 8 with b = 8, 9, 10, 12 (codebooks
 *     of more than 256 centroids are taken in chunks of 256); for b = 8 decode attention
 *     for c = 8, 4 and 2 with any number of query heads per KV head (a CTA serves up to 4, 2, 1 of them);
 *     and for decode attention of CQ-8c10b (head_dim 128, c = 8, b = 10).
 *     Every other supported shape runs on generic sm_100a kernels (never on the CPU).
 *   - Inputs must be finite.
 *
 * Code layout (version cq_layout_version() == 1).  Codes of one (sequence, head)
 * are stored in blocks of CQ_TOKEN_BLOCK = 16 tokens, group-major inside a block:
 *
 *   byte offset of (seq s, head h, token t, group g) =
 *       (((s * n_heads + h) * NB + t / 16) * G + g) * 16 + t % 16,   NB = ceil(max_tokens / 16)
 *
 * so the 16 codes of one group for 16 consecutive tokens are one aligned 16-byte
 * word.  For b > 8 a block of one head is G * (16 + 2 * (b - 8)) bytes: first the
 * G 16-byte words above, holding the low byte of every code, then G words of
 * 2 * (b - 8) bytes, word g holding the upper b - 8 bits of group g's 16 codes,
 * token k at bits [k * (b - 8), (k + 1) * (b - 8)) of the little-endian word:
 *
 *   block start of (s, h, t)  = ((s * n_heads + h) * NB + t / 16) * G * (16 + 2 * (b - 8))
 *   low byte of (.., g)       = block start + g * 16 + t % 16
 *   upper bits of (.., g)     = block start + G * 16 + g * 2 * (b - 8), bit (t % 16) * (b - 8) onwards
 *
 * cq_codes_to_rowmajor / cq_codes_from_rowmajor convert to and from the plain
 * [n_seq][max_tokens][n_heads][G] order (uint8 per code for b <= 8, uint16 for b > 8).
 * cq_codes_bytes() is the size of a code buffer (a multiple of 16).
 */
#ifndef CQ_H_
#define CQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CQ_TOKEN_BLOCK 16

typedef enum {
    CQ_OK = 0,
    CQ_ERR_NULL = -1,        /* a required pointer is NULL                                  */
    CQ_ERR_SHAPE = -2,       /* zero / negative dims, c does not divide head_dim, Hq % Hkv, */
                             /* token range outside [0, max_tokens]                         */
    CQ_ERR_UNSUPPORTED = -3, /* b not in {1..8, 9, 10, 12, 16}, head_dim > 256, tables too  */
                             /* large for shared memory                                     */
    CQ_ERR_ALIGN = -4,       /* a pointer is not aligned as documented                      */
    CQ_ERR_WORKSPACE = -5,   /* workspace smaller than the matching *_workspace_bytes()     */
    CQ_ERR_CUDA = -6         /* a CUDA runtime call or launch failed                        */
} cq_status;

/* Version of the code layout described above. */
int cq_layout_version(void);

/* Static, human-readable name of a cq_status value. */
const char *cq_status_string(int status);

/*
 * Bytes of one code buffer (K or V) for n_seq sequences of capacity max_tokens:
 * n_seq * n_heads * ceil(max_tokens / 16) * G * 16 (the paper's "bits per FPN"
 * b / c of Section 4, with b rounded up to one byte and the capacity rounded up
 * to a token block).  Returns 0 for invalid arguments.
 */
size_t cq_codes_bytes(int64_t n_seq, int64_t max_tokens, int n_heads, int head_dim, int c, int b);

/*
 * CQ encode (Section 3.2): for every vector and every group g, the index
 *   argmin_j  sum_{i<c} (x[g*c+i] - codebooks[h][g][j][i])^2 ,  lowest j on exact ties,
 * evaluated in fp32 (distances that differ by less than about 1e-6 relative may
 * resolve either way).
 *
 *   x_fp16       [n_seq][n_tokens][n_heads][head_dim] fp16, 16-byte aligned
 *   codebooks    [n_heads][G][2^b][c] fp32, 16-byte aligned
 *   seq_offsets  NULL, or [n_seq] int32: per-sequence first cache position
 *   codes_out    code buffer of cq_codes_bytes(n_seq, max_tokens, ...) bytes, 16-byte
 *                aligned; token i of sequence s is written at cache position
 *                token_offset + (seq_offsets ? seq_offsets[s] : 0) + i.  Positions
 *                outside [0, max_tokens) are skipped.  Other positions are untouched
 *                (appending one token rewrites G single bytes per head).
 * Requires 0 <= token_offset and, without seq_offsets, token_offset + n_tokens <= max_tokens.
 */
int cq_encode(const void *x_fp16, const float *codebooks, const int32_t *seq_offsets,
              int64_t n_seq, int64_t n_tokens, int64_t token_offset, int64_t max_tokens,
              int n_heads, int head_dim, int c, int b, void *codes_out, void *stream);

/*
 * cq_encode for the key and the value embeddings of the same tokens (Section 3.2 quantises
 * both, each with its own codebooks): the result is that of two cq_encode calls, in one
 * launch where the shape has a tuned encode kernel.  k_fp16 / v_fp16, k_cb / v_cb and the two
 * code buffers are laid out as in cq_encode; the two code buffers must differ.
 */
int cq_encode_kv(const void *k_fp16, const void *v_fp16, const float *k_cb, const float *v_cb,
                 const int32_t *seq_offsets, int64_t n_seq, int64_t n_tokens, int64_t token_offset,
                 int64_t max_tokens, int n_heads, int head_dim, int c, int b,
                 void *k_codes_out, void *v_codes_out, void *stream);

/*
 * Layout converters.  rowmajor is uint8 [n_seq][max_tokens][n_heads][G] (uint16 for b > 8).
 * to_rowmajor reads every position < max_tokens of the library layout;
 * from_rowmajor writes every position < max_tokens (block padding is zeroed).
 */
int cq_codes_to_rowmajor(const void *codes, int64_t n_seq, int64_t max_tokens, int n_heads,
                         int head_dim, int c, int b, void *rowmajor_out, void *stream);
int cq_codes_from_rowmajor(const void *rowmajor, int64_t n_seq, int64_t max_tokens, int n_heads,
                           int head_dim, int c, int b, void *codes_out, void *stream);

/*
 * Workspace of cq_decode_attn: split-K partials (running max, normaliser and
 * head_dim accumulators per (sequence, query head, context split)).
 * Returns 0 for invalid arguments.
 */
size_t cq_decode_attn_workspace_bytes(int n_seq, int n_q_heads, int n_kv_heads, int head_dim,
                                      int c, int b, int64_t max_tokens);

/*
 * Single-query decode attention over a CQ-coded cache.  For sequence s and query
 * head hq (which reads KV head hq / (n_q_heads / n_kv_heads)), over the first
 * n = seq_lens[s] cached tokens:
 *
 *   s_t = scale * <q, Khat_t>,  p = softmax(s_0..s_{n-1}),  out = sum_t p_t Vhat_t     (Eq. 1)
 *
 * where Khat_t / Vhat_t are the CQ reconstructions of token t (Section 3.2).  The
 * kernels never form Khat or Vhat: scores are sums over groups of a per-query table
 * LUT[g][j] = scale * <q_g, k_cb[g][j]>, softmax is online over context splits,
 * softmax weights are accumulated in bins per V code and the bins are multiplied
 * by the V centroids -- an exact re-association of Eq. 1, evaluated in fp32.
 *
 *   q_fp16     [n_seq][n_q_heads][head_dim] fp16
 *   k_codes, v_codes   code buffers in the library layout, capacity max_tokens,
 *                      n_kv_heads heads, 16-byte aligned
 *   k_cb, v_cb [n_kv_heads][G][2^b][c] fp32
 *   seq_lens   [n_seq] int32, each in [0, max_tokens]; values outside are clamped;
 *              seq_lens[s] == 0 gives a zero output row
 *   out        [n_seq][n_q_heads][head_dim] fp32
 *   workspace  at least cq_decode_attn_workspace_bytes(...) bytes, 16-byte aligned;
 *              contents on entry are ignored
 */
int cq_decode_attn(const void *q_fp16, const void *k_codes, const void *v_codes,
                   const float *k_cb, const float *v_cb, const int32_t *seq_lens, float scale,
                   int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                   int64_t max_tokens, float *out, void *workspace, size_t workspace_bytes,
                   void *stream);

/*
 * cq_decode_attn for callers that have no device memory to give as a workspace and cannot
 * obtain any.  (The paper has no counterpart to this entry point; it exists for the way the
 * library gets embedded.)  Typical cases: a serving process that handed every free byte of
 * HBM to its KV-cache pool at start-up, so a later cudaMalloc fails or stalls the device; or
 * a plug-in that is called with nothing but the raw input and output pointers and has no
 * route to its host's allocator.
 *
 * The split-K partials live in a fixed array of CQ_STATIC_WORKSPACE_BYTES bytes that is part
 * of the library image: every GPU that loads the library holds these bytes until the process
 * exits.  The function allocates and frees nothing, on the host or on the device.
 *
 *   - Arguments, layouts and result are those of cq_decode_attn, minus the workspace.
 *   - Shapes whose partials need more than CQ_STATIC_WORKSPACE_BYTES
 *     (cq_decode_attn_workspace_bytes(...) tells) are rejected with CQ_ERR_WORKSPACE and
 *     nothing is launched; use cq_decode_attn with your own workspace for those.
 *   - The first call on each device looks up the device address of the array (the device
 *     must be current, as for every call); make that first call before any stream capture
 *     begins.  A failure of the look-up is reported as CQ_ERR_CUDA.  The address is kept
 *     for the life of the process: after cudaDeviceReset (or any other teardown of the
 *     device's primary context) it is stale, so do not call this entry point again in a
 *     process that has reset the device.
 *   - All calls on a device share the one array.  It keeps what the last call left in it;
 *     that is harmless, because every call overwrites each partial it later reads and
 *     nothing has to start at zero.  Two calls that overlap on the GPU (different streams,
 *     or different host threads without ordering) race on the array and give wrong results:
 *     order them on one stream or with events.
 */
#define CQ_STATIC_WORKSPACE_BYTES (4u << 20)
int cq_decode_attn_static(const void *q_fp16, const void *k_codes, const void *v_codes,
                          const float *k_cb, const float *v_cb, const int32_t *seq_lens, float scale,
                          int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                          int64_t max_tokens, float *out, void *stream);

/*
 * Decode attention over a cache whose KEY codes were taken before the rotary position
 * embedding (last sentence of Section 3.2: CQ quantises keys before RoPE; Section 2.1:
 * the key transformation includes the positional encoding).  The key that enters Eq. 1
 * is the reconstructed key of token t rotated by the angles of position t:
 *   K_a = k_a cos - k_b sin,  K_b = k_b cos + k_a sin    for every channel pair (a, b),
 * with pair i's cosine and sine at position t read from rope_cos[t][i], rope_sin[t][i]
 * (fp32 [max_tokens][head_dim / 2], the tables a model caches; position = token index in
 * the cache).  pairing CQ_ROPE_HALF: (a, b) = (i, i + head_dim/2), the LLaMA / Mistral
 * convention; CQ_ROPE_INTERLEAVED: (2i, 2i + 1).  The paper fixes neither; both are
 * readings of this library.  q is used as given (already rotated for its own position);
 * values are not rotated.  Every other argument, the workspace size
 * (cq_decode_attn_workspace_bytes) and the output are those of cq_decode_attn.
 * CQ_ERR_UNSUPPORTED when a pair would not lie in whole groups (odd number of groups for
 * CQ_ROPE_HALF, odd c for CQ_ROPE_INTERLEAVED).  The score of a token is no longer a sum
 * of per-code table entries.  head_dim 128 with b = 8, c in {4, 8}, CQ_ROPE_HALF and 8-byte
 * aligned tables run on a tuned kernel (keys dequantised from fp16 centroids in shared
 * memory and rotated in registers; the cosines and sines of the tokens between two table
 * reads follow by the angle-addition rule and are checked against the tables, which are
 * read row by row when they are not of the rotary form); every other case on a generic
 * sm_100a kernel.  cq_decode_attn_rope_variant picks the kernel: 0 = automatic,
 * 1 = generic, 2 = tuned (CQ_ERR_UNSUPPORTED where it does not apply).
 */
#define CQ_ROPE_HALF 0
#define CQ_ROPE_INTERLEAVED 1
int cq_decode_attn_rope(const void *q_fp16, const void *k_codes, const void *v_codes,
                        const float *k_cb, const float *v_cb, const int32_t *seq_lens,
                        const float *rope_cos, const float *rope_sin, int pairing, float scale,
                        int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                        int64_t max_tokens, float *out, void *workspace, size_t workspace_bytes,
                        void *stream);
int cq_decode_attn_rope_variant(const void *q_fp16, const void *k_codes, const void *v_codes,
                        const float *k_cb, const float *v_cb, const int32_t *seq_lens,
                        const float *rope_cos, const float *rope_sin, int pairing, float scale,
                        int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                        int64_t max_tokens, float *out, void *workspace, size_t workspace_bytes,
                        int variant, void *stream);

/*
 * Causal attention of a run of new tokens over the CQ-coded cache: a prompt, or a chunk of
 * one.  Section 2.1 of the paper: Eq. 1 gives the output of the current token from the keys
 * and values of all tokens up to and including it; this call applies it to each of the
 * n_q_tokens newest cached tokens of every sequence, K and V being the CQ reconstructions
 * (Section 3.2).  The codes of the new tokens must already be in the cache (cq_encode /
 * cq_encode_kv with token_offset = old length): seq_lens[s] counts them.  Query i of
 * sequence s sits at position seq_lens[s] - n_q_tokens + i and attends the cached tokens
 * 0 ... that position:
 *
 *   s_t = scale * <q_i, Khat_t>,  p = softmax(s_0 .. s_pos),  out_i = sum_t p_t Vhat_t
 *
 *   q_fp16  device, fp16 [n_seq][n_q_tokens][n_q_heads][head_dim], 16-byte aligned
 *   out     device, fp32 [n_seq][n_q_tokens][n_q_heads][head_dim], 16-byte aligned
 *   codes, codebooks, seq_lens, scale, the head mapping: as for cq_decode_attn
 *
 * A query whose position is negative (seq_lens[s] < n_q_tokens) has nothing to attend and
 * gets a zero row.  No workspace.  head_dim 128 with one byte per code and c = 2, 4 or 8
 * (and a number of query heads per KV head that divides 64) runs on tensor cores: the
 * codes are turned back into fp16 vectors tile by tile, so results carry fp16 rounding of
 * the centroids and of the softmax weights (within the library's attention tolerance);
 * every other supported shape runs on a plain kernel.  CQ_ERR_SHAPE for n_q_tokens < 1 or
 * > max_tokens.
 */
int cq_prefill_attn(const void *q_fp16, const void *k_codes, const void *v_codes,
                    const float *k_cb, const float *v_cb, const int32_t *seq_lens, float scale,
                    int n_seq, int n_q_tokens, int n_q_heads, int n_kv_heads, int head_dim,
                    int c, int b, int64_t max_tokens, float *out, void *stream);
/* The same with an explicit kernel choice (tests, benchmarks): 0 = automatic, 1 = plain
 * kernel, 2 = tensor-core kernel (CQ_ERR_UNSUPPORTED when the shape has none). */
int cq_prefill_attn_variant(const void *q_fp16, const void *k_codes, const void *v_codes,
                            const float *k_cb, const float *v_cb, const int32_t *seq_lens, float scale,
                            int n_seq, int n_q_tokens, int n_q_heads, int n_kv_heads, int head_dim,
                            int c, int b, int64_t max_tokens, float *out, int variant, void *stream);

/*
 * Same operation with an explicit kernel choice, for tests and benchmarks:
 * variant 0 = automatic (what cq_decode_attn uses), 1 = generic kernel,
 * 2 = tuned kernel (CQ_ERR_UNSUPPORTED when the shape has none), 3 = tuned kernel
 * with one table word per query head, also for the shapes (CQ-8c8b with a multiple
 * of four query heads per KV head) where 2 takes the kernel that shares table words
 * between query heads; the same as 2 for every other shape.
 */
int cq_decode_attn_variant(const void *q_fp16, const void *k_codes, const void *v_codes,
                           const float *k_cb, const float *v_cb, const int32_t *seq_lens, float scale,
                           int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                           int64_t max_tokens, float *out, void *workspace, size_t workspace_bytes,
                           int variant, void *stream);

/* cq_encode with an explicit kernel choice: 0 = automatic, 1 = generic kernel,
 * 2 = the tuned kernels built on warp-level tensor-core instructions
 * (CQ_ERR_UNSUPPORTED when the shape has none), 3 = the few-vector kernel: one
 * warp per (vector, group) with the group's codebook in shared memory, which
 * variant 0 picks for appends of up to 128 vectors per head when the shape has no
 * tuned kernel (CQ_ERR_UNSUPPORTED when 2^b * c * 4 bytes exceed 48 KiB),
 * 4 = the bulk kernel with accumulators in tensor memory (head_dim 128, b = 8,
 * c in {2, 4, 8}, else CQ_ERR_UNSUPPORTED), which variant 0 picks for these shapes
 * once the input fills the device.  Every variant returns the same codes. */
int cq_encode_variant(const void *x_fp16, const float *codebooks, const int32_t *seq_offsets,
                      int64_t n_seq, int64_t n_tokens, int64_t token_offset, int64_t max_tokens,
                      int n_heads, int head_dim, int c, int b, void *codes_out, int variant,
                      void *stream);

/*
 * Centroid learning (Section 3.2.1): for every (head, group) an independent k-means problem
 * over the n_vec group vectors of a calibration tensor -- Eq. 5, or Eq. 6 when `weights` gives
 * every group vector its importance (the paper's g^T g of that group) -- with k-means++
 * initialisation and a fixed number of k-means iterations (Section 4.3).
 *
 *   x_fp16     [n_vec][n_heads][head_dim] fp16, 16-byte aligned
 *   weights    NULL (Eq. 5), or [n_vec][n_heads][G] fp32, non-negative (Eq. 6)
 *   uniforms   [n_heads][G][2^b] fp64 in [0, 1): the random draws of k-means++, supplied by the
 *              caller (the library draws nothing).  Centre 0 of a problem is vector
 *              floor(u_0 n_vec); centre k is the first vector whose running sum of w_i D_i, in
 *              index order and in fp64, reaches u_k times the total (D_i: squared distance to
 *              the nearest centre chosen so far)
 *   codebooks  [n_heads][G][2^b][c] fp32, 16-byte aligned
 *   objective_out  NULL, or [n_heads][G] fp64: sum_i w_i ||x_i - CQ(x_i)||^2 of the last
 *              assignment (measured against the codebooks that assignment used)
 *   workspace  at least cq_learn_workspace_bytes(...) bytes, 16-byte aligned
 *
 * cq_kmeanspp_init writes the initial centroids; cq_lloyd_step performs one iteration
 * (assignment = cq_encode, then every centroid moves to the weighted mean of its members; a
 * centroid without members stays; codebooks_in and codebooks_out must differ);
 * cq_learn_centroids runs the initialisation and n_iters iterations.
 */
size_t cq_learn_workspace_bytes(int64_t n_vec, int n_heads, int head_dim, int c, int b);
int cq_kmeanspp_init(const void *x_fp16, const float *weights, const double *uniforms, int64_t n_vec,
                     int n_heads, int head_dim, int c, int b, float *codebooks_out, void *workspace,
                     size_t workspace_bytes, void *stream);
int cq_lloyd_step(const void *x_fp16, const float *weights, const float *codebooks_in, int64_t n_vec,
                  int n_heads, int head_dim, int c, int b, float *codebooks_out, double *objective_out,
                  void *workspace, size_t workspace_bytes, void *stream);
int cq_learn_centroids(const void *x_fp16, const float *weights, const double *uniforms, int64_t n_vec,
                       int n_heads, int head_dim, int c, int b, int n_iters, float *codebooks_out,
                       double *objective_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * One decode step of one layer on DEVICE buffers: the new token's key and value
 * vectors are encoded (CQ encode, Section 3.2, as cq_encode does) and appended at
 * position seq_lens[s] of every sequence, and the step's query attends over
 * seq_lens[s] + 1 tokens (Eq. 1, as cq_decode_attn does).  For head_dim 128 with
 * b = 8 and c in {2, 4, 8} (the shapes with tuned decode kernels) the append
 * happens INSIDE the attention launch: the CTAs whose part of the context holds
 * the new position work the codes out, use them, and one of them writes them to
 * the cache; the step is then one attention launch, plus the merge of the partials
 * where contexts are split over CTAs (cq_decode_step_launches tells).  Every other
 * shape runs cq_encode_kv and cq_decode_attn one after the other.
 *
 *   q_fp16       [n_seq][n_q_heads][head_dim] fp16, device
 *   k_new_fp16, v_new_fp16   [n_seq][n_kv_heads][head_dim] fp16, device, 16-byte aligned
 *   seq_lens     [n_seq] int32, device: tokens cached BEFORE the step; not modified (the caller
 *                adds one to its own copy).  A sequence already at max_tokens gets no new token
 *                and attends over its max_tokens cached ones.
 *   k_codes, v_codes   device, layout of cq_encode; one byte per group is written per sequence
 *                and KV head.  Must not alias each other.
 *   out          [n_seq][n_q_heads][head_dim] fp32, device
 *   workspace    device, 16-byte aligned, at least cq_decode_step_workspace_bytes(...) bytes
 * Errors: as cq_decode_attn.  Asynchronous on `stream`.
 */
size_t cq_decode_step_workspace_bytes(int n_seq, int n_q_heads, int n_kv_heads, int head_dim,
                                      int c, int b, int64_t max_tokens);
/* Kernel launches of one cq_decode_step call on this shape (1: the attention kernel appends the
 * token and, with one part of the context per CTA, also writes the output; 2: plus the merge of
 * the partials; 4: lengths plus one, append, attention, merge); 0 for an unsupported shape. */
int cq_decode_step_launches(int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                            int64_t max_tokens);
int cq_decode_step(const void *q_fp16, const void *k_new_fp16, const void *v_new_fp16,
                   const int32_t *seq_lens, void *k_codes, void *v_codes, const float *k_cb,
                   const float *v_cb, float scale, int n_seq, int n_q_heads, int n_kv_heads,
                   int head_dim, int c, int b, int64_t max_tokens, float *out, void *workspace,
                   size_t workspace_bytes, void *stream);

/*
 * One decode step of one layer driven from HOST buffers (the end-to-end path):
 * copies the step's query and the new token's key and value vectors to the
 * device, runs cq_decode_step (the new token's codes appended at position
 * seq_lens_host[s] of every sequence, attention over seq_lens_host[s] + 1 tokens)
 * and copies the result back.  Synchronises `stream` before returning.
 *
 *   q_host       [n_seq][n_q_heads][head_dim] fp16   (pinned memory recommended)
 *   k_new_host, v_new_host   [n_seq][n_kv_heads][head_dim] fp16
 *                (when q_host, k_new_host and v_new_host lie back to back in host memory, in
 *                this order, the three travel in one copy instead of three)
 *   seq_lens_host [n_seq] int32: tokens already cached, each < max_tokens
 *   k_codes, v_codes, k_cb, v_cb   device, as in cq_decode_attn (codes are updated)
 *   out_host     [n_seq][n_q_heads][head_dim] fp32
 *   workspace    device, at least cq_decode_step_host_workspace_bytes(...) bytes
 */
size_t cq_decode_step_host_workspace_bytes(int n_seq, int n_q_heads, int n_kv_heads, int head_dim,
                                           int c, int b, int64_t max_tokens);
int cq_decode_step_host(const void *q_host, const void *k_new_host, const void *v_new_host,
                        const int32_t *seq_lens_host, void *k_codes, void *v_codes,
                        const float *k_cb, const float *v_cb, float scale,
                        int n_seq, int n_q_heads, int n_kv_heads, int head_dim, int c, int b,
                        int64_t max_tokens, float *out_host, void *workspace, size_t workspace_bytes,
                        void *stream);

#ifdef __cplusplus
}
#endif
#endif /* CQ_H_ */
