// Generic sm_100a kernels of the CQ library: they accept every supported (head_dim, c, b)
// and favour plainness over speed.  The tuned kernels live in cq_encode.cu / cq_decode.cu.
#include "cq_common.cuh"
#include "cq_bulk_copy.cuh"

namespace cq {

// ------------------------------------------------------------------------------------------
// Encode (Section 3.2 of the paper): nearest centroid in L2 per group of c contiguous channels.
// One thread per (sequence, head, group, token); the token index is the fastest-varying one
// so that a warp reads one codebook (broadcast) and writes consecutive bytes of a code word.
// ------------------------------------------------------------------------------------------
__global__ void encode_generic_kernel(const __half* __restrict__ x, const float* __restrict__ cb,
                                      const int32_t* __restrict__ seq_offsets, Shape sh, int64_t n_tokens,
                                      int64_t token_offset, uint8_t* __restrict__ codes)
{
    const int n_heads = sh.n_kv_heads;
    const int64_t total = sh.n_seq * n_heads * sh.G * n_tokens;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx % n_tokens;
        int64_t rest = idx / n_tokens;
        const int g = (int)(rest % sh.G);
        rest /= sh.G;
        const int h = (int)(rest % n_heads);
        const int64_t s = rest / n_heads;
        const int64_t pos = token_offset + (seq_offsets ? seq_offsets[s] : 0) + i;
        if (pos < 0 || pos >= sh.max_tokens) continue;
        const __half* xv = x + ((s * n_tokens + i) * n_heads + h) * (int64_t)sh.head_dim + g * sh.c;
        const float* cg = cb + ((int64_t)h * sh.G + g) * sh.K * sh.c;
        float best = INFINITY;
        int arg = 0;
        for (int j = 0; j < sh.K; ++j) {
            float d = 0.f;
            for (int k = 0; k < sh.c; ++k) {
                const float diff = __half2float(xv[k]) - cg[j * sh.c + k];
                d = fmaf(diff, diff, d);
            }
            if (d < best) {   // strict: lowest index wins exact ties
                best = d;
                arg = j;
            }
        }
        const int k = (int)(pos % kTokenBlock);
        codes[code_word_offset(sh, n_heads, s, h, pos / kTokenBlock, g) + k] = (uint8_t)arg;
        if (sh.hb) {
            // The upper bits share a byte with other tokens, which other threads write: the bits are
            // replaced with atomics on the aligned 32-bit word that holds the byte.
            const int bit = k * sh.hb;
            const uintptr_t a = reinterpret_cast<uintptr_t>(codes) +
                                (uintptr_t)code_high_offset(sh, n_heads, s, h, pos / kTokenBlock, g) + (bit >> 3);
            unsigned int* w = reinterpret_cast<unsigned int*>(a & ~(uintptr_t)3);
            const int shift = (int)(a & 3) * 8 + (bit & 7);
            atomicAnd(w, ~((unsigned int)((1 << sh.hb) - 1) << shift));
            atomicOr(w, (unsigned int)(arg >> 8) << shift);
        }
    }
}

cudaError_t launch_encode_generic(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                  int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st)
{
    const int64_t total = sh.n_seq * sh.n_kv_heads * sh.G * n_tokens;
    if (total == 0) return cudaSuccess;
    const int threads = 256;
    const int64_t blocks = (total + threads - 1) / threads;
    const int64_t cap = (int64_t)device_sm_count() * 64;
    const int grid = (int)(blocks < cap ? blocks : cap);
    encode_generic_kernel<<<grid, threads, 0, st>>>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Encode of a few vectors per head (the append of a decode step).  One CTA per (head, group,
// run of 8 vectors): the group's codebook is staged in shared memory, channel-major, together
// with one vector per warp, and the lanes of a warp share the 2^b centroids.  Distances are
// formed exactly as in encode_generic_kernel; the lowest index wins ties.  The kernel is
// latency-bound, so everything it reads from global memory is requested before the one barrier.
// ------------------------------------------------------------------------------------------
constexpr int kSmallWarps = 8;
constexpr int kSmallVecPerCta = kSmallWarps;

__global__ void __launch_bounds__(kSmallWarps * 32)
encode_small_kernel(const __half* __restrict__ x, const float* __restrict__ cb, const int32_t* __restrict__ seq_offsets,
                    Shape sh, int64_t n_tokens, int64_t token_offset, uint8_t* __restrict__ codes)
{
    extern __shared__ __align__(16) float cbt[];            // [c][K], then [warps][c] for the vectors
    const int n_heads = sh.n_kv_heads;
    const int prob = blockIdx.x % (n_heads * sh.G);
    const int64_t run = blockIdx.x / (n_heads * sh.G);
    const int h = prob / sh.G, g = prob % sh.G;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* xs = cbt + sh.K * sh.c + warp * sh.c;
    const int64_t n_vec = sh.n_seq * n_tokens;
    const int64_t v = run * kSmallVecPerCta + warp;
    const int64_t s = v / n_tokens, i = v % n_tokens;
    int64_t pos = -1;
    const __half* xv = x + ((s * n_tokens + i) * n_heads + h) * (int64_t)sh.head_dim + g * sh.c;
    __half x_first = __float2half(0.f);          // requested now, stored after the codebook has been requested too
    if (v < n_vec) {
        pos = token_offset + (seq_offsets ? seq_offsets[s] : 0) + i;
        if (lane < sh.c) x_first = xv[lane];
    }
    const float* cg = cb + (int64_t)prob * sh.K * sh.c;
    for (int e = threadIdx.x; e < sh.K * sh.c; e += blockDim.x) cbt[(e % sh.c) * sh.K + e / sh.c] = cg[e];
    if (v < n_vec) {
        if (lane < sh.c) xs[lane] = __half2float(x_first);
        for (int k = lane + 32; k < sh.c; k += 32) xs[k] = __half2float(xv[k]);
    }
    __syncthreads();
    if (pos >= 0 && pos < sh.max_tokens) {                                  // same decision in every lane
        float best = INFINITY;
        int arg = 0;
        for (int j = lane; j < sh.K; j += 32) {
            float d = 0.f;
            for (int k = 0; k < sh.c; ++k) {
                const float diff = xs[k] - cbt[k * sh.K + j];
                d = fmaf(diff, diff, d);
            }
            if (d < best) {       // j rises: the lowest index of this lane wins ties
                best = d;
                arg = j;
            }
        }
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
            if (ob < best || (ob == best && oa < arg)) {
                best = ob;
                arg = oa;
            }
        }
        if (lane == 0) {
            const int k = (int)(pos % kTokenBlock);
            codes[code_word_offset(sh, n_heads, s, h, pos / kTokenBlock, g) + k] = (uint8_t)arg;
            if (sh.hb) {
                const int bit = k * sh.hb;
                const uintptr_t a = reinterpret_cast<uintptr_t>(codes) +
                                    (uintptr_t)code_high_offset(sh, n_heads, s, h, pos / kTokenBlock, g) + (bit >> 3);
                unsigned int* w = reinterpret_cast<unsigned int*>(a & ~(uintptr_t)3);
                const int shift = (int)(a & 3) * 8 + (bit & 7);
                atomicAnd(w, ~((unsigned int)((1 << sh.hb) - 1) << shift));
                atomicOr(w, (unsigned int)(arg >> 8) << shift);
            }
        }
    }
}

static size_t small_smem(const Shape& sh) { return (size_t)(sh.K + kSmallWarps) * sh.c * sizeof(float); }
bool encode_small_supported(const Shape& sh) { return small_smem(sh) <= 48 * 1024; }

cudaError_t launch_encode_small(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st)
{
    const int64_t n_vec = sh.n_seq * n_tokens;
    if (n_vec == 0) return cudaSuccess;
    const int64_t runs = (n_vec + kSmallVecPerCta - 1) / kSmallVecPerCta;
    const int64_t grid = runs * sh.n_kv_heads * sh.G;
    if (grid > 0x7fffffff) return cudaErrorInvalidValue;
    encode_small_kernel<<<(unsigned)grid, kSmallWarps * 32, small_smem(sh), st>>>(
        x, cb, seq_offsets, sh, n_tokens, token_offset, codes);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Layout converters between the library layout and [n_seq][max_tokens][n_heads][G].
// One thread per code word (16 tokens of one group).
// ------------------------------------------------------------------------------------------
__global__ void to_rowmajor_kernel(const uint8_t* __restrict__ codes, Shape sh, uint8_t* __restrict__ rm)
{
    const int n_heads = sh.n_kv_heads;
    const int64_t words = sh.n_seq * n_heads * sh.n_blocks * sh.G;
    for (int64_t w = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; w < words; w += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(w % sh.G);
        int64_t rest = w / sh.G;
        const int64_t blk = rest % sh.n_blocks;
        rest /= sh.n_blocks;
        const int h = (int)(rest % n_heads);
        const int64_t s = rest / n_heads;
        const uint8_t* block = codes + code_word_offset(sh, n_heads, s, h, blk, 0);
        for (int k = 0; k < kTokenBlock; ++k) {
            const int64_t t = blk * kTokenBlock + k;
            if (t >= sh.max_tokens) continue;
            const int code = read_code(block, sh, g, k);
            const int64_t e = ((s * sh.max_tokens + t) * n_heads + h) * sh.G + g;
            if (sh.hb) reinterpret_cast<uint16_t*>(rm)[e] = (uint16_t)code;
            else rm[e] = (uint8_t)code;
        }
    }
}

__global__ void from_rowmajor_kernel(const uint8_t* __restrict__ rm, Shape sh, uint8_t* __restrict__ codes)
{
    const int n_heads = sh.n_kv_heads;
    const int64_t words = sh.n_seq * n_heads * sh.n_blocks * sh.G;
    for (int64_t w = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; w < words; w += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(w % sh.G);
        int64_t rest = w / sh.G;
        const int64_t blk = rest % sh.n_blocks;
        rest /= sh.n_blocks;
        const int h = (int)(rest % n_heads);
        const int64_t s = rest / n_heads;
        uint8_t* dst = codes + code_word_offset(sh, n_heads, s, h, blk, g);
        uint8_t* dst_hi = codes + code_high_offset(sh, n_heads, s, h, blk, g);     // this thread owns the whole high word
        unsigned int hi_byte = 0;
        for (int k = 0; k < kTokenBlock; ++k) {
            const int64_t t = blk * kTokenBlock + k;
            const int64_t e = ((s * sh.max_tokens + t) * n_heads + h) * sh.G + g;
            int code = 0;
            if (t < sh.max_tokens) code = sh.hb ? (int)reinterpret_cast<const uint16_t*>(rm)[e] : (int)rm[e];
            dst[k] = (uint8_t)code;
            if (sh.hb) {
                const int bit = k * sh.hb;
                hi_byte |= (unsigned int)((code >> 8) & ((1 << sh.hb) - 1)) << (bit & 7);
                if (((bit + sh.hb) & 7) == 0) {
                    dst_hi[bit >> 3] = (uint8_t)hi_byte;
                    hi_byte = 0;
                }
            }
        }
    }
}

__global__ void add_one_kernel(const int32_t* __restrict__ src, int32_t* __restrict__ dst, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = src[i] + 1;
}

cudaError_t launch_add_one(const int32_t* src, int32_t* dst, int n, cudaStream_t st)
{
    add_one_kernel<<<(n + 255) / 256, 256, 0, st>>>(src, dst, n);
    return cudaGetLastError();
}

static int words_grid(const Shape& sh)
{
    const int64_t words = sh.n_seq * sh.n_kv_heads * sh.n_blocks * sh.G;
    const int64_t blocks = (words + 255) / 256;
    const int64_t cap = (int64_t)device_sm_count() * 32;
    return (int)(blocks < cap ? (blocks > 0 ? blocks : 1) : cap);
}

cudaError_t launch_to_rowmajor(const uint8_t* codes, const Shape& sh, uint8_t* rowmajor, cudaStream_t st)
{
    to_rowmajor_kernel<<<words_grid(sh), 256, 0, st>>>(codes, sh, rowmajor);
    return cudaGetLastError();
}

cudaError_t launch_from_rowmajor(const uint8_t* rowmajor, const Shape& sh, uint8_t* codes, cudaStream_t st)
{
    from_rowmajor_kernel<<<words_grid(sh), 256, 0, st>>>(rowmajor, sh, codes);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Decode attention, generic form.  One CTA per (context split, query head, sequence):
//   LUT[g][j] = scale*log2(e) * <q_g, Ck[g][j]>            (scores live in the log2 domain)
//   per tile of blockDim tokens: s_t = sum_g LUT[g][kcode], online max, p_t = 2^(s_t - m),
//   bins[g][vcode] += p_t (shared-memory float atomics)
//   acc[g*c+i] = sum_j bins[g][j] * Cv[g][j][i];  partial = (m, l, acc)
// The partials of all splits are merged by merge_kernel.
// ------------------------------------------------------------------------------------------
constexpr int kGenericThreads = 256;        // CTA size when several CTAs fit an SM
constexpr int kGenericThreadsMax = 1024;    // CTA size when the tables leave room for one CTA only

__device__ inline float block_reduce_max(float v, float* red)
{
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, red[w]);
    __syncthreads();
    return r;
}

__device__ inline float block_reduce_sum(float v, float* red)
{
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r += red[w];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kGenericThreadsMax)
decode_generic_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                      const float* __restrict__ kcb, const float* __restrict__ vcb,
                      const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int n_splits,
                      float* __restrict__ partials)
{
    extern __shared__ __align__(16) float smem_f[];
    float* lut = smem_f;                       // [G][K]
    float* bins = lut + sh.G * sh.K;           // [G][K]
    __shared__ float red[kGenericThreadsMax / 32];

    const int split = blockIdx.x % n_splits;
    const int hq = (blockIdx.x / n_splits) % sh.n_q_heads;
    const int64_t s = blockIdx.x / (n_splits * sh.n_q_heads);
    const int hkv = hq / sh.R;
    const int GK = sh.G * sh.K;

    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int64_t nblk = (n + kTokenBlock - 1) / kTokenBlock;
    const int64_t t_begin = nblk * split / n_splits * kTokenBlock;
    int64_t t_end = nblk * (split + 1) / n_splits * kTokenBlock;
    if (t_end > n) t_end = n;

    float* part = partials + ((s * sh.n_q_heads + hq) * n_splits + split) * (int64_t)partial_stride(sh.head_dim);
    if (t_end <= t_begin) {          // empty split: neutral element of the merge
        if (threadIdx.x == 0) { part[0] = -INFINITY; part[1] = 0.f; }
        for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) part[2 + d] = 0.f;
        return;
    }

    const __half* qv = q + (s * sh.n_q_heads + hq) * (int64_t)sh.head_dim;
    for (int e = threadIdx.x; e < GK; e += blockDim.x) {
        const int g = e / sh.K;
        const float* cj = kcb + ((int64_t)hkv * GK + e) * sh.c;
        float dot = 0.f;
        for (int k = 0; k < sh.c; ++k) dot = fmaf(__half2float(qv[g * sh.c + k]), cj[k], dot);
        lut[e] = dot * scale_log2e;
        bins[e] = 0.f;
    }
    __syncthreads();

    const uint8_t* kbase = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint8_t* vbase = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    float m_run = -INFINITY;
    float l_thr = 0.f;
    for (int64_t t0 = t_begin; t0 < t_end; t0 += blockDim.x) {
        const int64_t t = t0 + threadIdx.x;
        const bool valid = t < t_end;
        const int64_t block0 = (t / kTokenBlock) * sh.block_bytes;
        const int k16 = (int)(t % kTokenBlock);
        float sc = -INFINITY;
        if (valid) {
            sc = 0.f;
            for (int g = 0; g < sh.G; ++g) sc += lut[g * sh.K + read_code(kbase + block0, sh, g, k16)];
        }
        const float m_tile = block_reduce_max(sc, red);
        if (m_tile > m_run) {
            const float f = exp2f(m_run - m_tile);      // 0 when m_run is -inf
            for (int e = threadIdx.x; e < GK; e += blockDim.x) bins[e] *= f;
            l_thr *= f;
            m_run = m_tile;
            __syncthreads();
        }
        if (valid) {
            const float p = exp2f(sc - m_run);
            l_thr += p;
            for (int g = 0; g < sh.G; ++g) atomicAdd(&bins[g * sh.K + read_code(vbase + block0, sh, g, k16)], p);
        }
        __syncthreads();
    }
    const float l = block_reduce_sum(l_thr, red);
    if (threadIdx.x == 0) { part[0] = m_run; part[1] = l; }
    // bins x V centroids: a warp per output channel, its lanes share the code values
    for (int d = threadIdx.x >> 5; d < sh.head_dim; d += blockDim.x >> 5) {
        const int g = d / sh.c, k = d % sh.c;
        const float* cv = vcb + ((int64_t)hkv * GK + g * sh.K) * sh.c + k;
        float a = 0.f;
        for (int j = threadIdx.x & 31; j < sh.K; j += 32) a = fmaf(bins[g * sh.K + j], cv[j * sh.c], a);
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if ((threadIdx.x & 31) == 0) part[2 + d] = a;
    }
}

// ------------------------------------------------------------------------------------------
// Decode attention over codes of keys that were quantised BEFORE the rotary position embedding
// (last sentence of Section 3.2).  The key of Eq. 1 is the reconstruction rotated by its position,
// so the score is no longer a sum of per-(group, code) table entries: for the channel pair (a, b)
// with cosine cs and sine sn at the token's position,
//   q_a K_a + q_b K_b = cs (q_a k_a + q_b k_b) + sn (q_b k_a - q_a k_b),   k = reconstructed key.
// One thread per token gathers the token's centroids and forms that sum over the D/2 pairs; the
// V side, the online softmax and the partials are those of decode_generic_kernel.
// pairing 0: (a, b) = (i, i + D/2); pairing 1: (a, b) = (2i, 2i + 1).
// ------------------------------------------------------------------------------------------
constexpr int kRopeThreads = 1024;


__global__ void __launch_bounds__(kRopeThreads)
decode_rope_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                   const float* __restrict__ kcb, const float* __restrict__ vcb,
                   const int32_t* __restrict__ seq_lens, const float* __restrict__ rope_cos,
                   const float* __restrict__ rope_sin, int pairing, float scale_log2e, Shape sh, int n_splits,
                   int stage_codebook, float* __restrict__ partials)
{
    extern __shared__ __align__(16) float smem_f[];
    float* bins = smem_f;                      // [G][K]
    float* qsm = bins + sh.G * sh.K;           // [D]
    float* kcb_s = qsm + sh.head_dim;          // [G][K][c]: the KV head's key codebook, when it fits
    __shared__ float red[kRopeThreads / 32];
    __shared__ __align__(8) uint64_t book_bar;      // counts the bytes of the staged codebook

    const int split = blockIdx.x % n_splits;
    const int hq = (blockIdx.x / n_splits) % sh.n_q_heads;
    const int64_t s = blockIdx.x / (n_splits * sh.n_q_heads);
    const int hkv = hq / sh.R;
    const int GK = sh.G * sh.K;
    const int P = sh.head_dim / 2;

    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int64_t nblk = (n + kTokenBlock - 1) / kTokenBlock;
    const int64_t t_begin = nblk * split / n_splits * kTokenBlock;
    int64_t t_end = nblk * (split + 1) / n_splits * kTokenBlock;
    if (t_end > n) t_end = n;

    float* part = partials + ((s * sh.n_q_heads + hq) * n_splits + split) * (int64_t)partial_stride(sh.head_dim);
    if (t_end <= t_begin) {          // empty split: neutral element of the merge
        if (threadIdx.x == 0) { part[0] = -INFINITY; part[1] = 0.f; }
        for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) part[2 + d] = 0.f;
        return;
    }

    const __half* qv = q + (s * sh.n_q_heads + hq) * (int64_t)sh.head_dim;
    for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) qsm[d] = __half2float(qv[d]);
    for (int e = threadIdx.x; e < GK; e += blockDim.x) bins[e] = 0.f;
    const float* kcb_h = kcb + (int64_t)hkv * GK * sh.c;
    bool staged_late = false;                  // the staged copy did not arrive in time
    if (stage_codebook) {
        // Centroid gathers then come from shared memory.  One thread hands the copy to the bulk-copy
        // engine in pieces of 32 KiB.  If the barrier does not complete within its poll limit, the CTA
        // leaves the staging area alone and gathers from global memory instead (the copy may still be
        // writing there), and waits once more before it ends, so that no copy outlives the CTA.
        const uint32_t book_bytes = (uint32_t)GK * sh.c * sizeof(float);
        if (threadIdx.x == 0) {
            mbar_init(&book_bar, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            mbar_expect_tx(&book_bar, book_bytes);
            for (uint32_t off = 0; off < book_bytes; off += 32768u) {
                const uint32_t piece = book_bytes - off < 32768u ? book_bytes - off : 32768u;
                bulk_copy_g2s(reinterpret_cast<char*>(kcb_s) + off, reinterpret_cast<const char*>(kcb_h) + off, piece, &book_bar);
            }
        }
        staged_late = __syncthreads_or(mbar_wait(&book_bar, 0) ? 0 : 1) != 0;      // same decision in every thread
        if (!staged_late) kcb_h = kcb_s;
    }
    __syncthreads();

    const uint8_t* kbase = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint8_t* vbase = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    // 16-byte accesses need c and D/2 to be multiples of 4 and 16-byte aligned tables and codebooks
    const bool vec4 = sh.c % 4 == 0 && P % 4 == 0 &&
                      ((reinterpret_cast<uintptr_t>(rope_cos) | reinterpret_cast<uintptr_t>(rope_sin) |
                        reinterpret_cast<uintptr_t>(kcb_h)) & 15u) == 0;
    float m_run = -INFINITY;
    float l_thr = 0.f;
    for (int64_t t0 = t_begin; t0 < t_end; t0 += blockDim.x) {
        const int64_t t = t0 + threadIdx.x;
        const bool valid = t < t_end;
        const int64_t block0 = (t / kTokenBlock) * sh.block_bytes;
        const int k16 = (int)(t % kTokenBlock);
        float sc = -INFINITY;
        if (valid) {
            const float* cs = rope_cos + t * P;
            const float* sn = rope_sin + t * P;
            float acc = 0.f;
            if (pairing == 0 && vec4) {
                // Four pairs per 16-byte load of the token's cos / sin row and of the two centroids; the
                // loads of 32 pairs are issued together, since their latency is what this loop waits for.
                constexpr int kAhead = 4;
                const int half_groups = sh.G / 2;
                for (int i0 = 0; i0 < P; i0 += 4 * kAhead) {
                    float4 c4[kAhead], s4[kAhead];
#pragma unroll
                    for (int u = 0; u < kAhead; ++u)
                        if (i0 + 4 * u < P) {
                            c4[u] = *reinterpret_cast<const float4*>(cs + i0 + 4 * u);
                            s4[u] = *reinterpret_cast<const float4*>(sn + i0 + 4 * u);
                        }
#pragma unroll
                    for (int u = 0; u < kAhead; ++u) {
                        const int i = i0 + 4 * u;
                        if (i >= P) break;
                        const int g = i / sh.c, k = i % sh.c;
                        const float* ca = kcb_h + ((int64_t)g * sh.K + read_code(kbase + block0, sh, g, k16)) * sh.c;
                        const float* cb2 = kcb_h + ((int64_t)(g + half_groups) * sh.K +
                                                    read_code(kbase + block0, sh, g + half_groups, k16)) * sh.c;
                        const float4 a4 = *reinterpret_cast<const float4*>(ca + k);
                        const float4 b4 = *reinterpret_cast<const float4*>(cb2 + k);
                        const float4 qa4 = *reinterpret_cast<const float4*>(qsm + i);
                        const float4 qb4 = *reinterpret_cast<const float4*>(qsm + i + P);
                        acc = fmaf(c4[u].x, fmaf(qa4.x, a4.x, qb4.x * b4.x), acc);
                        acc = fmaf(s4[u].x, fmaf(qb4.x, a4.x, -qa4.x * b4.x), acc);
                        acc = fmaf(c4[u].y, fmaf(qa4.y, a4.y, qb4.y * b4.y), acc);
                        acc = fmaf(s4[u].y, fmaf(qb4.y, a4.y, -qa4.y * b4.y), acc);
                        acc = fmaf(c4[u].z, fmaf(qa4.z, a4.z, qb4.z * b4.z), acc);
                        acc = fmaf(s4[u].z, fmaf(qb4.z, a4.z, -qa4.z * b4.z), acc);
                        acc = fmaf(c4[u].w, fmaf(qa4.w, a4.w, qb4.w * b4.w), acc);
                        acc = fmaf(s4[u].w, fmaf(qb4.w, a4.w, -qa4.w * b4.w), acc);
                    }
                }
            } else if (pairing == 0) {
                const int half_groups = sh.G / 2;
                for (int g = 0; g < half_groups; ++g) {
                    const float* ca = kcb_h + ((int64_t)g * sh.K + read_code(kbase + block0, sh, g, k16)) * sh.c;
                    const float* cb2 = kcb_h + ((int64_t)(g + half_groups) * sh.K +
                                                read_code(kbase + block0, sh, g + half_groups, k16)) * sh.c;
                    for (int k = 0; k < sh.c; ++k) {
                        const int i = g * sh.c + k;
                        const float ka = ca[k], kb = cb2[k], qa = qsm[i], qb = qsm[i + P];
                        acc = fmaf(cs[i], fmaf(qa, ka, qb * kb), acc);
                        acc = fmaf(sn[i], fmaf(qb, ka, -qa * kb), acc);
                    }
                }
            } else {
                for (int g = 0; g < sh.G; ++g) {
                    const float* cg = kcb_h + ((int64_t)g * sh.K + read_code(kbase + block0, sh, g, k16)) * sh.c;
                    for (int k = 0; k < sh.c; k += 2) {
                        const int a = g * sh.c + k, i = a >> 1;
                        const float ka = cg[k], kb = cg[k + 1], qa = qsm[a], qb = qsm[a + 1];
                        acc = fmaf(cs[i], fmaf(qa, ka, qb * kb), acc);
                        acc = fmaf(sn[i], fmaf(qb, ka, -qa * kb), acc);
                    }
                }
            }
            sc = acc * scale_log2e;
        }
        const float m_tile = block_reduce_max(sc, red);
        if (m_tile > m_run) {
            const float f = exp2f(m_run - m_tile);      // 0 when m_run is -inf
            for (int e = threadIdx.x; e < GK; e += blockDim.x) bins[e] *= f;
            l_thr *= f;
            m_run = m_tile;
            __syncthreads();
        }
        if (valid) {
            const float p = exp2f(sc - m_run);
            l_thr += p;
            for (int g = 0; g < sh.G; ++g) atomicAdd(&bins[g * sh.K + read_code(vbase + block0, sh, g, k16)], p);
        }
        __syncthreads();
    }
    const float l = block_reduce_sum(l_thr, red);
    if (threadIdx.x == 0) { part[0] = m_run; part[1] = l; }
    // bins x V centroids: a warp per output channel, its lanes share the code values
    for (int d = threadIdx.x >> 5; d < sh.head_dim; d += blockDim.x >> 5) {
        const int g = d / sh.c, k = d % sh.c;
        const float* cv = vcb + ((int64_t)hkv * GK + g * sh.K) * sh.c + k;
        float a = 0.f;
        for (int j = threadIdx.x & 31; j < sh.K; j += 32) a = fmaf(bins[g * sh.K + j], cv[j * sh.c], a);
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if ((threadIdx.x & 31) == 0) part[2 + d] = a;
    }
    // a staged copy that was late must have landed before the CTA's shared memory is given up
    if (staged_late) mbar_wait(&book_bar, 0);
}

int decode_generic_splits(const Shape& sh)
{
    // enough CTAs for a few waves of the SMs, at least 256 tokens per split
    const int64_t items = sh.n_seq * sh.n_q_heads;
    int64_t want = ((int64_t)device_sm_count() * 8 + items - 1) / (items > 0 ? items : 1);
    const int64_t cap = (sh.max_tokens + 255) / 256;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    return (int)want;
}

// out[d] = sum_p 2^(m_p - M) acc_p[d] / sum_p 2^(m_p - M) l_p,  M = max_p m_p  (log-sum-exp merge)
__global__ void merge_kernel(const float* __restrict__ partials, int n_parts, Shape sh, float* __restrict__ out)
{
    const int hq = blockIdx.x % sh.n_q_heads;
    const int64_t s = blockIdx.x / sh.n_q_heads;
    const int stride = partial_stride(sh.head_dim);
    const float* base = partials + (s * sh.n_q_heads + hq) * (int64_t)n_parts * stride;
    float M = -INFINITY;
    for (int p = 0; p < n_parts; ++p) M = fmaxf(M, base[p * stride]);
    float* o = out + (s * sh.n_q_heads + hq) * (int64_t)sh.head_dim;
    if (M == -INFINITY) {           // empty context
        for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) o[d] = 0.f;
        return;
    }
    float L = 0.f;
    for (int p = 0; p < n_parts; ++p) {
        const float m = base[p * stride];
        if (m != -INFINITY) L += exp2f(m - M) * base[p * stride + 1];
    }
    for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) {
        float a = 0.f;
        for (int p = 0; p < n_parts; ++p) {
            const float m = base[p * stride];
            if (m != -INFINITY) a = fmaf(exp2f(m - M), base[p * stride + 2 + d], a);
        }
        o[d] = a / L;
    }
}

cudaError_t launch_merge(const float* partials, int n_parts, const Shape& sh, float* out, cudaStream_t st)
{
    const unsigned grid = (unsigned)(sh.n_q_heads * sh.n_seq);
    merge_kernel<<<grid, 128, 0, st>>>(partials, n_parts, sh, out);
    return cudaGetLastError();
}

cudaError_t launch_decode_generic(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                  const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                  float* out, float* partials, cudaStream_t st)
{
    int n_splits = decode_generic_splits(sh);
    const size_t smem = (size_t)2 * sh.G * sh.K * sizeof(float);
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_generic_kernel), (int)smem, 32);
    if (e != cudaSuccess) return e;
    // tables of more than a third of an SM's shared memory: fewer, larger CTAs keep the SM's warps busy
    const int threads = smem > 72 * 1024 ? (smem > 110 * 1024 ? kGenericThreadsMax : 512) : kGenericThreads;
    if (threads == kGenericThreadsMax) {
        // one CTA per SM, each paying a table build over the whole codebook: split the contexts only as far
        // as two CTAs per SM need it (never into more partial slots than the workspace holds)
        const int64_t items = sh.n_seq * sh.n_q_heads;
        int64_t want = (2 * (int64_t)device_sm_count() + items - 1) / items;
        const int64_t cap = (sh.max_tokens + threads - 1) / threads;
        if (want > cap) want = cap;
        if (want < 1) want = 1;
        if (want < n_splits) n_splits = (int)want;
    }
    const unsigned grid = (unsigned)(n_splits * sh.n_q_heads * sh.n_seq);
    decode_generic_kernel<<<grid, threads, smem, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh,
                                                               n_splits, partials);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_merge(partials, n_splits, sh, out, st);
}

cudaError_t launch_decode_rope(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                               const float* vcb, const int32_t* seq_lens, const float* rope_cos, const float* rope_sin,
                               int pairing, float scale, const Shape& sh, float* out, float* partials, cudaStream_t st)
{
    // One CTA fills an SM and stages a codebook, so contexts are split only as far as the SMs need it
    // (and never into more partial slots than the workspace holds: those of decode_generic_splits).
    int n_splits = decode_generic_splits(sh);
    {
        const int64_t items = sh.n_seq * sh.n_q_heads;
        int64_t want = (2 * (int64_t)device_sm_count() + items - 1) / items;
        const int64_t cap = (sh.max_tokens + kRopeThreads - 1) / kRopeThreads;
        if (want > cap) want = cap;
        if (want < 1) want = 1;
        if (want < n_splits) n_splits = (int)want;
    }
    size_t smem = ((size_t)sh.G * sh.K + sh.head_dim) * sizeof(float);
    const size_t book = (size_t)sh.G * sh.K * sh.c * sizeof(float);
    // the staged copy starts after the bins and the query and moves 16-byte pieces: both must be 16-byte multiples
    const int stage = (sh.G * sh.K + sh.head_dim) % 4 == 0 && (sh.G * sh.K * sh.c) % 4 == 0 &&
                      smem + book <= (size_t)220 * 1024;
    if (stage) smem += book;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_rope_kernel), (int)smem, 33);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(n_splits * sh.n_q_heads * sh.n_seq);
    decode_rope_kernel<<<grid, kRopeThreads, smem, st>>>(q, kc, vc, kcb, vcb, seq_lens, rope_cos, rope_sin, pairing,
                                                         scale * kLog2e, sh, n_splits, stage, partials);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_merge(partials, n_splits, sh, out, st);
}

}  // namespace cq
