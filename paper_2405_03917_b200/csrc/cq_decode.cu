// Tuned decode-attention kernels for head_dim 128, b = 8 (one byte per code).
//
// Formulation (an exact re-association of Eq. 1 of the paper with K and V replaced by
// their CQ reconstructions, Section 3.2):
//   LUT[h][g][j]  = scale*log2(e) * <q_h,g , Ck[g][j]>          per-query table, shared memory
//   s_t[h]        = sum_g LUT[h][g][kcode[t][g]]                scores, log2 domain
//   w_t[h]        = round(2^(s_t[h] - e))                       integer softmax weight, unit 2^e
//   bins[h][g][j] += w_t[h]   for j = vcode[t][g]               integer bins, shared memory
//   acc[h][g*c+i] = sum_j bins[h][g][j] * Cv[g][j][i],  l[h] = sum_j bins[h][0][j]
// and the partial (e, l, acc) of every context chunk goes to the log-sum-exp merge.
//
// Why integers: on sm_100a a shared-memory `red.add.u32` retires a warp's 32 bank-distinct
// updates in about one cycle, while the f32 / f16x2 / u64 forms run several times slower.
// Integer adds are also associative, so the result does not depend on the order in which
// warps reach a bin.  The unit exponent e is kept at least 26 bits below the running maximum
// score and is coarsened (bins shifted right, with rounding) whenever a score would need more
// than 30 bits or a bin could overflow 32 bits; both events are rare and cost one pass over
// the bins.
//
// Shared-memory traffic, not HBM, is what limits this kernel once the code stream is
// coalesced: each (token, group, query head) costs one 4-byte table lookup and one 4-byte
// bin update.  The tables are therefore laid out so that every warp instruction touches 32
// distinct banks whatever the codes are:
//   row j (256 bytes) of a table holds, for code value j, 32-word "planes"; word w of a
//   plane belongs to one (group, query head | replica) pair, and lane (r, p) = (lane/4,
//   lane%4) of a warp uses word  16*(r/4) + 4*((r+m)%4) + p  (16 groups) or
//   4*((r+m)%8) + p  (32 groups) for its m-th code word, which is a bijection lanes ->
//   banks for every m.
// A lane quad r owns one 16-token block; lane p of the quad owns the groups congruent to
// p mod 4.  Table entries are stored as half2 (hi, lo) pairs, so a looked-up word is
// directly one register of an m16n8k16 A fragment: an MMA against an all-ones B matrix
// sums the quad's lookups (all groups of a token) in fp32 and leaves the token's score in
// every lane of the quad, which is exactly where the V-side bin updates need it.
#include "cq_common.cuh"

namespace cq {

namespace {

constexpr int kRows = 256;            // code values
constexpr int kRowBytes = 256;        // bytes per table row
constexpr int kUnitBits = 27;         // weight of the running-maximum token: (2^26, 2^27]
constexpr int kMaxWeightBits = 30;    // a score may exceed the unit exponent by at most this

template <int G, int R>
struct Cfg {
    static_assert(G == 16 || G == 32, "tuned decode kernels cover 16 and 32 groups");
    static constexpr int kC = 128 / G;                                  // channels per group
    static constexpr bool kHalfRows = (G == 16);                         // quads 0-3 / 4-7 use different 16-word halves
    static constexpr bool kReplica = (G == 16 && R == 1);                // the two halves are copies of one table
    static constexpr int kLaneHeads = (G == 16 && R >= 2) ? R / 2 : R;   // query heads a lane serves
    static constexpr int kPlanes = kLaneHeads;                           // 32-word planes per table row
    static constexpr int kSlots = G / 4;                                 // code words (16 tokens each) per lane
    static constexpr int kBlocksPerIter = (G == 16 && R >= 2) ? 4 : 8;   // 16-token blocks per warp iteration
    static constexpr int kWarps = (kPlanes == 1) ? 8 : 16;
    static constexpr int kThreads = kWarps * 32;
    static constexpr int kMinBlocks = (kPlanes == 1) ? (G == 16 ? 3 : 2) : 1;
    static constexpr int kRoundTokens = kWarps * kBlocksPerIter * 16;    // tokens a CTA handles per iteration
    static_assert(kPlanes == 1 || kPlanes == 2, "table rows hold one or two planes");
    // One plane: K and V planes share a row (K at +0, V at +128).  Two planes: separate tables.
    static constexpr int kVOffset = (kPlanes == 1) ? 128 : kRows * kRowBytes;
    static constexpr int kTableBytes = (kPlanes == 1) ? kRows * kRowBytes : 2 * kRows * kRowBytes;
    static constexpr int kCtlBytes = 64 + R * 128 * 4;                   // control words + scaled query
    static constexpr int kSmemBytes = kTableBytes + kCtlBytes;

    // word inside a plane that lane (r, p) uses for its m-th code word
    __device__ static __forceinline__ int word(int r, int p, int m)
    {
        return kHalfRows ? 16 * (r >> 2) + 4 * ((r + m) & 3) + p : 4 * ((r + m) & 7) + p;
    }
    // group / query head (relative to the KV head's first query head) of a table word
    __device__ static __forceinline__ int group_of(int w) { return kHalfRows ? (w & 15) : w; }
    __device__ static __forceinline__ int head_of(int plane, int w)
    {
        if (!kHalfRows) return plane;
        if (R == 1) return 0;
        return 2 * plane + (w >> 4);
    }
};

struct Ctl {
    int rmax[3];        // per-iteration maximum score of the CTA (order-preserving int encoding)
    float lut_absmax;   // largest |LUT| entry, as float bits (non-negative, so int order works)
};

__device__ __forceinline__ int enc_float(float f)
{
    const int i = __float_as_int(f);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float dec_float(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

__device__ __forceinline__ uint4 ldg_codes(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// D += A * ones: sums, per fragment row, the 16 halves the quad holds for that row.
__device__ __forceinline__ void mma_rowsum(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3)
{
    const uint32_t ones = 0x3c003c00u;   // half2(1, 1)
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(ones), "r"(ones));
}

// byte `k` (0..15) of a 16-byte code word
__device__ __forceinline__ uint32_t word32(const uint4& w, int k)
{
    return (k >> 2) == 0 ? w.x : (k >> 2) == 1 ? w.y : (k >> 2) == 2 ? w.z : w.w;
}
// table byte offset code*256 + lane_off for token k of a code word (lane_off < 256)
__device__ __forceinline__ uint32_t row_index(const uint4& w, int k, uint32_t lane_off)
{
    return __byte_perm(word32(w, k), lane_off, 0x5504u | ((uint32_t)(k & 3) << 4));
}

template <int G, int R>
__global__ void __launch_bounds__(Cfg<G, R>::kThreads, Cfg<G, R>::kMinBlocks)
decode_tuned_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                    const float* __restrict__ kcb, const float* __restrict__ vcb,
                    const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int chunk_tokens, int n_parts,
                    float* __restrict__ partials)
{
    using C = Cfg<G, R>;
    constexpr int kC = C::kC;
    extern __shared__ __align__(1024) uint8_t smem[];
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + C::kTableBytes);
    float* qs = reinterpret_cast<float*>(smem + C::kTableBytes + 64);      // [R][128], scaled by scale*log2(e)

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, p = lane & 3;

    // work item: (context part, sequence, KV head); parts are the slowest index so that the
    // always-populated first parts start first
    const int hkv = blockIdx.x % sh.n_kv_heads;
    const int64_t s = (blockIdx.x / sh.n_kv_heads) % sh.n_seq;
    const int part = (int)(blockIdx.x / (sh.n_kv_heads * sh.n_seq));

    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int64_t t_begin = (int64_t)part * chunk_tokens;
    const int64_t t_end = (t_begin + chunk_tokens < n) ? t_begin + chunk_tokens : n;
    const int stride = partial_stride(128);
    float* part_base = partials + ((s * sh.n_q_heads + (int64_t)hkv * R) * n_parts + part) * stride;
    // partial of query head hkv*R + h: part_base + h * n_parts * stride
    if (t_begin >= t_end) {
        for (int i = threadIdx.x; i < R * stride; i += C::kThreads) {
            const int h = i / stride, d = i % stride;
            part_base[(int64_t)h * n_parts * stride + d] = d == 0 ? -INFINITY : 0.f;
        }
        return;
    }

    // ---------------------------------------------------------------- set-up: query, LUT, bins
    if (threadIdx.x < 3) ctl->rmax[threadIdx.x] = INT_MIN;
    if (threadIdx.x == 3) ctl->lut_absmax = 0.f;
    for (int i = threadIdx.x; i < R * 128; i += C::kThreads)
        qs[i] = __half2float(q[(s * sh.n_q_heads + (int64_t)hkv * R) * 128 + i]) * scale_log2e;
    __syncthreads();

    // lane `lane` fills word `lane` of every plane, for the code values j = warp, warp + kWarps, ...
    {
        float absmax = 0.f;
        const int g = C::group_of(lane);
        float qreg[C::kPlanes][kC];
#pragma unroll
        for (int pl = 0; pl < C::kPlanes; ++pl)
#pragma unroll
            for (int i = 0; i < kC; ++i) qreg[pl][i] = qs[C::head_of(pl, lane) * 128 + g * kC + i];
        const float* cg = kcb + ((int64_t)hkv * G + g) * kRows * kC;
#pragma unroll 4
        for (int j = warp; j < kRows; j += C::kWarps) {
            float cv[kC];
            if (kC == 8) {
                const float4 a = *reinterpret_cast<const float4*>(cg + j * 8);
                const float4 b = *reinterpret_cast<const float4*>(cg + j * 8 + 4);
                cv[0] = a.x; cv[1] = a.y; cv[2] = a.z; cv[3] = a.w;
                cv[4 % kC] = b.x; cv[5 % kC] = b.y; cv[6 % kC] = b.z; cv[7 % kC] = b.w;
            } else {
                const float4 a = *reinterpret_cast<const float4*>(cg + j * 4);
                cv[0] = a.x; cv[1] = a.y; cv[2] = a.z; cv[3] = a.w;
            }
#pragma unroll
            for (int pl = 0; pl < C::kPlanes; ++pl) {
                float dot = 0.f;
#pragma unroll
                for (int i = 0; i < kC; ++i) dot = fmaf(qreg[pl][i], cv[i], dot);
                absmax = fmaxf(absmax, fabsf(dot));
                *reinterpret_cast<float*>(smem + j * kRowBytes + pl * 128 + lane * 4) = dot;
                *reinterpret_cast<uint32_t*>(smem + C::kVOffset + j * kRowBytes + pl * 128 + lane * 4) = 0u;
            }
        }
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 16));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 8));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 4));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 2));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 1));
        if (lane == 0) atomicMax(reinterpret_cast<int*>(&ctl->lut_absmax), __float_as_int(absmax));
    }
    __syncthreads();
    // Entries become half2 (hi, lo) of LUT * 2^-kexp, with kexp chosen so that |hi| < 2^15.
    int kexp = 0;
    {
        int ex;
        frexpf(ctl->lut_absmax, &ex);            // absmax < 2^ex
        kexp = ex > 15 ? ex - 15 : 0;
    }
    const float lut_scale = exp2f((float)kexp);     // scores in table units * lut_scale = log2-domain scores
    {
        const float inv = exp2f(-(float)kexp);
#pragma unroll 4
        for (int j = warp; j < kRows; j += C::kWarps)
#pragma unroll
            for (int pl = 0; pl < C::kPlanes; ++pl) {
                uint32_t* e = reinterpret_cast<uint32_t*>(smem + j * kRowBytes + pl * 128 + lane * 4);
                const float v = __uint_as_float(*e) * inv;
                const __half hi = __float2half_rn(v);
                const __half lo = __float2half_rn(v - __half2float(hi));
                *e = (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
            }
    }
    __syncthreads();

    // ---------------------------------------------------------------- main loop over the chunk
    const int64_t blk0 = t_begin / kTokenBlock;
    const int64_t blk_lim = (t_end + kTokenBlock - 1) / kTokenBlock;       // blocks holding a valid token
    const int n_iters = (int)((t_end - t_begin + C::kRoundTokens - 1) / C::kRoundTokens);
    const int qb = (C::kBlocksPerIter == 8) ? r : (r & 3);                 // block of this quad inside the warp's iteration
    const uint4* kbase = reinterpret_cast<const uint4*>(kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0));
    const uint4* vbase = reinterpret_cast<const uint4*>(vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0));

    uint32_t lane_off[C::kSlots];      // byte offset of this lane's word inside a plane, per code word
    int slot_group[C::kSlots];
#pragma unroll
    for (int m = 0; m < C::kSlots; ++m) {
        const int w = C::word(r, p, m);
        lane_off[m] = 4u * w;
        slot_group[m] = C::group_of(w);
    }

    uint4 kw[C::kSlots], vw[C::kSlots];
    auto load_words = [&](uint4 (&dst)[C::kSlots], const uint4* base, int64_t blk) {
        if (blk < blk_lim) {
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m) dst[m] = ldg_codes(base + blk * G + slot_group[m]);
        } else {
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m) dst[m] = make_uint4(0u, 0u, 0u, 0u);
        }
    };

    float e_unit = -INFINITY;              // log2 of the weight unit; integer-valued once set
    unsigned long long bin_bound = 0;      // upper bound on every bin
    load_words(kw, kbase, blk0 + (int64_t)warp * C::kBlocksPerIter + qb);

    for (int it = 0; it < n_iters; ++it) {
        const int64_t blk = blk0 + ((int64_t)it * C::kWarps + warp) * C::kBlocksPerIter + qb;
        load_words(vw, vbase, blk);

        // K side: scores of this quad's 16 tokens, for the query heads this lane serves
        float sc[C::kLaneHeads][16];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj)
#pragma unroll
            for (int u = 0; u < C::kLaneHeads; ++u) {
                float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int m = 0; m < C::kSlots; m += 2) {
                    const uint32_t a0 = *reinterpret_cast<const uint32_t*>(smem + u * 128 + row_index(kw[m], jj, lane_off[m]));
                    const uint32_t a1 = *reinterpret_cast<const uint32_t*>(smem + u * 128 + row_index(kw[m], jj + 8, lane_off[m]));
                    const uint32_t a2 = *reinterpret_cast<const uint32_t*>(smem + u * 128 + row_index(kw[m + 1], jj, lane_off[m + 1]));
                    const uint32_t a3 = *reinterpret_cast<const uint32_t*>(smem + u * 128 + row_index(kw[m + 1], jj + 8, lane_off[m + 1]));
                    mma_rowsum(d, a0, a1, a2, a3);
                }
                sc[u][jj] = d[0];
                sc[u][jj + 8] = d[2];
            }

        // mask tokens past the end of the context, take the maximum
        const int64_t tok0 = blk * kTokenBlock;
        float mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < 16; ++k)
#pragma unroll
            for (int u = 0; u < C::kLaneHeads; ++u) {
                const float v = (tok0 + k < t_end) ? sc[u][k] * lut_scale : -INFINITY;
                sc[u][k] = v;
                mx = fmaxf(mx, v);
            }
        const int wmax = __reduce_max_sync(0xffffffffu, enc_float(mx));
        if (lane == 0) atomicMax(&ctl->rmax[it % 3], wmax);
        __syncthreads();
        const float round_max = dec_float(ctl->rmax[it % 3]);
        if (threadIdx.x == 0) ctl->rmax[(it + 2) % 3] = INT_MIN;

        // the next iteration's K words travel while the V side runs
        load_words(kw, kbase, blk + (int64_t)C::kWarps * C::kBlocksPerIter);

        if (round_max > -INFINITY) {
            // unit exponent for this round (every thread computes the same values)
            const float cm = ceilf(round_max);
            float e_new = e_unit;
            if (!(cm - e_unit <= (float)kMaxWeightBits)) e_new = cm - (float)kUnitBits;
            unsigned long long bound;
            for (;;) {
                const float shf = e_new - e_unit;                                     // >= 0, +inf on first use
                bound = (shf >= 64.f) ? 0ull : (bin_bound >> (int)shf);
                const float dexp = cm - e_new;                                        // <= kMaxWeightBits
                const unsigned long long wtop = dexp <= 0.f ? 1ull : (1ull << (int)dexp);
                bound += 1ull + (unsigned long long)C::kRoundTokens * (wtop + (wtop >> 20) + 1ull);
                if (bound < (1ull << 32)) break;
                e_new += 2.f;
            }
            if (e_new > e_unit && e_unit > -INFINITY) {
                const float shf = e_new - e_unit;
                const int k = shf >= 32.f ? 32 : (int)shf;
                for (int i = threadIdx.x; i < kRows * 32 * C::kPlanes; i += C::kThreads) {
                    uint32_t* bp = reinterpret_cast<uint32_t*>(smem + C::kVOffset + (i / (32 * C::kPlanes)) * kRowBytes +
                                                               (i % (32 * C::kPlanes)) * 4);
                    const uint32_t v = *bp;
                    *bp = k >= 32 ? 0u : (v >> k) + ((v >> (k - 1)) & 1u);
                }
                __syncthreads();
            }
            e_unit = e_new;
            bin_bound = bound;

            // V side: integer weights into the bins of this lane's groups
#pragma unroll
            for (int k = 0; k < 16; ++k)
#pragma unroll
                for (int u = 0; u < C::kLaneHeads; ++u) {
                    const uint32_t w = __float2uint_rn(ex2(sc[u][k] - e_unit));
#pragma unroll
                    for (int m = 0; m < C::kSlots; ++m)
                        atomicAdd(reinterpret_cast<unsigned int*>(smem + C::kVOffset + u * 128 +
                                                                  row_index(vw[m], k, lane_off[m])), w);
                }
        }
    }
    __syncthreads();

    // ---------------------------------------------------------------- epilogue: bins x V centroids
    // lane `lane` owns word `lane` of every plane and sums over the code values of its warp.
    {
        const int g = C::group_of(lane);
        const float* cg = vcb + ((int64_t)hkv * G + g) * kRows * kC;
        float acc[C::kPlanes][kC];
        float lsum[C::kPlanes];
#pragma unroll
        for (int pl = 0; pl < C::kPlanes; ++pl) {
            lsum[pl] = 0.f;
#pragma unroll
            for (int i = 0; i < kC; ++i) acc[pl][i] = 0.f;
        }
#pragma unroll 4
        for (int j = warp; j < kRows; j += C::kWarps) {
            float cv[kC];
            if (kC == 8) {
                const float4 a = *reinterpret_cast<const float4*>(cg + j * 8);
                const float4 b = *reinterpret_cast<const float4*>(cg + j * 8 + 4);
                cv[0] = a.x; cv[1] = a.y; cv[2] = a.z; cv[3] = a.w;
                cv[4 % kC] = b.x; cv[5 % kC] = b.y; cv[6 % kC] = b.z; cv[7 % kC] = b.w;
            } else {
                const float4 a = *reinterpret_cast<const float4*>(cg + j * 4);
                cv[0] = a.x; cv[1] = a.y; cv[2] = a.z; cv[3] = a.w;
            }
#pragma unroll
            for (int pl = 0; pl < C::kPlanes; ++pl) {
                const float bv = (float)*reinterpret_cast<const uint32_t*>(smem + C::kVOffset + j * kRowBytes + pl * 128 + lane * 4);
                lsum[pl] += bv;
#pragma unroll
                for (int i = 0; i < kC; ++i) acc[pl][i] = fmaf(bv, cv[i], acc[pl][i]);
            }
        }
        if (C::kReplica) {       // the two halves of the plane are partial sums of the same bins
#pragma unroll
            for (int i = 0; i < kC; ++i) acc[0][i] += __shfl_xor_sync(0xffffffffu, acc[0][i], 16);
            lsum[0] += __shfl_xor_sync(0xffffffffu, lsum[0], 16);
        }
        __syncthreads();         // every warp is done reading the K table region reused below
        // scratch (over the K table rows, which are no longer needed): [warp][plane][lane][kC + 1]
        float* scratch = reinterpret_cast<float*>(smem);
        static_assert(C::kWarps * C::kPlanes * 32 * (kC + 1) * 4 <= C::kTableBytes, "scratch must fit the tables");
        // The scratch overwrites table rows (with one plane, bins included): the barrier above
        // guarantees that every bin has been read.
#pragma unroll
        for (int pl = 0; pl < C::kPlanes; ++pl) {
            float* dst = scratch + ((warp * C::kPlanes + pl) * 32 + lane) * (kC + 1);
#pragma unroll
            for (int i = 0; i < kC; ++i) dst[i] = acc[pl][i];
            dst[kC] = lsum[pl];
        }
        __syncthreads();
        // one thread per (query head, channel): sum the warps' partial sums, write the partial
        for (int o = threadIdx.x; o < R * 130; o += C::kThreads) {
            const int h = o / 130, d = o % 130;
            float* dstp = part_base + (int64_t)h * n_parts * stride;
            if (d == 0) {
                dstp[0] = e_unit;                 // reference exponent of this partial (log2 domain)
                continue;
            }
            // word / plane that holds (head h, group gg)
            const int gg = d == 1 ? 0 : (d - 2) / kC;
            const int ch = d == 1 ? kC : (d - 2) % kC;
            int pl, w;
            if (C::kHalfRows) {
                pl = (R <= 2) ? 0 : h / 2;
                w = (R == 1 ? 0 : (h & 1) * 16) + gg;
            } else {
                pl = h;
                w = gg;
            }
            float sum = 0.f;
#pragma unroll
            for (int wp = 0; wp < C::kWarps; ++wp) sum += scratch[((wp * C::kPlanes + pl) * 32 + w) * (kC + 1) + ch];
            dstp[d] = sum;
        }
    }
}

template <int G, int R>
cudaError_t launch_cfg(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                       const int32_t* seq_lens, float scale, const Shape& sh, int chunk_tokens, int n_parts,
                       float* partials, cudaStream_t st)
{
    using C = Cfg<G, R>;
    cudaError_t e = cudaFuncSetAttribute(decode_tuned_kernel<G, R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         C::kSmemBytes);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(sh.n_seq * sh.n_kv_heads * n_parts);
    decode_tuned_kernel<G, R><<<grid, C::kThreads, C::kSmemBytes, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh,
                                                                        chunk_tokens, n_parts, partials);
    return cudaGetLastError();
}

// Context chunk per CTA: a multiple of the CTA's round, at least 2048 tokens, small enough for
// about eight CTA waves on 148 SMs when the batch allows it.
template <int G, int R>
int chunk_for(const Shape& sh)
{
    using C = Cfg<G, R>;
#ifdef CQ_TUNE_CHUNK_TOKENS
    return CQ_TUNE_CHUNK_TOKENS;
#endif
    const int64_t items = sh.n_seq * sh.n_kv_heads;
    const int64_t slots = 148 * C::kMinBlocks;
    int64_t splits = (slots * 8 + items - 1) / items;
    int64_t chunk = (sh.max_tokens + splits - 1) / splits;
    if (chunk < 2048) chunk = 2048;
    chunk = (chunk + C::kRoundTokens - 1) / C::kRoundTokens * C::kRoundTokens;
    return (int)chunk;
}

int chunk_dispatch(const Shape& sh)
{
    if (sh.G == 16 && sh.R == 1) return chunk_for<16, 1>(sh);
    if (sh.G == 16 && sh.R == 2) return chunk_for<16, 2>(sh);
    if (sh.G == 16 && sh.R == 4) return chunk_for<16, 4>(sh);
    if (sh.G == 32 && sh.R == 1) return chunk_for<32, 1>(sh);
    if (sh.G == 32 && sh.R == 2) return chunk_for<32, 2>(sh);
    return 0;
}

}  // namespace

bool decode_tuned_supported(const Shape& sh)
{
    if (sh.head_dim != 128 || sh.b != 8) return false;
    if (sh.max_tokens > ((int64_t)1 << 30)) return false;
    return (sh.G == 16 && (sh.R == 1 || sh.R == 2 || sh.R == 4)) || (sh.G == 32 && (sh.R == 1 || sh.R == 2));
}

int decode_tuned_parts(const Shape& sh)
{
    const int chunk = chunk_dispatch(sh);
    if (chunk <= 0) return 1;
    return (int)((sh.max_tokens + chunk - 1) / chunk);
}

cudaError_t launch_decode_tuned(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh, float* out,
                                float* partials, cudaStream_t st)
{
    const int chunk = chunk_dispatch(sh);
    if (chunk <= 0) return cudaErrorNotSupported;
    const int n_parts = decode_tuned_parts(sh);
    cudaError_t e = cudaErrorNotSupported;
    if (sh.G == 16 && sh.R == 1) e = launch_cfg<16, 1>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, chunk, n_parts, partials, st);
    else if (sh.G == 16 && sh.R == 2) e = launch_cfg<16, 2>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, chunk, n_parts, partials, st);
    else if (sh.G == 16 && sh.R == 4) e = launch_cfg<16, 4>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, chunk, n_parts, partials, st);
    else if (sh.G == 32 && sh.R == 1) e = launch_cfg<32, 1>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, chunk, n_parts, partials, st);
    else if (sh.G == 32 && sh.R == 2) e = launch_cfg<32, 2>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, chunk, n_parts, partials, st);
    if (e != cudaSuccess) return e;
    return launch_merge(partials, n_parts, sh, out, st);
}

}  // namespace cq
