// Tuned encode kernels for head_dim 128, b = 8, c in {2, 4, 8} (CQ-2c8b, -4c8b, -8c8b).
//
// CQ encode (Section 3.2 of the paper, the map CQ(.) of Eq. 5): every group of c contiguous
// channels of a vector is replaced by the index of its nearest centroid in L2 distance,
// lowest index on exact ties.
//
// Method.  For 16 vectors x 8 centroids of one group, one m16n8k16 tensor-core MMA (fp16
// operands, fp32 accumulation) evaluates
//     d_j ~ ||x_g||^2 - 2 <x_g, C_j> + ||C_j||^2
// with the fp32 centroids and norms carried as sums of three (or two) fp16 terms, so every
// product is exact and only the fp32 accumulation rounds.  The k-slots of the MMA hold, in
// pairs (one 32-bit register each):
//     A: x words | x words | x words | (1, 1)        | (X_hi, X_lo) | (1, 0)
//     B: -2C_hi  | -2C_lo  | -2C_lo2 | (N_hi, N_lo)  | (1, 1)       | (N_lo2, 0)
// (N = ||C_j||^2, X = ||x_g||^2; c = 8 needs two MMAs per tile, c = 4 drops N_lo2).
// The accumulator lanes then keep, per vector, the smallest score of four subsets of their
// columns, with the centroid index packed into the low mantissa byte (one 3-input min per two
// scores).  The smallest of a quad's 16 subset minima names the winner's subset, whose 16
// centroids are evaluated exactly (direct form sum (x - C)^2 in fp32); the second smallest subset
// minimum bounds every other centroid from below, and the exact winner is accepted only if that
// bound is farther away than a bound on the evaluation error.  Otherwise (near-ties, exact ties
// across subsets, out-of-range codebooks) the warp recomputes that (vector, group) over all 256
// centroids exactly, lowest index on ties -- the arithmetic of the generic kernel.
//
// The selection, not the tensor pipe, is what bounds this kernel: the ALU pipe (min / logic,
// 64 lanes per clock and SM) is about 77 % busy, the tensor pipe about 14 %.
#include "cq_common.cuh"

namespace cq {

namespace {

constexpr int kEncWarps = 8;
constexpr int kEncThreads = kEncWarps * 32;
constexpr float kInfBits = __builtin_huge_valf();

template <int kC>
struct EncCfg {
    static constexpr int G = 128 / kC;
    static constexpr int kSteps = (kC == 8) ? 2 : 1;          // MMAs (k-steps of 16 slots) per tile
    static constexpr int kBufWords = kSteps * 256 * 8;        // 32-bit words of one prepared codebook
};

struct EncCtl {
    int range_flag[2];     // non-zero: the prepared group holds values fp16 cannot carry
    float nmax[2];         // largest ||C_j||^2 of the prepared group (float bits, non-negative)
};

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    return (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
}

// v = t0 + t1 + t2 with fp16 terms (t2 absorbs what two terms leave, about 2^-33 |v| remains)
__device__ __forceinline__ void split3(float v, float& t0, float& t1, float& t2)
{
    t0 = __half2float(__float2half_rn(v));
    const float r1 = v - t0;
    t1 = __half2float(__float2half_rn(r1));
    t2 = __half2float(__float2half_rn(r1 - t1));
}

__device__ __forceinline__ float min3f(float a, float b, float c)
{
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// D = A * B (no accumulator to clear beforehand)
__device__ __forceinline__ void mma_f16_first(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Prepares the B operand of group g of head h: thread t handles centroid t.
// Layout: word (j * 8 + p * 2 + q) of a k-step holds slot pair p + 4 q of centroid j, so that
// lane (n, p) of the MMA reads its (b0, b1) for centroid nt * 8 + n as one 8-byte word.
template <int kC>
__device__ __forceinline__ void prepare_group(const float* __restrict__ cb_g, uint32_t* buf, EncCtl* ctl, int slot)
{
    const int j = threadIdx.x;
    float cv[kC];
    if (kC == 2) {
        const float2 a = *reinterpret_cast<const float2*>(cb_g + j * 2);
        cv[0] = a.x; cv[1] = a.y;
    } else {
        const float4 a = *reinterpret_cast<const float4*>(cb_g + j * kC);
        cv[0] = a.x; cv[1] = a.y; cv[2 % kC] = a.z; cv[3 % kC] = a.w;
        if (kC == 8) {
            const float4 b = *reinterpret_cast<const float4*>(cb_g + j * kC + 4);
            cv[4 % kC] = b.x; cv[5 % kC] = b.y; cv[6 % kC] = b.z; cv[7 % kC] = b.w;
        }
    }
    float nrm = 0.f, amax = 0.f;
    float t0[kC], t1[kC], t2[kC];
#pragma unroll
    for (int i = 0; i < kC; ++i) {
        nrm = fmaf(cv[i], cv[i], nrm);
        amax = fmaxf(amax, fabsf(cv[i]));
        split3(-2.f * cv[i], t0[i], t1[i], t2[i]);
    }
    float n0, n1, n2;
    split3(nrm, n0, n1, n2);
    if (!(amax < 16000.f) || !(nrm < 60000.f)) atomicOr(&ctl->range_flag[slot], 1);
    atomicMax(reinterpret_cast<int*>(&ctl->nmax[slot]), __float_as_int(nrm));
    const uint32_t ones = 0x3c003c00u;               // half2(1, 1)
    uint32_t pr[EncCfg<kC>::kSteps][8];
    if (kC == 2) {
        pr[0][0] = pack_half2(t0[0], t0[1]);
        pr[0][1] = pack_half2(t1[0], t1[1]);
        pr[0][2] = pack_half2(t2[0], t2[1]);
        pr[0][3] = pack_half2(n0, n1);
        pr[0][4] = ones;
        pr[0][5] = pack_half2(n2, 0.f);
        pr[0][6] = 0u;
        pr[0][7] = 0u;
    } else if (kC == 4) {
        pr[0][0] = pack_half2(t0[0], t0[1]);
        pr[0][1] = pack_half2(t0[2 % kC], t0[3 % kC]);
        pr[0][2] = pack_half2(t1[0], t1[1]);
        pr[0][3] = pack_half2(t1[2 % kC], t1[3 % kC]);
        pr[0][4] = pack_half2(t2[0], t2[1]);
        pr[0][5] = pack_half2(t2[2 % kC], t2[3 % kC]);
        pr[0][6] = pack_half2(n0, n1);
        pr[0][7] = ones;
    } else {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            pr[0][w] = pack_half2(t0[(2 * w) % kC], t0[(2 * w + 1) % kC]);
            pr[0][4 + w] = pack_half2(t1[(2 * w) % kC], t1[(2 * w + 1) % kC]);
            pr[kC == 8 ? 1 : 0][w] = pack_half2(t2[(2 * w) % kC], t2[(2 * w + 1) % kC]);
        }
        pr[kC == 8 ? 1 : 0][4] = pack_half2(n0, n1);
        pr[kC == 8 ? 1 : 0][5] = ones;
        pr[kC == 8 ? 1 : 0][6] = pack_half2(n2, 0.f);
        pr[kC == 8 ? 1 : 0][7] = 0u;
    }
#pragma unroll
    for (int st = 0; st < EncCfg<kC>::kSteps; ++st) {
        uint32_t* dst = buf + st * 256 * 8 + j * 8;
        // word p * 2 + q holds pair p + 4 q
        *reinterpret_cast<uint4*>(dst) = make_uint4(pr[st][0], pr[st][4], pr[st][1], pr[st][5]);
        *reinterpret_cast<uint4*>(dst + 4) = make_uint4(pr[st][2], pr[st][6], pr[st][3], pr[st][7]);
    }
}

// The A operand of one m-tile for one group, from the x words this lane owns.
// xw[half] is the 32-bit word (two channels) of row r (half 0) / r + 8 (half 1) that lane p uses,
// X[half] the squared norm of the row's group.
template <int kC>
__device__ __forceinline__ void build_a(const uint32_t (&xw)[2], const float (&X)[2], int p,
                                        uint32_t (&a)[EncCfg<kC>::kSteps][4])
{
    const uint32_t ones = 0x3c003c00u, one_zero = 0x00003c00u;   // half2(1, 1), half2(1, 0)
    uint32_t xn[2];
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        const float x0 = __half2float(__float2half_rn(X[hf]));
        xn[hf] = pack_half2(x0, X[hf] - x0);
    }
    if (kC == 2) {
        // pairs: 0-2 x, 3 (1,1), 4 (X_hi, X_lo), 5 (1,0), 6-7 zero
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            a[0][hf] = p < 3 ? xw[hf] : ones;                                   // pair p
            a[0][2 + hf] = p == 0 ? xn[hf] : (p == 1 ? one_zero : 0u);          // pair p + 4
        }
    } else if (kC == 4) {
        // pairs: 0-5 x (word p % 2), 6 (1,1), 7 (X_hi, X_lo)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            a[0][hf] = xw[hf];
            a[0][2 + hf] = p < 2 ? xw[hf] : (p == 2 ? ones : xn[hf]);
        }
    } else {
        // step 0: pairs 0-3 x (word p), 4-7 x (word p); step 1: 0-3 x, 4 (1,1), 5 (X), 6 (1,0), 7 zero
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            a[0][hf] = xw[hf];
            a[0][2 + hf] = xw[hf];
            a[EncCfg<kC>::kSteps - 1][hf] = xw[hf];
            a[EncCfg<kC>::kSteps - 1][2 + hf] = p == 0 ? ones : (p == 1 ? xn[hf] : (p == 2 ? one_zero : 0u));
        }
    }
}

// Exact nearest centroid of one group of one vector, computed by the whole warp:
// d_j = sum_i (x_i - C_ji)^2 in fp32 (same operation order as the generic kernel), lowest j on ties.
template <int kC>
__device__ __forceinline__ int exact_code(const float (&xg)[kC], const float* __restrict__ cb_g, int lane, float* dist)
{
    float best = kInfBits;
    int arg = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int j = t * 32 + lane;
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < kC; ++i) {
            const float diff = xg[i] - cb_g[j * kC + i];
            d = fmaf(diff, diff, d);
        }
        if (d < best) { best = d; arg = j; }        // j increases with t: strict < keeps the lowest index
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (ob < best || (ob == best && oa < arg)) { best = ob; arg = oa; }
    }
    *dist = best;
    return arg;
}

// kMT: 16-vector m-tiles per warp (4 for bulk encode, 1 when there are few vectors).
// A launch covers one tensor, or two of the same shape (the key and the value of an append):
// blockIdx.y picks (x, cb, codes) or (x2, cb2, codes2).
// kWide: 2^b > 256 centroids per group (b = 9, 10, 12): the group's codebook is taken in chunks of
// 256 centroids, each chunk exactly as a codebook of b = 8, and the chunk winners are compared by
// their exact distances (the earlier chunk wins ties, so the lowest index still does).
template <int kC, int kMT, bool kWide>
__global__ void __launch_bounds__(kEncThreads, 2)
encode_tuned_kernel(const __half* __restrict__ x1, const float* __restrict__ cb1, const int32_t* __restrict__ seq_offsets,
                    Shape sh, int64_t n_tokens, int64_t token_offset, uint8_t* __restrict__ codes1, int groups_per_cta,
                    const __half* __restrict__ x2, const float* __restrict__ cb2, uint8_t* __restrict__ codes2)
{
    const __half* x = blockIdx.y ? x2 : x1;
    const float* cb = blockIdx.y ? cb2 : cb1;
    uint8_t* codes = blockIdx.y ? codes2 : codes1;
    using C = EncCfg<kC>;
    constexpr int G = C::G;
    constexpr int kTileVecs = kEncWarps * kMT * 16;
    extern __shared__ __align__(16) uint32_t enc_smem[];
    uint32_t* bbuf[2] = {enc_smem, enc_smem + C::kBufWords};
    EncCtl* ctl = reinterpret_cast<EncCtl*>(enc_smem + 2 * C::kBufWords);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, p = lane & 3;
    const int n_heads = sh.n_kv_heads;
    const int64_t n_vec = sh.n_seq * n_tokens;

    const int n_gsplit = (G + groups_per_cta - 1) / groups_per_cta;
    const int gs = blockIdx.x % n_gsplit;
    const int h = (blockIdx.x / n_gsplit) % n_heads;
    const int64_t tile = blockIdx.x / (n_gsplit * n_heads);
    const int g_begin = gs * groups_per_cta;
    const int g_end = g_begin + groups_per_cta < G ? g_begin + groups_per_cta : G;

    // rows of this lane: vector v_row[mt][half] = v0 + mt*16 + r + 8*half
    const int64_t v0 = tile * kTileVecs + (int64_t)warp * (kMT * 16);
    const __half* xrow0 = x + (v0 * n_heads + h) * 128;              // row of vector v0, head h
    const int64_t row_stride = (int64_t)n_heads * 128;               // halves between consecutive vectors
    // word of the group that lane p feeds to the MMA: c = 2 -> word 0, c = 4 -> word p % 2, c = 8 -> word p
    const int wsel = kC == 2 ? 0 : (kC == 4 ? (p & 1) : p);

    if (threadIdx.x < 2) { ctl->range_flag[threadIdx.x] = 0; ctl->nmax[threadIdx.x] = 0.f; }
    __syncthreads();
    const int n_chunks = kWide ? sh.K / 256 : 1;
    const int n_steps = (g_end - g_begin) * n_chunks;
    // centroids of step st: chunk st % n_chunks of group g_begin + st / n_chunks
    auto chunk_ptr = [&](int st) {
        return cb + (((int64_t)h * G + g_begin + st / n_chunks) * n_chunks + st % n_chunks) * 256 * kC;
    };
    prepare_group<kC>(chunk_ptr(0), bbuf[0], ctl, 0);
    float dkeep[kWide ? kMT : 1][2];           // best exact distance and code over the chunks seen so far
    int ckeep[kWide ? kMT : 1][2];

    for (int st = 0; st < n_steps; ++st) {
        const int g = g_begin + st / n_chunks, ch = st % n_chunks;
        const int cur = st & 1;
        __syncthreads();                       // bbuf[cur] is complete; bbuf[cur ^ 1] is no longer read
        const bool out_of_range = ctl->range_flag[cur] != 0;
        const float nmax = ctl->nmax[cur];
        __syncthreads();                       // everyone has read the control words of `cur`
        if (threadIdx.x == 0) { ctl->range_flag[cur ^ 1] = 0; ctl->nmax[cur ^ 1] = 0.f; }
        __syncthreads();
        if (st + 1 < n_steps) prepare_group<kC>(chunk_ptr(st + 1), bbuf[cur ^ 1], ctl, cur ^ 1);
        const float* cb_g = chunk_ptr(st);

        // A operands of this warp's m-tiles
        uint32_t a[kMT][C::kSteps][4];
        uint32_t xwreg[kMT][2];            // the x word this lane loaded, per row
        float Xrow[kMT][2];
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt) {
            uint32_t xw[2];
            float X[2];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int64_t v = v0 + mt * 16 + r + 8 * hf;
                xw[hf] = 0u;
                X[hf] = 0.f;
                if (v < n_vec) {
                    const uint32_t* gp = reinterpret_cast<const uint32_t*>(xrow0 + (mt * 16 + r + 8 * hf) * row_stride + g * kC);
                    xw[hf] = gp[wsel];
                    // squared norm of the whole group (every lane of the quad computes the same value)
#pragma unroll
                    for (int w = 0; w < kC / 2; ++w) {
                        const uint32_t ww = (kC == 2) ? xw[hf] : gp[w];
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww));
                        X[hf] = fmaf(f.x, f.x, X[hf]);
                        X[hf] = fmaf(f.y, f.y, X[hf]);
                    }
                }
                Xrow[mt][hf] = X[hf];
                xwreg[mt][hf] = xw[hf];
            }
            build_a<kC>(xw, X, p, a[mt]);
        }

        // Selection.  Every lane keeps, per row, the smallest score of four subsets of its columns
        // (n-tile index mod 4), index packed into the low mantissa byte: one 3-input min per two
        // scores.  The smallest of the quad's 16 subset minima names the winner's subset; its 16
        // centroids are then evaluated exactly, and the second smallest subset minimum bounds every
        // other centroid from below.
        float sb[kMT][2][4];
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int q = 0; q < 4; ++q) sb[mt][hf][q] = kInfBits;

        const uint32_t keep = 0xffffff00u;
        const uint2* bsrc = reinterpret_cast<const uint2*>(bbuf[cur]) + lane;
#pragma unroll 2
        for (int nt0 = 0; nt0 < 32; nt0 += 4) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int nt = nt0 + q;
                uint2 b[C::kSteps];
#pragma unroll
                for (int st = 0; st < C::kSteps; ++st) b[st] = bsrc[st * 1024 + nt * 32];
                const uint32_t i0 = nt * 8, i1 = nt * 8 + 1;      // centroid index without the lane's 2p
#pragma unroll
                for (int mt = 0; mt < kMT; ++mt) {
                    float d[4];
                    mma_f16_first(d, a[mt][0], b[0].x, b[0].y);
#pragma unroll
                    for (int st = 1; st < C::kSteps; ++st) mma_f16(d, a[mt][st], b[st].x, b[st].y);
                    const float v0p = __uint_as_float((__float_as_uint(d[0]) & keep) | i0);
                    const float v1p = __uint_as_float((__float_as_uint(d[1]) & keep) | i1);
                    const float v2p = __uint_as_float((__float_as_uint(d[2]) & keep) | i0);
                    const float v3p = __uint_as_float((__float_as_uint(d[3]) & keep) | i1);
                    sb[mt][0][q] = min3f(sb[mt][0][q], v0p, v1p);
                    sb[mt][1][q] = min3f(sb[mt][1][q], v2p, v3p);
                }
            }
        }

        // merge the quad, evaluate the winner's subset exactly, certify, store
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float b, s2;
                {
                    const uint32_t pb = 2u * p;
                    const float t0 = __uint_as_float(__float_as_uint(sb[mt][hf][0]) | pb);
                    const float t1 = __uint_as_float(__float_as_uint(sb[mt][hf][1]) | pb);
                    const float t2 = __uint_as_float(__float_as_uint(sb[mt][hf][2]) | pb);
                    const float t3 = __uint_as_float(__float_as_uint(sb[mt][hf][3]) | pb);
                    const float lo01 = fminf(t0, t1), hi01 = fmaxf(t0, t1), lo23 = fminf(t2, t3), hi23 = fmaxf(t2, t3);
                    b = fminf(lo01, lo23);
                    s2 = min3f(fmaxf(lo01, lo23), hi01, hi23);
                }
#pragma unroll
                for (int o = 1; o <= 2; o <<= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, b, o);
                    const float os = __shfl_xor_sync(0xffffffffu, s2, o);
                    const float t = fmaxf(b, ob);
                    b = fminf(b, ob);
                    s2 = min3f(s2, os, t);
                }
                // the winner's subset: lane pw of the quad, n-tiles qw, qw + 4, ..., qw + 28
                const int jw = (int)(__float_as_uint(b) & 0xffu);
                const int pw = (jw >> 1) & 3, qw = (jw >> 3) & 3;
                float xg[kC];
#pragma unroll
                for (int w = 0; w < kC / 2; ++w) {
                    const uint32_t ww = kC == 2 ? xwreg[mt][hf] : __shfl_sync(0xffffffffu, xwreg[mt][hf], (lane & ~3) | w);
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww));
                    xg[2 * w] = f.x;
                    xg[(2 * w + 1) % kC] = f.y;
                }
                float dbest = kInfBits;
                int code = 0;
#pragma unroll
                for (int tt = 0; tt < 2; ++tt) {
                    const int j0 = (qw + 4 * (2 * p + tt)) * 8 + 2 * pw;       // centroids j0, j0 + 1 (ascending over tt)
                    float cc[2 * kC];
#pragma unroll
                    for (int w = 0; w < 2 * kC; w += 4) {
                        const float4 t4 = *reinterpret_cast<const float4*>(cb_g + j0 * kC + w);
                        cc[w] = t4.x; cc[w + 1] = t4.y; cc[w + 2] = t4.z; cc[w + 3] = t4.w;
                    }
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        float dd = 0.f;
#pragma unroll
                        for (int i = 0; i < kC; ++i) {
                            const float diff = xg[i] - cc[e * kC + i];
                            dd = fmaf(diff, diff, dd);
                        }
                        if (dd < dbest) { dbest = dd; code = j0 + e; }         // ascending j: strict < keeps the lowest
                    }
                }
#pragma unroll
                for (int o = 1; o <= 2; o <<= 1) {
                    const float od = __shfl_xor_sync(0xffffffffu, dbest, o);
                    const int oc = __shfl_xor_sync(0xffffffffu, code, o);
                    if (od < dbest || (od == dbest && oc < code)) { dbest = od; code = oc; }
                }
                const int64_t v = v0 + mt * 16 + r + 8 * hf;
                const float ss = __uint_as_float(__float_as_uint(s2) & keep);
                // Evaluation error of a score: fp32 accumulation of up to ~20 terms bounded by
                // 2 (X + N) in magnitude, plus the mantissa byte given to the index.  dbest is exact.
                const float tau = 1.6e-5f * (Xrow[mt][hf] + nmax) + 6.2e-5f * fabsf(ss);
                const bool certain = !out_of_range && (ss - dbest > tau);
                // exact recomputation of the uncertain rows, one row at a time by the whole warp
                unsigned pending = __ballot_sync(0xffffffffu, !certain && p == 0 && v < n_vec);
                while (pending) {
                    const int src = __ffs(pending) - 1;          // lane with p == 0 of the row's quad
                    pending &= pending - 1;
                    // gather the row's group: lane src + w holds word w (c = 8), word w % 2 (c = 4), the word (c = 2)
                    float xg[kC];
#pragma unroll
                    for (int w = 0; w < kC / 2; ++w) {
                        const uint32_t ww = __shfl_sync(0xffffffffu, xwreg[mt][hf], src + (kC == 2 ? 0 : w));
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww));
                        xg[2 * w] = f.x;
                        xg[(2 * w + 1) % kC] = f.y;
                    }
                    float ed;
                    const int ec = exact_code<kC>(xg, cb_g, lane, &ed);
                    if ((lane & ~3) == src) { code = ec; dbest = ed; }
                }
                if (kWide) {
                    // dbest is the exact distance of `code` within this chunk: keep the best chunk so far
                    const int m = kWide ? mt : 0;
                    if (ch == 0 || dbest < dkeep[m][hf]) { dkeep[m][hf] = dbest; ckeep[m][hf] = code + 256 * ch; }
                    if (ch + 1 < n_chunks) continue;
                    code = ckeep[m][hf];
                }
                if (p == 0 && v < n_vec) {
                    const int64_t s = v / n_tokens, i = v % n_tokens;
                    const int64_t pos = token_offset + (seq_offsets ? seq_offsets[s] : 0) + i;
                    if (pos >= 0 && pos < sh.max_tokens) {
                        const int k = (int)(pos % kTokenBlock);
                        codes[code_word_offset(sh, n_heads, s, h, pos / kTokenBlock, g) + k] = (uint8_t)code;
                        if (kWide) {        // upper bits: replaced in the 32-bit word that other tokens share
                            const int bit = k * sh.hb;
                            const uintptr_t a = reinterpret_cast<uintptr_t>(codes) +
                                                (uintptr_t)code_high_offset(sh, n_heads, s, h, pos / kTokenBlock, g) + (bit >> 3);
                            unsigned int* w = reinterpret_cast<unsigned int*>(a & ~(uintptr_t)3);
                            const int shift = (int)(a & 3) * 8 + (bit & 7);
                            atomicAnd(w, ~((unsigned int)((1 << sh.hb) - 1) << shift));
                            atomicOr(w, (unsigned int)(code >> 8) << shift);
                        }
                    }
                }
            }
    }
}

template <int kC, int kMT, bool kWide = false>
cudaError_t launch_enc(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh, int64_t n_tokens,
                       int64_t token_offset, uint8_t* codes, cudaStream_t st, const __half* x2 = nullptr,
                       const float* cb2 = nullptr, uint8_t* codes2 = nullptr)
{
    using C = EncCfg<kC>;
    constexpr int kTileVecs = kEncWarps * kMT * 16;
    const int64_t n_vec = sh.n_seq * n_tokens;
    const int64_t tiles = (n_vec + kTileVecs - 1) / kTileVecs;
    // split the groups over CTAs while the grid would leave SMs idle
    int64_t n_gsplit = (2 * (int64_t)device_sm_count() + tiles * sh.n_kv_heads - 1) / (tiles * sh.n_kv_heads);
    if (n_gsplit > C::G) n_gsplit = C::G;
    if (n_gsplit < 1) n_gsplit = 1;
    const int groups_per_cta = (int)((C::G + n_gsplit - 1) / n_gsplit);
    n_gsplit = (C::G + groups_per_cta - 1) / groups_per_cta;
    const int64_t grid = tiles * sh.n_kv_heads * n_gsplit;
    if (grid > 0x7fffffff) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)2 * C::kBufWords * 4 + sizeof(EncCtl);
    // call-site slots of ensure_dynamic_smem: 16 ... 27, one per template instance
    constexpr int kSlot = 16 + 4 * (kC == 2 ? 0 : kC == 4 ? 1 : 2) + 2 * (kMT == 1 ? 0 : 1) + (kWide ? 1 : 0);
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(encode_tuned_kernel<kC, kMT, kWide>), (int)smem, kSlot);
    if (e != cudaSuccess) return e;
    encode_tuned_kernel<kC, kMT, kWide><<<dim3((unsigned)grid, x2 ? 2u : 1u), kEncThreads, smem, st>>>(
        x, cb, seq_offsets, sh, n_tokens, token_offset, codes, groups_per_cta, x2, cb2, codes2);
    return cudaGetLastError();
}

}  // namespace

bool encode_tuned_supported(const Shape& sh)
{
    if (sh.head_dim != 128 || !(sh.c == 2 || sh.c == 4 || sh.c == 8)) return false;
    return sh.b == 8 || sh.b == 9 || sh.b == 10 || sh.b == 12;       // whole chunks of 256 centroids
}

cudaError_t launch_encode_tuned(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh,
                                int64_t n_tokens, int64_t token_offset, uint8_t* codes, cudaStream_t st,
                                const __half* x2, const float* cb2, uint8_t* codes2, bool allow_tc)
{
    const int64_t n_vec = sh.n_seq * n_tokens;
    if (n_vec == 0) return cudaSuccess;
    const bool few = n_vec * sh.n_kv_heads < (int64_t)device_sm_count() * 512 * 2;    // not enough vectors for 64 per warp
    if (allow_tc && !few && encode_tc_supported(sh))
        return launch_encode_tc(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
    if (sh.b > 8) {
        switch (sh.c) {
            case 2: return few ? launch_enc<2, 1, true>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2)
                               : launch_enc<2, 4, true>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
            case 4: return few ? launch_enc<4, 1, true>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2)
                               : launch_enc<4, 4, true>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
            case 8: return few ? launch_enc<8, 1, true>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2)
                               : launch_enc<8, 4, true>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
            default: return cudaErrorNotSupported;
        }
    }
    switch (sh.c) {
        case 2: return few ? launch_enc<2, 1>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2)
                           : launch_enc<2, 4>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
        case 4: return few ? launch_enc<4, 1>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2)
                           : launch_enc<4, 4>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
        case 8: return few ? launch_enc<8, 1>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2)
                           : launch_enc<8, 4>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace cq
