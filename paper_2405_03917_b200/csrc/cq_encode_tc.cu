// Bulk encode on the fifth-generation tensor cores (tcgen05, accumulators in tensor memory) for
// head_dim 128, b = 8, c in {2, 4, 8}: the kernel for prefill-sized inputs.
//
// CQ encode (Section 3.2 of the paper, the map CQ(.) of Eq. 5): every group of c contiguous
// channels of a vector is replaced by the index of its nearest centroid in L2 distance, lowest
// index on exact ties.
//
// Arithmetic: that of encode_tuned_kernel.  For 128 vectors x 128 centroids of one group ONE
// tcgen05.mma (M = 128, N = 128, K = 16; two of them, accumulating, for c = 8) evaluates
//     d_j ~ ||x_g||^2 - 2 <x_g, C_j> + ||C_j||^2
// with the fp32 centroids and norms carried as sums of three fp16 terms, so that every product is
// exact and only the fp32 accumulation rounds.  K slots, in pairs:
//     c = 2   A: x | x | x | (1,1) | (X_hi,X_lo) | (1,0) | 0 | 0
//             B: t0 | t1 | t2 | (N_hi,N_lo) | (1,1) | (N_lo2,0) | 0 | 0        (-2C = t0 + t1 + t2)
//     c = 4   A: x x | x x | x x | (1,1) | (X_hi,X_lo)      B: t0 t0 | t1 t1 | t2 t2 | (N_hi,N_lo) | (1,1)
//     c = 8   two K steps: (x x x x | x x x x) against (t0 | t1), then (x x x x | (1,1), X, (1,0), 0)
//             against (t2 | N, (1,1), (N_lo2,0), 0)
// What differs is where the scores go.  The accumulator tile lives in tensor memory, row i in
// lane i, and a thread reads the 256 scores of ITS row with tcgen05.ld: no accumulator registers
// to clear, no B fragments to fetch in the selecting warps, no quad to merge, and - because the
// winner is found by exact re-evaluation anyway - no index packed into every score.  A thread
// keeps the minimum of each of 16 subsets of the centroids (index mod 16), one 3-input min per
// two scores; the subset with the smallest minimum is evaluated exactly (16 centroids, direct form
// sum (x - C)^2 in fp32, lowest index on ties) and the second smallest subset minimum bounds
// every other centroid from below.  The exact winner is accepted if that bound is farther away
// than a bound on the evaluation error; otherwise (near-ties, ties across subsets, codebooks
// fp16 cannot carry) the warp recomputes that row over all 256 centroids exactly.
//
// A CTA is one tile of 128 vectors of one head: 4 warps, warp w owning the tensor memory lanes
// 32 w ... 32 w + 31, and 128 tensor-memory columns, so that four CTAs (three for c = 8, whose
// operands take more shared memory) live on an SM and fill each other's waits.  The accumulator is
// therefore 128 x 128: the scores of a step arrive in two halves (centroids 0-127, then 128-255)
// through the same columns, and the operand preparation and the row finishing are placed behind
// the MMA issues.  A CTA takes up to eight row tiles through every group before it moves to the
// next group, so a group's centroids are prepared once per up to 1024 vectors.
#include "cq_common.cuh"

namespace cq {

namespace {

constexpr int kTcThreads = 128;
constexpr int kTcTileVecs = 128;          // vectors of a row tile
constexpr float kTcInf = __builtin_huge_valf();

template <int kC>
struct TcCfg {
    static constexpr int G = 128 / kC;
    static constexpr int kSteps = (kC == 8) ? 2 : 1;              // K steps (16 fp16 slots each)
    static constexpr int kATile = 128 * 32;                       // bytes of one A tile of one K step
    static constexpr int kBTile = 256 * 32;
    static constexpr int kABuf = kSteps * kATile;
    static constexpr int kBBuf = kSteps * kBTile;
    static constexpr int kCbf = 256 * kC * 4;                     // the group's centroids as fp32
    static constexpr int kMaxLogRt = (kC == 8) ? 2 : 3;           // up to 2^kMaxLogRt row tiles per CTA
    static constexpr int kCtasPerSm = (kC == 8) ? 3 : 4;
    static constexpr int kAOff = 0;                               // [2 buffers]
    static constexpr int kBOff = kAOff + 2 * kABuf;               // [2 buffers]
    static constexpr int kCbfOff = kBOff + 2 * kBBuf;             // [2 slots]
    static constexpr int kRowOff = kCbfOff + 2 * kCbf;            // [row tiles][128 threads] row records
    static constexpr int kCtlOff = kRowOff + (1 << kMaxLogRt) * kTcThreads * 16;
    static constexpr int kUsedBytes = kCtlOff + 256;
    // at least 46 KiB, so that a fifth CTA (for which no tensor memory would be left) never fits an SM
    static constexpr int kSmemBytes = kUsedBytes > 46 * 1024 ? kUsedBytes : 46 * 1024;
    static_assert(kCtasPerSm * (kSmemBytes + 1024) <= 228 * 1024, "shared memory of an SM");
    static_assert((kCtasPerSm + 1) * (kSmemBytes + 1024) > 228 * 1024, "one CTA too many would fit");
};

constexpr int kTcColumns = 128;            // tensor-memory columns of a CTA

// What a thread needs of one of its rows, worked out once: where the vector's head slice starts and where its code of
// group 0 goes (the code of group g follows kTokenBlock * g bytes on).
struct TcRow {
    const __half* x;           // null: no such vector
    int64_t code_offset;       // negative: the token has no position in the cache
};
static_assert(sizeof(TcRow) == 16, "row record");

struct TcCtl {
    int range_flag[2][8];      // per warp and pass, non-zero: those centroids of the prepared group hold values fp16 cannot carry
    float nmax[2][8];          // per warp and pass, the largest ||C_j||^2 among those centroids
    uint32_t tmem_base;
    int wait_failed;           // a wait on an MMA barrier gave up
    uint64_t bar[2];           // completion of the MMA of the low / high half of a step
};

__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t tc_pack_half2(float lo, float hi)
{
    return (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
}

// v = t0 + t1 + t2 with fp16 terms (t2 absorbs what two terms leave, about 2^-33 |v| remains)
__device__ __forceinline__ void tc_split3(float v, float& t0, float& t1, float& t2)
{
    t0 = __half2float(__float2half_rn(v));
    const float r1 = v - t0;
    t1 = __half2float(__float2half_rn(r1));
    t2 = __half2float(__float2half_rn(r1 - t1));
}

__device__ __forceinline__ float tc_min3(float a, float b, float c)
{
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Shared-memory matrix descriptor of a K-major operand tile without swizzle: the 16-byte chunk kc (8 fp16 K slots)
// of row r sits at kc * rows * 16 + r * 16 bytes, so a core matrix (8 rows x 16 bytes) is 128 contiguous bytes, the
// next 8 rows follow 128 bytes on (stride byte offset) and the next K chunk rows * 16 bytes on (leading byte offset).
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t chunk_stride_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fffu);
    d |= (uint64_t)((chunk_stride_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((128u >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;                      // descriptor version of sm_100
    return d;
}

// D[128 x 128] (+)= A[128 x 16] * B[128 x 16]^T, fp16 operands from shared memory, fp32 accumulator in tensor memory
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    // instruction descriptor: D fp32, A and B fp16, both K-major, N = 128, M = 128
    const uint32_t idesc = (1u << 4) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0) : "memory");
}

// Starts the load of 32 consecutive accumulator columns of this thread's row; the values are there after tc_ld_wait.
__device__ __forceinline__ void tc_ld32_issue(float (&v)[32], uint32_t taddr)
{
    uint32_t* u = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
                 : "r"(taddr) : "memory");
}
// Waits for the loads issued so far.  The registers pass through the statement, so that nothing that uses them is
// scheduled ahead of the wait.
__device__ __forceinline__ void tc_ld_wait(float (&v)[32])
{
    uint32_t* u = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]), "+r"(u[4]), "+r"(u[5]), "+r"(u[6]), "+r"(u[7]), "+r"(u[8]), "+r"(u[9]), "+r"(u[10]), "+r"(u[11]), "+r"(u[12]), "+r"(u[13]), "+r"(u[14]), "+r"(u[15]), "+r"(u[16]), "+r"(u[17]), "+r"(u[18]), "+r"(u[19]), "+r"(u[20]), "+r"(u[21]), "+r"(u[22]), "+r"(u[23]), "+r"(u[24]), "+r"(u[25]), "+r"(u[26]), "+r"(u[27]), "+r"(u[28]), "+r"(u[29]), "+r"(u[30]), "+r"(u[31])
                 :: "memory");
}

// Waits for the phase with the given parity; gives up after a bounded number of polls (returns false).
__device__ __forceinline__ bool tc_wait(uint64_t* bar, uint32_t parity)
{
    for (int poll = 0; poll < (1 << 22); ++poll) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(tc_smem_u32(bar)), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// Exact nearest centroid of one group of one vector, computed by the whole warp:
// d_j = sum_i (x_i - C_ji)^2 in fp32 (same operation order as the generic kernel), lowest j on ties.
template <int kC>
__device__ __forceinline__ int tc_exact_code(const float (&xg)[kC], const float* cbf, int lane, float* dist)
{
    float best = kTcInf;
    int arg = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int j = t * 32 + lane;
        float d = 0.f;
#pragma unroll
        for (int i = 0; i < kC; ++i) {
            const float diff = xg[i] - cbf[j * kC + i];
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


// Centroid j of a group, from global memory into registers.
template <int kC>
__device__ __forceinline__ void tc_fetch_centroid(const float* __restrict__ cb_g, int j, float (&cv)[kC])
{
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
}

// B operand of one group, one centroid: K slots as in the header comment; keeps the fp32 centroid for the exact
// evaluations; every warp leaves its largest squared norm and its range flag of this pass in the control block.
template <int kC>
__device__ __forceinline__ void tc_prepare_b(const float (&cv)[kC], int j, unsigned char* bbuf, float* cbf, TcCtl* ctl, int slot, int pass)
{
    using C = TcCfg<kC>;
    if (kC == 2) {
        *reinterpret_cast<float2*>(cbf + j * 2) = make_float2(cv[0], cv[1]);
    } else {
#pragma unroll
        for (int w = 0; w < kC; w += 4)
            *reinterpret_cast<float4*>(cbf + j * kC + w) = make_float4(cv[w], cv[w + 1], cv[(w + 2) % kC], cv[(w + 3) % kC]);
    }
    float nrm = 0.f, amax = 0.f;
    float t0[kC], t1[kC], t2[kC];
#pragma unroll
    for (int i = 0; i < kC; ++i) {
        nrm = fmaf(cv[i], cv[i], nrm);
        amax = fmaxf(amax, fabsf(cv[i]));
        tc_split3(-2.f * cv[i], t0[i], t1[i], t2[i]);
    }
    float n0, n1, n2;
    tc_split3(nrm, n0, n1, n2);
    const bool bad = !(amax < 16000.f) || !(nrm < 60000.f);
    const unsigned any_bad = __ballot_sync(0xffffffffu, bad);
    const float wmax = __uint_as_float(__reduce_max_sync(0xffffffffu, bad ? 0u : __float_as_uint(nrm)));   // nrm >= 0: bits order as values
    if ((threadIdx.x & 31) == 0) {
        ctl->range_flag[slot][pass * 4 + (threadIdx.x >> 5)] = any_bad != 0;
        ctl->nmax[slot][pass * 4 + (threadIdx.x >> 5)] = wmax;
    }
    const uint32_t ones = 0x3c003c00u;               // half2(1, 1)
    uint32_t pr[C::kSteps][8];
    if (kC == 2) {
        pr[0][0] = tc_pack_half2(t0[0], t0[1]);
        pr[0][1] = tc_pack_half2(t1[0], t1[1]);
        pr[0][2] = tc_pack_half2(t2[0], t2[1]);
        pr[0][3] = tc_pack_half2(n0, n1);
        pr[0][4] = ones;
        pr[0][5] = tc_pack_half2(n2, 0.f);
        pr[0][6] = 0u;
        pr[0][7] = 0u;
    } else if (kC == 4) {
        pr[0][0] = tc_pack_half2(t0[0], t0[1]);
        pr[0][1] = tc_pack_half2(t0[2 % kC], t0[3 % kC]);
        pr[0][2] = tc_pack_half2(t1[0], t1[1]);
        pr[0][3] = tc_pack_half2(t1[2 % kC], t1[3 % kC]);
        pr[0][4] = tc_pack_half2(t2[0], t2[1]);
        pr[0][5] = tc_pack_half2(t2[2 % kC], t2[3 % kC]);
        pr[0][6] = tc_pack_half2(n0, n1);
        pr[0][7] = ones;
    } else {
        constexpr int kLast = C::kSteps - 1;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            pr[0][w] = tc_pack_half2(t0[(2 * w) % kC], t0[(2 * w + 1) % kC]);
            pr[0][4 + w] = tc_pack_half2(t1[(2 * w) % kC], t1[(2 * w + 1) % kC]);
            pr[kLast][w] = tc_pack_half2(t2[(2 * w) % kC], t2[(2 * w + 1) % kC]);
        }
        pr[kLast][4] = tc_pack_half2(n0, n1);
        pr[kLast][5] = ones;
        pr[kLast][6] = tc_pack_half2(n2, 0.f);
        pr[kLast][7] = 0u;
    }
#pragma unroll
    for (int s = 0; s < C::kSteps; ++s) {
        unsigned char* dst = bbuf + s * C::kBTile + j * 16;
        *reinterpret_cast<uint4*>(dst) = make_uint4(pr[s][0], pr[s][1], pr[s][2], pr[s][3]);              // K slots 0 ... 7
        *reinterpret_cast<uint4*>(dst + 256 * 16) = make_uint4(pr[s][4], pr[s][5], pr[s][6], pr[s][7]);   // K slots 8 ... 15
    }
}

// The kC / 2 words (two fp16 channels each) of one group of one vector, from global memory.
template <int kC>
__device__ __forceinline__ void tc_fetch_x(const __half* gp, uint32_t (&xw)[kC / 2])
{
    if (kC == 2) {
        xw[0] = *reinterpret_cast<const uint32_t*>(gp);
    } else if (kC == 4) {
        const uint2 t = *reinterpret_cast<const uint2*>(gp);
        xw[0] = t.x; xw[1 % (kC / 2)] = t.y;
    } else {
        const uint4 t = *reinterpret_cast<const uint4*>(gp);
        xw[0] = t.x; xw[1 % (kC / 2)] = t.y; xw[2 % (kC / 2)] = t.z; xw[3 % (kC / 2)] = t.w;
    }
}

// A operand row of one vector for one group.  xw: the group's words, X its squared norm; atile: the row tile's first K step.
template <int kC>
__device__ __forceinline__ void tc_build_a(const uint32_t (&xw)[kC / 2], float X, unsigned char* atile, int row)
{
    using C = TcCfg<kC>;
    const uint32_t ones = 0x3c003c00u, one_zero = 0x00003c00u;   // half2(1, 1), half2(1, 0)
    const float x0 = __half2float(__float2half_rn(X));
    const uint32_t xn = tc_pack_half2(x0, X - x0);
    uint4 lo[C::kSteps], hi[C::kSteps];
    if (kC == 2) {
        lo[0] = make_uint4(xw[0], xw[0], xw[0], ones);
        hi[0] = make_uint4(xn, one_zero, 0u, 0u);
    } else if (kC == 4) {
        lo[0] = make_uint4(xw[0], xw[1 % (kC / 2)], xw[0], xw[1 % (kC / 2)]);
        hi[0] = make_uint4(xw[0], xw[1 % (kC / 2)], ones, xn);
    } else {
        constexpr int kLast = C::kSteps - 1;
        const uint4 xs = make_uint4(xw[0], xw[1 % (kC / 2)], xw[2 % (kC / 2)], xw[3 % (kC / 2)]);
        lo[0] = xs;
        hi[0] = xs;
        lo[kLast] = xs;
        hi[kLast] = make_uint4(ones, xn, one_zero, 0u);
    }
#pragma unroll
    for (int s = 0; s < C::kSteps; ++s) {
        unsigned char* dst = atile + s * C::kATile + row * 16;
        *reinterpret_cast<uint4*>(dst) = lo[s];
        *reinterpret_cast<uint4*>(dst + 128 * 16) = hi[s];
    }
}

static_assert(sizeof(TcCtl) <= 256, "control block");

// One step = one row tile (128 vectors) against one group.  A CTA takes 2^log_rt row tiles through its groups;
// blockIdx.x = (block of row tiles, head, group split).
template <int kC>
__global__ void __launch_bounds__(kTcThreads, TcCfg<kC>::kCtasPerSm)
encode_tc_kernel(const __half* __restrict__ x1, const float* __restrict__ cb1, const int32_t* __restrict__ seq_offsets,
                 Shape sh, int64_t n_tokens, int64_t token_offset, uint8_t* __restrict__ codes1, int groups_per_cta, int log_rt,
                 const __half* __restrict__ x2, const float* __restrict__ cb2, uint8_t* __restrict__ codes2)
{
    const __half* x = blockIdx.y ? x2 : x1;
    const float* cb = blockIdx.y ? cb2 : cb1;
    uint8_t* codes = blockIdx.y ? codes2 : codes1;
    using C = TcCfg<kC>;
    constexpr int G = C::G;
    extern __shared__ __align__(1024) unsigned char tc_smem[];
    TcCtl* ctl = reinterpret_cast<TcCtl*>(tc_smem + C::kCtlOff);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = threadIdx.x;                         // row within the tile = tensor memory lane
    const int n_heads = sh.n_kv_heads;
    const int64_t n_vec = sh.n_seq * n_tokens;

    const int n_gsplit = (G + groups_per_cta - 1) / groups_per_cta;
    const int gs = blockIdx.x % n_gsplit;
    const int h = (blockIdx.x / n_gsplit) % n_heads;
    const int64_t tile_block = blockIdx.x / (n_gsplit * n_heads);
    const int g_begin = gs * groups_per_cta;
    const int g_end = g_begin + groups_per_cta < G ? g_begin + groups_per_cta : G;
    const int rt_mask = (1 << log_rt) - 1;
    const int n_steps = (g_end - g_begin) << log_rt;     // step st: group g_begin + (st >> log_rt), row tile st & rt_mask

    // tensor memory (warp 0 allocates the CTA's columns and frees them at the end), the MMA barriers
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&ctl->tmem_base)), "n"(kTcColumns) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 32) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem_u32(&ctl->bar[0])) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem_u32(&ctl->bar[1])) : "memory");
        ctl->wait_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctl->tmem_base);
    const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);

    auto a_buf = [&](int buf) { return tc_smem + C::kAOff + buf * C::kABuf; };
    auto b_buf = [&](int buf) { return tc_smem + C::kBOff + buf * C::kBBuf; };
    auto cbf_slot = [&](int slot) { return reinterpret_cast<float*>(tc_smem + C::kCbfOff + slot * C::kCbf); };
    TcRow* rows = reinterpret_cast<TcRow*>(tc_smem + C::kRowOff) + threadIdx.x;      // record of row tile r: rows[r * kTcThreads]
    for (int r = 0; r <= rt_mask; ++r) {
        const int64_t v = (tile_block * (rt_mask + 1) + r) * kTcTileVecs + row;
        TcRow rec;
        rec.x = nullptr;
        rec.code_offset = -1;
        if (v < n_vec) {
            rec.x = x + (v * n_heads + h) * 128;
            const int64_t s = v / n_tokens, i = v % n_tokens;
            const int64_t pos = token_offset + (seq_offsets ? seq_offsets[s] : 0) + i;
            if (pos >= 0 && pos < sh.max_tokens) rec.code_offset = code_word_offset(sh, n_heads, s, h, pos / kTokenBlock, 0) + pos % kTokenBlock;
        }
        rows[r * kTcThreads] = rec;                      // read back by this thread only
    }

    // The vector's words travel global memory -> registers (fetch, half a step ahead) -> shared memory (build).
    uint32_t xw_pf[kC / 2];
    auto fetch = [&](int st) {
        const __half* xr = rows[(st & rt_mask) * kTcThreads].x;
#pragma unroll
        for (int w = 0; w < kC / 2; ++w) xw_pf[w] = 0u;
        if (xr) tc_fetch_x<kC>(xr + (g_begin + (st >> log_rt)) * kC, xw_pf);
    };
    uint32_t xw_nxt[kC / 2];
    float X_nxt;
    auto build = [&](int st) {
        const int gslot = (st >> log_rt) & 1;
        if ((st & rt_mask) == 0) {                       // a new group: centroids threadIdx.x and threadIdx.x + 128
            const float* cb_g = cb + ((int64_t)h * G + g_begin + (st >> log_rt)) * 256 * kC;
            float cv[2][kC];
            tc_fetch_centroid<kC>(cb_g, threadIdx.x, cv[0]);
            tc_fetch_centroid<kC>(cb_g, threadIdx.x + 128, cv[1]);
            tc_prepare_b<kC>(cv[0], threadIdx.x, b_buf(gslot), cbf_slot(gslot), ctl, gslot, 0);
            tc_prepare_b<kC>(cv[1], threadIdx.x + 128, b_buf(gslot), cbf_slot(gslot), ctl, gslot, 1);
        }
        X_nxt = 0.f;
#pragma unroll
        for (int w = 0; w < kC / 2; ++w) {
            xw_nxt[w] = xw_pf[w];
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&xw_pf[w]));
            X_nxt = fmaf(f.x, f.x, X_nxt);
            X_nxt = fmaf(f.y, f.y, X_nxt);
        }
        tc_build_a<kC>(xw_pf, X_nxt, a_buf(st & 1), row);
    };
    // the MMA of one half of step st (half 1 = centroids 128 ... 255), then the commit that arrives on that half's
    // barrier when it is done
    auto issue = [&](int st, int half) {
        const uint32_t a0 = tc_smem_u32(a_buf(st & 1)), b0 = tc_smem_u32(b_buf((st >> log_rt) & 1)) + half * (128 * 16);
#pragma unroll
        for (int s = 0; s < C::kSteps; ++s)
            tc_mma(tmem_base, tc_desc(a0 + s * C::kATile, 128 * 16), tc_desc(b0 + s * C::kBTile, 256 * 16), s > 0 ? 1u : 0u);
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem_u32(&ctl->bar[half])) : "memory");
    };
    // minima of the 16 subsets (centroid index mod 16) over the 128 scores of the half that is in tensor memory
    auto scan_half = [&](float (&sb)[16]) {
        float va[32], vb[32];
        auto consume = [&](const float (&v)[32]) {
#pragma unroll
            for (int q = 0; q < 16; ++q) sb[q] = tc_min3(sb[q], v[q], v[q + 16]);
        };
        tc_ld32_issue(va, taddr);
        tc_ld_wait(va);
        tc_ld32_issue(vb, taddr + 32);
        consume(va);
        tc_ld_wait(vb);
        tc_ld32_issue(va, taddr + 64);
        consume(vb);
        tc_ld_wait(va);
        tc_ld32_issue(vb, taddr + 96);
        consume(va);
        tc_ld_wait(vb);
        consume(vb);
    };

    fetch(0);
    build(0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        issue(0, 0);
    }

    for (int st = 0; st < n_steps; ++st) {
        const int g = g_begin + (st >> log_rt), slot = (st >> log_rt) & 1;
        uint32_t xw[kC / 2];
#pragma unroll
        for (int w = 0; w < kC / 2; ++w) xw[w] = xw_nxt[w];
        const float X = X_nxt;
        if (st + 1 < n_steps) fetch(st + 1);

        bool scores_valid = *reinterpret_cast<volatile int*>(&ctl->wait_failed) == 0;
        if (scores_valid && !tc_wait(&ctl->bar[0], (uint32_t)(st & 1))) {
            ctl->wait_failed = 1;                        // never expected: every row of this CTA goes the exact way from here on
            scores_valid = false;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float sb[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) sb[q] = kTcInf;
        scan_half(sb);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();                                 // the low half has been read: its columns take the high half
        if (threadIdx.x == 0 && *reinterpret_cast<volatile int*>(&ctl->wait_failed) == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue(st, 1);
        }
        if (st + 1 < n_steps) build(st + 1);             // while the MMA of the high half runs

        if (scores_valid && !tc_wait(&ctl->bar[1], (uint32_t)(st & 1))) {
            ctl->wait_failed = 1;
            scores_valid = false;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        scan_half(sb);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();                                 // tensor memory is free again; the operands of step st + 1 are complete
        if (threadIdx.x == 0 && st + 1 < n_steps && *reinterpret_cast<volatile int*>(&ctl->wait_failed) == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            issue(st + 1, 0);
        }

        // control words of this step's group
        bool out_of_range;
        float nmax;
        {
            const int4 f0 = *reinterpret_cast<const int4*>(&ctl->range_flag[slot][0]);
            const int4 f1 = *reinterpret_cast<const int4*>(&ctl->range_flag[slot][4]);
            out_of_range = (f0.x | f0.y | f0.z | f0.w | f1.x | f1.y | f1.z | f1.w) != 0;
            const float4 m0 = *reinterpret_cast<const float4*>(&ctl->nmax[slot][0]);
            const float4 m1 = *reinterpret_cast<const float4*>(&ctl->nmax[slot][4]);
            nmax = fmaxf(fmaxf(fmaxf(m0.x, m0.y), fmaxf(m0.z, m0.w)), fmaxf(fmaxf(m1.x, m1.y), fmaxf(m1.z, m1.w)));
        }
        const float* cbf = cbf_slot(slot);

        // smallest and second smallest subset minimum (a tournament of (smallest, second) pairs); the subset number
        // rides in the low four mantissa bits, which also makes the 16 values differ
        float m1v, s2;
        {
            float lo[8], hi[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float ta = __uint_as_float((__float_as_uint(sb[2 * i]) & ~15u) | (uint32_t)(2 * i));
                const float tb = __uint_as_float((__float_as_uint(sb[2 * i + 1]) & ~15u) | (uint32_t)(2 * i + 1));
                lo[i] = fminf(ta, tb);
                hi[i] = fmaxf(ta, tb);
            }
#pragma unroll
            for (int n = 4; n >= 1; n >>= 1)
#pragma unroll
                for (int i = 0; i < n; ++i) {
                    const float m = fminf(lo[i], lo[i + n]);
                    hi[i] = tc_min3(fmaxf(lo[i], lo[i + n]), hi[i], hi[i + n]);
                    lo[i] = m;
                }
            m1v = lo[0];
            s2 = hi[0];
        }
        const int qw = (int)(__float_as_uint(m1v) & 15u);
        float xg[kC];
#pragma unroll
        for (int w = 0; w < kC / 2; ++w) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&xw[w]));
            xg[2 * w] = f.x;
            xg[2 * w + 1] = f.y;
        }
        // the winner's subset, exactly: centroids qw, qw + 16, ..., qw + 240; the smallest distance by a tournament in
        // which the lower index wins ties
        float dk[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int j = qw + 16 * k;
            float cc[kC];
            if (kC == 2) {
                const float2 t2 = *reinterpret_cast<const float2*>(cbf + j * 2);
                cc[0] = t2.x; cc[1] = t2.y;
            } else {
#pragma unroll
                for (int w = 0; w < kC; w += 4) {
                    const float4 t4 = *reinterpret_cast<const float4*>(cbf + j * kC + w);
                    cc[w] = t4.x; cc[w + 1] = t4.y; cc[(w + 2) % kC] = t4.z; cc[(w + 3) % kC] = t4.w;
                }
            }
            float dd = 0.f;
#pragma unroll
            for (int i = 0; i < kC; ++i) {
                const float diff = xg[i] - cc[i];
                dd = fmaf(diff, diff, dd);
            }
            dk[k] = dd;
        }
        int ik[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const bool right = dk[2 * i + 1] < dk[2 * i];        // strict: the lower index keeps a tie
            ik[i] = right ? 2 * i + 1 : 2 * i;
            dk[i] = right ? dk[2 * i + 1] : dk[2 * i];
        }
#pragma unroll
        for (int n = 4; n >= 1; n >>= 1)
#pragma unroll
            for (int i = 0; i < n; ++i) {
                const bool right = dk[2 * i + 1] < dk[2 * i];
                ik[i] = right ? ik[2 * i + 1] : ik[2 * i];
                dk[i] = right ? dk[2 * i + 1] : dk[2 * i];
            }
        float dbest = dk[0];
        int code = qw + 16 * ik[0];
        // Evaluation error of a score: fp32 accumulation of up to ~20 terms bounded by 2 (X + N) in magnitude, plus
        // the four mantissa bits given to the subset number.  dbest is exact.
        const float ss = __uint_as_float(__float_as_uint(s2) & ~15u);
        const float tau = 1.6e-5f * (X + nmax) + 4e-6f * fabsf(ss);
        const bool certain = scores_valid && !out_of_range && (ss - dbest > tau);
        const TcRow rec = rows[(st & rt_mask) * kTcThreads];
        const bool live = rec.x != nullptr;
        // exact recomputation of the uncertain rows, one row at a time by the whole warp
        unsigned pending = __ballot_sync(0xffffffffu, !certain && live);
        while (pending) {
            const int src = __ffs(pending) - 1;
            pending &= pending - 1;
            float xs[kC];
#pragma unroll
            for (int w = 0; w < kC / 2; ++w) {
                const uint32_t ww = __shfl_sync(0xffffffffu, xw[w], src);
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww));
                xs[2 * w] = f.x;
                xs[2 * w + 1] = f.y;
            }
            float ed;
            const int ec = tc_exact_code<kC>(xs, cbf, lane, &ed);
            if (lane == src) { code = ec; dbest = ed; }
        }
        if (rec.code_offset >= 0) codes[rec.code_offset + g * kTokenBlock] = (uint8_t)code;
    }

    // every MMA that was issued has been waited for (or the wait gave up); hand the tensor memory back
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTcColumns) : "memory");
    }
}

template <int kC>
cudaError_t launch_enc_tc(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh, int64_t n_tokens,
                          int64_t token_offset, uint8_t* codes, cudaStream_t st, const __half* x2, const float* cb2, uint8_t* codes2)
{
    using C = TcCfg<kC>;
    const int64_t n_vec = sh.n_seq * n_tokens;
    const int64_t tiles = (n_vec + kTcTileVecs - 1) / kTcTileVecs;
    const int64_t slots = C::kCtasPerSm * (int64_t)device_sm_count();          // CTAs in flight
    // row tiles per CTA: as many as leave four waves of CTAs
    int log_rt = C::kMaxLogRt;
    while (log_rt > 0 && ((tiles + (1 << log_rt) - 1) >> log_rt) * sh.n_kv_heads < 4 * slots) --log_rt;
    const int64_t blocks = (tiles + (1 << log_rt) - 1) >> log_rt;
    // split the groups over CTAs while the grid would leave SMs idle
    int64_t n_gsplit = (slots + blocks * sh.n_kv_heads - 1) / (blocks * sh.n_kv_heads);
    if (n_gsplit > C::G) n_gsplit = C::G;
    if (n_gsplit < 1) n_gsplit = 1;
    const int groups_per_cta = (int)((C::G + n_gsplit - 1) / n_gsplit);
    n_gsplit = (C::G + groups_per_cta - 1) / groups_per_cta;
    const int64_t grid = blocks * sh.n_kv_heads * n_gsplit;
    if (grid > 0x7fffffff) return cudaErrorInvalidConfiguration;
    constexpr int kSlot = 44 + (kC == 2 ? 0 : kC == 4 ? 1 : 2);       // call-site slots 44 ... 46 of ensure_dynamic_smem
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(encode_tc_kernel<kC>), C::kSmemBytes, kSlot);
    if (e != cudaSuccess) return e;
    encode_tc_kernel<kC><<<dim3((unsigned)grid, x2 ? 2u : 1u), kTcThreads, C::kSmemBytes, st>>>(
        x, cb, seq_offsets, sh, n_tokens, token_offset, codes, groups_per_cta, log_rt, x2, cb2, codes2);
    return cudaGetLastError();
}

}  // namespace

bool encode_tc_supported(const Shape& sh)
{
    return sh.head_dim == 128 && sh.b == 8 && (sh.c == 2 || sh.c == 4 || sh.c == 8);
}

cudaError_t launch_encode_tc(const __half* x, const float* cb, const int32_t* seq_offsets, const Shape& sh, int64_t n_tokens,
                             int64_t token_offset, uint8_t* codes, cudaStream_t st, const __half* x2, const float* cb2, uint8_t* codes2)
{
    if (sh.n_seq * n_tokens == 0) return cudaSuccess;
    switch (sh.c) {
        case 2: return launch_enc_tc<2>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
        case 4: return launch_enc_tc<4>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
        case 8: return launch_enc_tc<8>(x, cb, seq_offsets, sh, n_tokens, token_offset, codes, st, x2, cb2, codes2);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace cq
