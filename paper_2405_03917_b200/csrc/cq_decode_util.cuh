// Device helpers shared by the tuned decode-attention kernels (sm_100a).
#pragma once

#include "cq_common.cuh"

namespace cq {

namespace {

constexpr int kRows = 256;            // code values
constexpr int kRowBytes = 256;        // bytes per table row
constexpr int kUnitBits = 27;         // weight of the running-maximum token: (2^26, 2^27]
constexpr int kMaxWeightBits = 30;    // a score may exceed the unit exponent by at most this
constexpr unsigned int kBinLimit256 = 16000000u;   // bins stay below 2^32: bound on their sum, in units of 256
constexpr int kUnset = INT_MIN;                    // no score seen yet

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

// Barrier 1 of the CTA, for the coarsening events: warps reach it from different places of the
// code (bar.sync counts arrivals per barrier, whatever instruction they come from).
__device__ __forceinline__ void event_barrier(int n_threads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(n_threads) : "memory");
}

// 2^d for an integer d; 0 below the normal range, saturates at 2^127
__device__ __forceinline__ float pow2i(int d)
{
    d = d > 127 ? 127 : d;
    return d < -126 ? 0.f : __int_as_float((127 + d) << 23);
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One centroid into registers.  The asm statements keep the loads where the code puts them: the
// units of a codebook are loaded one unit ahead of their use, not all at once.
__device__ __forceinline__ float4 ldg_f4(const float* p)
{
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
// `wide`: an 8-channel centroid is one 32-byte load (the lanes of a warp then read one contiguous
// KiB; two 16-byte loads at a 32-byte lane stride touch every sector twice).  Needs 32-byte
// aligned codebooks, which the launcher checks.
template <int kC>
__device__ __forceinline__ void load_centroid(const float* p, float (&cv)[kC], bool wide)
{
    static_assert(kC == 2 || kC == 4 || kC == 8, "centroids of 2, 4 or 8 channels");
    if (kC == 2) {
        asm volatile("ld.global.nc.v2.f32 {%0,%1}, [%2];" : "=f"(cv[0]), "=f"(cv[1 % kC]) : "l"(p) : "memory");
        return;
    }
    if (kC == 8 && wide) {
        asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(cv[0]), "=f"(cv[1]), "=f"(cv[2]), "=f"(cv[3]), "=f"(cv[4 % kC]), "=f"(cv[5 % kC]),
                       "=f"(cv[6 % kC]), "=f"(cv[7 % kC])
                     : "l"(p) : "memory");
        return;
    }
    const float4 a = ldg_f4(p);
    cv[0] = a.x; cv[1 % kC] = a.y; cv[2 % kC] = a.z; cv[3 % kC] = a.w;
    if (kC == 8) {
        const float4 b = ldg_f4(p + 4);
        cv[4 % kC] = b.x; cv[5 % kC] = b.y; cv[6 % kC] = b.z; cv[7 % kC] = b.w;
    }
}

// Work items are handed out longest context first: with contexts of different lengths the CTAs that start
// last are then the short ones, and the launch ends more evenly.  Returns the sequence whose context is the
// `rank`-th longest (ties: lower index first).  Every warp finds it by itself - lane j holds the length of
// sequence j and counts, by shuffles, the sequences that come before its own - so no barrier and no shared
// memory are needed.  Batches of more than 32 sequences keep their own order (the search would cost more
// than it gains).  Entered by whole warps.
__device__ __forceinline__ int seq_by_rank(const int32_t* __restrict__ seq_lens, int n_seq, int64_t max_tokens, int rank)
{
    if (n_seq > 32 || n_seq < 2) return rank;
    const int lane = threadIdx.x & 31;
    int mine = lane < n_seq ? seq_lens[lane] : -1;
    mine = mine < 0 ? (lane < n_seq ? 0 : -1) : (mine > max_tokens ? (int)max_tokens : mine);
    int before = 0;
    for (int k = 0; k < n_seq; ++k) {
        const int other = __shfl_sync(0xffffffffu, mine, k);
        before += (other > mine || (other == mine && k < lane)) ? 1 : 0;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, lane < n_seq && before == rank);
    return hit ? __ffs(hit) - 1 : rank;
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

}  // namespace

}  // namespace cq
