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
// Integer adds are also associative, so a bin does not depend on the order in which warps
// reach it.  Every query head has its own unit exponent e: it starts 27 bits below the first
// scores' maximum, and it is coarsened (bins shifted right, with rounding) only when a score
// would need more than 30 bits or the running total of the weights - a bound on every bin -
// would pass 2^32.  Warps reserve their weights on that total with one atomic add and do not
// wait for each other; a coarsening is a rare event that every warp joins (see `coarsen`).
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
#include "cq_decode_util.cuh"

namespace cq {

namespace {


template <int G, int R>
struct Cfg {
    static_assert(G == 16 || G == 32 || (G == 64 && R == 1), "tuned decode kernels cover 16, 32 and (one query head) 64 groups");
    static constexpr int kC = 128 / G;                                  // channels per group
    // 64 groups: the two half warps take the same four 16-token blocks, quads 0-3 the groups 0-31 and quads
    // 4-7 the groups 32-63 (second plane of a table row); they exchange their partial scores with one shuffle.
    static constexpr bool kHalfGroups = (G == 64);
    static constexpr bool kHalfRows = (G == 16);                         // quads 0-3 / 4-7 use different 16-word halves
    static constexpr bool kReplica = (G == 16 && R == 1);                // the two halves are copies of one table
    static constexpr int kLaneHeads = (G == 16 && R >= 2) ? R / 2 : R;   // query heads a lane serves
    static constexpr int kPlanes = kHalfGroups ? 2 : kLaneHeads;         // 32-word planes per table row
    static constexpr int kSlots = kHalfGroups ? 8 : G / 4;               // code words (16 tokens each) per lane
    static constexpr int kBlocksPerIter = ((G == 16 && R >= 2) || kHalfGroups) ? 4 : 8;   // 16-token blocks per warp iteration
    static constexpr int kWarps = (kPlanes == 1) ? 8 : 16;
    static constexpr int kThreads = kWarps * 32;
    static constexpr int kMinBlocks = (kPlanes == 1) ? 2 : 1;     // 128 registers per thread in every configuration
    static constexpr int kRoundTokens = kWarps * kBlocksPerIter * 16;    // tokens a CTA handles per iteration
    static_assert(kPlanes == 1 || kPlanes == 2, "table rows hold one or two planes");
    // One plane: K and V planes share a row (K at +0, V at +128).  Two planes: separate tables.
    static constexpr int kVOffset = (kPlanes == 1) ? 128 : kRows * kRowBytes;
    static constexpr int kTableBytes = (kPlanes == 1) ? kRows * kRowBytes : 2 * kRows * kRowBytes;
    static constexpr int kNewOffset = 128 + R * 128 * 4;                 // codes of an appended token: [key | value][64 groups]
    static constexpr int kCtlBytes = kNewOffset + 128;                   // control words + scaled query + those codes
    static constexpr int kSmemBytes = kTableBytes + kCtlBytes;

    // word inside a plane that lane (r, p) uses for its m-th code word
    __device__ static __forceinline__ int word(int r, int p, int m)
    {
        return kHalfRows ? 16 * (r >> 2) + 4 * ((r + m) & 3) + p : 4 * ((r + m) & 7) + p;
    }
    // group of a table word, and the (plane, word) that holds (group g, query head h of the KV head)
    __device__ static __forceinline__ int group_of(int w) { return kHalfRows ? (w & 15) : w; }
    __device__ static __forceinline__ int plane_of(int g, int h)
    {
        return kHalfGroups ? g >> 5 : (kHalfRows ? (R <= 2 ? 0 : h >> 1) : h);
    }
    __device__ static __forceinline__ int word_of(int g, int h)
    {
        return kHalfGroups ? (g & 31) : (kHalfRows ? (R == 1 ? 0 : (h & 1) * 16) + g : g);
    }
    // byte offset, inside a table row, of the plane that lane row r uses by itself (64 groups only)
    __device__ static __forceinline__ unsigned lane_plane_bytes(int r) { return kHalfGroups ? 128u * (unsigned)(r >> 2) : 0u; }
    // query head (of the KV head) that lane row r serves as its u-th head, and the head a table word belongs to
    __device__ static __forceinline__ int lane_head(int u, int r) { return kHalfRows ? (R == 1 ? 0 : 2 * u + (r >> 2)) : u; }
    __device__ static __forceinline__ int head_of_word(int word_in_row)
    {
        const int plane = word_in_row >> 5, w = word_in_row & 31;
        return kHalfGroups ? 0 : (kHalfRows ? (R == 1 ? 0 : 2 * plane + (w >> 4)) : plane);
    }
    // v[lane_head(u, r)] without indexing a register array by a run-time value
    template <int N>
    __device__ static __forceinline__ int pick(const int (&v)[N], int u, int r)
    {
        int out = v[0];
#pragma unroll
        for (int h = 1; h < N; ++h) out = lane_head(u, r) == h ? v[h] : out;
        return out;
    }
    static constexpr int kLog2Groups = kWarps == 16 ? 4 : 3;             // log2 of the warps that add to a head's bins per round
    static constexpr int kGroupsPerWarp = G / kWarps;
    static_assert(G % kWarps == 0 && kSlots % 4 == 0, "ownership of groups by warps; four code words per MMA");
};

struct Ctl {
    int e_cur[4];              // per query head: log2 of the weight unit of its bins (kUnset before the first tokens)
    unsigned int total[4];     // per query head: bound, in units of 256, on the sum of the weights added since the last coarsening
    int req_ref[4];            // coarsening request: largest score exponent the requesters need to represent
    int req_need[4];           // coarsening request: log2 bound of the largest round sum of one (half) warp
    int want;                  // non-zero: a warp asks every warp to stop adding and coarsen
    float lut_absmax;          // largest |LUT| entry, as float bits (non-negative, so int order works)
};
static_assert(sizeof(Ctl) <= 128, "control block");


// D = A * ones (+ C): sums, per fragment row, the 16 halves the quad holds for that row.
// Rows r (registers a0, a2) and r + 8 (a1, a3) carry two different tokens.
__device__ __forceinline__ void mma_rowsum_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3)
{
    const uint32_t ones = 0x3c003c00u;   // half2(1, 1)
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(ones), "r"(ones), "f"(0.f));
}
__device__ __forceinline__ void mma_rowsum_acc(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3)
{
    const uint32_t ones = 0x3c003c00u;
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(ones), "r"(ones));
}


// half2 (hi, lo) with hi + lo ~= v to about 22 bits: hi in the low half, lo in the high half
__device__ __forceinline__ uint32_t pack_hi_lo(float v)
{
    const __half hi = __float2half_rn(v);
    const __half lo = __float2half_rn(v - __half2float(hi));
    return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
}

// Sum of a[0..kC) over the 32 lanes of a warp, with the channels folded while they are exchanged:
// the step with lane mask 16 keeps half of the channels in each half warp, and so on, so that
// after log2(kC) steps every lane holds one channel; the remaining steps finish that channel.
// The result of lane L is the total of channel fold_channel_of<kC>(L).
template <int kC>
__device__ __forceinline__ int fold_channel_of(int lane)
{
    return kC == 8 ? ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1)
                   : ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
}
template <int kC>
__device__ __forceinline__ float fold_channels(const float (&a)[kC], int lane)
{
    float h4[kC / 2];
    {
        const bool up = lane & 16;
#pragma unroll
        for (int i = 0; i < kC / 2; ++i) {
            const float keep = up ? a[i + kC / 2] : a[i];
            const float send = up ? a[i] : a[i + kC / 2];
            h4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
    }
    float h2[kC / 4];
    {
        const bool up = lane & 8;
#pragma unroll
        for (int i = 0; i < kC / 4; ++i) {
            const float keep = up ? h4[i + kC / 4] : h4[i];
            const float send = up ? h4[i] : h4[i + kC / 4];
            h2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
    }
    float v;
    if (kC == 8) {
        const bool up = lane & 4;
        const float keep = up ? h2[1 % (kC / 4)] : h2[0];
        const float send = up ? h2[0] : h2[1 % (kC / 4)];
        v = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    } else {
        v = h2[0] + __shfl_xor_sync(0xffffffffu, h2[0], 4);
    }
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v;
}


// byte k (0..15) of a 16-byte code word replaced
__device__ __forceinline__ void put_code(uint4& w, int k, uint32_t code)
{
    const uint32_t keep = ~(0xffu << (8 * (k & 3))), put = code << (8 * (k & 3));
    if ((k >> 2) == 0) w.x = (w.x & keep) | put;
    else if ((k >> 2) == 1) w.y = (w.y & keep) | put;
    else if ((k >> 2) == 2) w.z = (w.z & keep) | put;
    else w.w = (w.w & keep) | put;
}

// The value codes of the token that the launch appends (CQ encode, Section 3.2), by the whole CTA: a warp takes
// the groups it owns, its lanes walk the centroids; d_j = sum_i (x_i - C_ji)^2 in fp32 in the order of the encode
// kernels, lowest index on ties.  The codes go to newcode[g] and, from the CTA that `writer` names, to position
// `pos` of the cache.  (The key codes come out of the table build, which reads the key centroids anyway.)
template <int kC, int kGroupsPerWarp>
__device__ __noinline__ void encode_new_value_tuned(uint8_t* newcode, const __half* __restrict__ v_new, uint8_t* vc_w,
                                                    const float* __restrict__ vcb, Shape sh, int64_t s, int hkv, int64_t pos,
                                                    bool writer)
{
    constexpr int G = 128 / kC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll 1
    for (int e = 0; e < kGroupsPerWarp; ++e) {
        const int g = warp * kGroupsPerWarp + e;
        const __half* xp = v_new + (s * sh.n_kv_heads + hkv) * 128 + g * kC;
        const float* cg = vcb + ((int64_t)hkv * G + g) * kRows * kC;
        float xg[kC];
#pragma unroll
        for (int i = 0; i < kC; ++i) xg[i] = __half2float(xp[i]);
        float cv[kRows / 32][kC];                     // all loads in flight at once
#pragma unroll
        for (int t = 0; t < kRows / 32; ++t) load_centroid<kC>(cg + (int64_t)(t * 32 + lane) * kC, cv[t], false);
        float best = INFINITY;
        int arg = 0;
#pragma unroll
        for (int t = 0; t < kRows / 32; ++t) {
            float d = 0.f;
#pragma unroll
            for (int i = 0; i < kC; ++i) {
                const float diff = xg[i] - cv[t][i];
                d = fmaf(diff, diff, d);
            }
            if (d < best) { best = d; arg = t * 32 + lane; }        // ascending: strict < keeps the lowest index
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
            if (ob < best || (ob == best && oa < arg)) { best = ob; arg = oa; }
        }
        if (lane == 0) {
            newcode[g] = (uint8_t)arg;
            if (writer) vc_w[code_word_offset(sh, sh.n_kv_heads, s, hkv, pos / kTokenBlock, g) + pos % kTokenBlock] = (uint8_t)arg;
        }
    }
}

// kAppend: the launch also encodes and appends one token per sequence (a second instance, so that the plain attention
// carries none of that code)
template <int G, int R, bool kShared, bool kAppend>
__global__ void __launch_bounds__(Cfg<G, R>::kThreads, Cfg<G, R>::kMinBlocks)
decode_tuned_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                    const float* __restrict__ kcb, const float* __restrict__ vcb,
                    const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int chunk_tokens, int n_parts,
                    int tail_first, int cb_aligned32, int kv_share, float* __restrict__ partials, float* __restrict__ out,
                    AppendArgs app)
{
    // out: non-null only when every item is one part; the CTA then normalises its partial itself (no merge launch).
    // R is the number of query heads one CTA serves.  A KV head with more query heads than that
    // (kv_share groups of R; kShared) is served by kv_share CTAs, which read the same codes and codebooks.
    using C = Cfg<G, R>;
    constexpr int kC = C::kC;
    extern __shared__ __align__(1024) uint8_t smem[];
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + C::kTableBytes);
    float* qs = reinterpret_cast<float*>(smem + C::kTableBytes + 128);     // [R][128], scaled by scale*log2(e)

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, p = lane & 3;

    // Work item: (context part, sequence, KV head); parts are the slowest index so that the
    // always-populated first parts start first.  With a tail (tail_first >= 0) the items before
    // tail_first take their whole context in one CTA, and each later item is spread over n_parts
    // CTAs of chunk_tokens each: those shorter CTAs start last and fill the last, partly empty
    // wave of the grid.
    const int n_head_groups = kShared ? sh.n_q_heads / R : sh.n_kv_heads;
    const int n_items = (int)(n_head_groups * sh.n_seq);
    int item = blockIdx.x % n_items;
    int part = (int)(blockIdx.x / n_items);
    bool whole = false;
    if (tail_first >= 0) {
        whole = (int)blockIdx.x < tail_first;
        item = whole ? blockIdx.x : tail_first + (blockIdx.x - tail_first) / n_parts;
        part = whole ? 0 : (blockIdx.x - tail_first) % n_parts;
    }
    const int head_group = item % n_head_groups;      // query heads head_group * R ... + R - 1
    const int hkv = kShared ? head_group / kv_share : head_group;
    const int64_t s = seq_by_rank(seq_lens, (int)sh.n_seq, sh.max_tokens, item / n_head_groups);

    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    // With an append, seq_lens counts the tokens cached before this launch: the new token takes position n and
    // the attention covers n + 1 tokens (a sequence at capacity gets no new token).
    const bool has_new = kAppend && app.k_new != nullptr && n < sh.max_tokens;
    if (has_new) ++n;
    const int64_t t_begin = (int64_t)part * chunk_tokens;
    const int64_t t_end = (whole || t_begin + chunk_tokens >= n) ? n : t_begin + chunk_tokens;
    const int stride = partial_stride(128);
    float* part_base = partials + ((s * sh.n_q_heads + (int64_t)head_group * R) * n_parts + part) * stride;
    // partial of query head head_group*R + h: part_base + h * n_parts * stride
    if (whole)          // the other partial slots of this item hold the neutral element of the merge
        for (int i = threadIdx.x; i < R * (n_parts - 1) * stride; i += C::kThreads) {
            const int h = i / ((n_parts - 1) * stride), d = i % ((n_parts - 1) * stride);
            part_base[(int64_t)h * n_parts * stride + stride + d] = d % stride == 0 ? -INFINITY : 0.f;
        }
    if (t_begin >= t_end) {
        for (int i = threadIdx.x; i < R * stride; i += C::kThreads) {
            const int h = i / stride, d = i % stride;
            part_base[(int64_t)h * n_parts * stride + d] = d == 0 ? -INFINITY : 0.f;
        }
        if (out)            // nothing to attend: the zero row of the merge
            for (int i = threadIdx.x; i < R * 128; i += C::kThreads) out[(s * sh.n_q_heads + (int64_t)head_group * R) * 128 + i] = 0.f;
        return;
    }

    // ---------------------------------------------------------------- addresses; the first centroids travel during the set-up
    const int64_t blk0 = t_begin / kTokenBlock;
    const int64_t blk_lim = (t_end + kTokenBlock - 1) / kTokenBlock;       // blocks holding a valid token
    const int n_iters = (int)((t_end - t_begin + C::kRoundTokens - 1) / C::kRoundTokens);
    const int qb = (C::kBlocksPerIter == 8) ? r : (r & 3);                 // block of this quad inside the warp's iteration
    // The new token, when its position is in this CTA's range: the CTA works its codes out itself (so do the CTAs of
    // the other query heads that share the KV head) and puts them into the code words it loads of that block; one
    // CTA per KV head also writes them to the cache.
    const bool new_here = kAppend && has_new && t_begin <= n - 1 && n - 1 < t_end;
    const int64_t new_blk = (n - 1) / kTokenBlock;
    const int new_tok = (int)((n - 1) % kTokenBlock);
    const bool new_writer = !kShared || head_group % kv_share == 0;
    uint8_t* newcode = smem + C::kTableBytes + C::kNewOffset;               // [key | value][64]
    uint32_t lane_off[C::kSlots];      // byte offset of this lane's word inside a plane, per code word
#pragma unroll
    for (int m = 0; m < C::kSlots; ++m) lane_off[m] = 4u * C::word(r, p, m) + C::lane_plane_bytes(r);
    // code words of this lane: word (block, group) sits at (block * G + group) * 16 bytes
    const uint8_t* kbase = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint8_t* vbase = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);

    uint4 kw[C::kSlots], vw[C::kSlots];
    auto load_words = [&](uint4 (&dst)[C::kSlots], const uint8_t* base, int64_t blk) {
        if (blk < blk_lim) {
            const uint8_t* bp = base + blk * (G * kTokenBlock);
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m)
                dst[m] = ldg_codes(reinterpret_cast<const uint4*>(bp + C::group_of(lane_off[m] >> 2) * kTokenBlock));
            if (kAppend && new_here && blk == new_blk) {
                const uint8_t* nc = newcode + (base == vbase ? 64 : 0);
#pragma unroll
                for (int m = 0; m < C::kSlots; ++m) put_code(dst[m], new_tok, nc[C::group_of(lane_off[m] >> 2)]);
            }
        } else {
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m) dst[m] = make_uint4(0u, 0u, 0u, 0u);
        }
    };

    // Codebooks are read in units of kJb * 32 centroids (32 registers per lane): a warp owns whole
    // groups, its lanes walk the code values, and the next unit is loaded while the current one is used.
    constexpr int kJb = (kC == 8) ? 4 : 8;
    constexpr int kUnitsPerGroup = (kRows / 32) / kJb;
    constexpr int kUnits = C::kGroupsPerWarp * kUnitsPerGroup;
    static_assert(kUnits % 2 == 0, "units are taken in pairs");
    auto load_unit = [&](float (&cv)[kJb][kC], const float* cb, int u) {
        const int g = warp * C::kGroupsPerWarp + u / kUnitsPerGroup;
        const float* cg = cb + (((int64_t)hkv * G + g) * kRows + (u % kUnitsPerGroup) * kJb * 32 + lane) * kC;
#pragma unroll
        for (int jb = 0; jb < kJb; ++jb) load_centroid<kC>(cg + jb * 32 * kC, cv[jb], cb_aligned32 != 0);
    };
    float cva[kJb][kC], cvb[kJb][kC];
    load_unit(cva, kcb, 0);

    // ---------------------------------------------------------------- set-up: query, LUT, bins
    if (threadIdx.x < 4) {
        ctl->e_cur[threadIdx.x] = kUnset;
        ctl->total[threadIdx.x] = 0u;
        ctl->req_ref[threadIdx.x] = kUnset;
        ctl->req_need[threadIdx.x] = kUnset;
    }
    if (threadIdx.x == 4) { ctl->want = 0; ctl->lut_absmax = 0.f; }
    for (int i = threadIdx.x; i < R * 128; i += C::kThreads)
        qs[i] = __half2float(q[(s * sh.n_q_heads + (int64_t)head_group * R) * 128 + i]) * scale_log2e;
    // bins start at zero (16-byte stores over the V planes)
    for (int i = threadIdx.x; i < kRows * 8 * C::kPlanes; i += C::kThreads)
        *reinterpret_cast<uint4*>(smem + C::kVOffset + (i / (8 * C::kPlanes)) * kRowBytes + (i % (8 * C::kPlanes)) * 16) =
            make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();

    // Table build.  A warp owns whole groups and its lanes walk the code values j, so the
    // codebook is read in contiguous runs.  A column of the table (fixed word, 32 consecutive
    // rows) would fall into one bank, so the build writes row j rotated by j words and a second
    // pass un-rotates every row.  Entries are half2 (hi, lo) of LUT * 2^-kexp; kexp = 0 unless an
    // entry reaches 2^15 (then the build is repeated once with the exponent that fits).
    if (kAppend && new_here)
        encode_new_value_tuned<kC, C::kGroupsPerWarp>(newcode + 64, app.v_new, app.vc_w, vcb, sh, s, hkv, n - 1, new_writer);
    // the new token's key, when this CTA appends it: its code of group g is the centroid nearest to it, found on the
    // way (d_j = sum_i (x_i - C_ji)^2 in fp32 in the order of the encode kernels, lowest index on ties)
    float xnew[kC], dnew = INFINITY;
    int jnew = 0;
    float lut_scale = 1.f;           // scores in table units * lut_scale = log2-domain scores
    for (int attempt = 0; attempt < 2; ++attempt) {
        const float inv = 1.f / lut_scale;
        float absmax = 0.f;
        const bool find_key = kAppend && new_here && attempt == 0;
        auto build_unit = [&](const float (&cv)[kJb][kC], int u) {
            const int g = warp * C::kGroupsPerWarp + u / kUnitsPerGroup;
            if (kAppend && find_key && u % kUnitsPerGroup == 0) {
                const __half* xp = app.k_new + (s * sh.n_kv_heads + hkv) * 128 + g * kC;
#pragma unroll
                for (int i = 0; i < kC; ++i) xnew[i] = __half2float(xp[i]);
                dnew = INFINITY;
                jnew = 0;
            }
            float qreg[R][kC];
#pragma unroll
            for (int h = 0; h < R; ++h)
#pragma unroll
                for (int i = 0; i < kC; ++i) qreg[h][i] = qs[h * 128 + g * kC + i] * inv;
#pragma unroll
            for (int jb = 0; jb < kJb; ++jb) {
                const int j = ((u % kUnitsPerGroup) * kJb + jb) * 32 + lane;
#pragma unroll
                for (int h = 0; h < R; ++h) {
                    float dot = 0.f;
#pragma unroll
                    for (int i = 0; i < kC; ++i) dot = fmaf(qreg[h][i], cv[jb][i], dot);
                    absmax = fmaxf(absmax, fabsf(dot));
                    const uint32_t e = pack_hi_lo(dot);
                    uint8_t* row = smem + j * kRowBytes + C::plane_of(g, h) * 128;
                    *reinterpret_cast<uint32_t*>(row + ((C::word_of(g, h) + j) & 31) * 4) = e;
                    if (C::kReplica) *reinterpret_cast<uint32_t*>(row + ((16 + g + j) & 31) * 4) = e;
                }
                if (kAppend && find_key) {
                    float d = 0.f;
#pragma unroll
                    for (int i = 0; i < kC; ++i) {
                        const float diff = xnew[i] - cv[jb][i];
                        d = fmaf(diff, diff, d);
                    }
                    if (d < dnew) { dnew = d; jnew = j; }        // a lane's j ascend: strict < keeps the lowest index
                }
            }
            if (kAppend && find_key && u % kUnitsPerGroup == kUnitsPerGroup - 1) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, dnew, o);
                    const int oa = __shfl_xor_sync(0xffffffffu, jnew, o);
                    if (ob < dnew || (ob == dnew && oa < jnew)) { dnew = ob; jnew = oa; }
                }
                if (lane == 0) {
                    newcode[g] = (uint8_t)jnew;
                    if (new_writer)
                        app.kc_w[code_word_offset(sh, sh.n_kv_heads, s, hkv, (n - 1) / kTokenBlock, g) + (n - 1) % kTokenBlock] = (uint8_t)jnew;
                }
            }
        };
        if (attempt == 1) load_unit(cva, kcb, 0);
#pragma unroll 1
        for (int u = 0; u < kUnits; u += 2) {
            load_unit(cvb, kcb, u + 1);
            build_unit(cva, u);
            if (u + 2 < kUnits) load_unit(cva, kcb, u + 2);
            build_unit(cvb, u + 1);
        }
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 16));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 8));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 4));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 2));
        absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, 1));
        if (lane == 0) atomicMax(reinterpret_cast<int*>(&ctl->lut_absmax), __float_as_int(absmax));
        __syncthreads();
        const float amax = ctl->lut_absmax;
        if (attempt == 1 || amax < 32768.f) break;       // same decision in every thread
        int ex;
        frexpf(amax, &ex);                                // amax < 2^ex
        lut_scale = exp2f((float)(ex - 15));
        __syncthreads();
        if (threadIdx.x == 0) ctl->lut_absmax = 0.f;
        __syncthreads();
    }
    // un-rotate: a warp owns rows warp, warp + kWarps, ...; eight (row, plane) pairs per step
    constexpr int kOwnRowPlanes = kRows / C::kWarps * C::kPlanes;
    static_assert(kOwnRowPlanes % 8 == 0, "row batches");
#pragma unroll 1
    for (int i0 = 0; i0 < kOwnRowPlanes; i0 += 8) {
        uint32_t e[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = warp + (i0 + k) / C::kPlanes * C::kWarps;
            const uint8_t* row = smem + j * kRowBytes + (i0 + k) % C::kPlanes * 128;
            e[k] = *reinterpret_cast<const uint32_t*>(row + ((lane + j) & 31) * 4);
        }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = warp + (i0 + k) / C::kPlanes * C::kWarps;
            uint8_t* row = smem + j * kRowBytes + (i0 + k) % C::kPlanes * 128;
            *reinterpret_cast<uint32_t*>(row + lane * 4) = e[k];
        }
    }
    __syncthreads();

    // ---------------------------------------------------------------- main loop over the chunk
    constexpr int kBatch = (C::kSlots * C::kLaneHeads >= 8) ? 2 : 4;       // tokens whose lookups are in flight together

    // Weight units.  Each query head's bins count in units of 2^e_cur[h].  A warp adds its tokens'
    // weights without waiting for the others as long as (a) its largest score fits the unit
    // (weight <= 2^kMaxWeightBits) and (b) its reservation keeps the head's running total - a bound
    // on every bin - below 2^32.  Otherwise it raises `want`; every warp joins the coarsening
    // event at its next check (or at the end of its loop): barrier, bins shifted right, new unit,
    // barrier.  No warp is inside its V side during an event, so bins and unit stay consistent.
    auto coarsen = [&]() {                       // entered by every thread, right after the event's first barrier
        int shift[R], e_next[R];
        unsigned int t_next[R];
        bool any_shift = false;
#pragma unroll
        for (int h = 0; h < R; ++h) {
            const int e = ctl->e_cur[h], cmr = ctl->req_ref[h], need = ctl->req_need[h];
            const unsigned int tot = ctl->total[h];
            int e_new = e;
            shift[h] = 0;
            t_next[h] = tot;
            if (cmr != kUnset) {
                // range: the largest score must fit; room: one round of every warp takes at most half of 2^32
                if (e == kUnset || cmr - e > kMaxWeightBits) e_new = cmr - kUnitBits;
                const int room = need + C::kLog2Groups - 31;
                if (need != kUnset && room > e_new) e_new = room;
            }
            if (e != kUnset) {
                // the weights already in the bins keep a sixteenth of the range at most after an event
                for (int tries = 0; tries < 24; ++tries) {              // 2 bits per try: bounded
                    const int k = e_new - e;
                    if ((k >= 32 ? 0u : tot >> k) < kBinLimit256 / 16u) break;
                    e_new += 2;
                }
                shift[h] = e_new - e;
                t_next[h] = (shift[h] >= 32 ? 0u : tot >> shift[h]) + 1u;
                any_shift = any_shift || shift[h] > 0;
            }
            e_next[h] = e_new;
        }
        if (any_shift) {
            for (int i = threadIdx.x; i < kRows * 32 * C::kPlanes; i += C::kThreads) {
                const int word = i % (32 * C::kPlanes);
                const int hw = C::head_of_word(word);
                int k = shift[0];
#pragma unroll
                for (int h = 1; h < R; ++h) k = hw == h ? shift[h] : k;
                if (k > 0) {
                    uint32_t* bp = reinterpret_cast<uint32_t*>(smem + C::kVOffset + (i / (32 * C::kPlanes)) * kRowBytes + word * 4);
                    const uint32_t v = *bp;
                    *bp = k >= 32 ? 0u : (v >> k) + ((v >> (k - 1)) & 1u);
                }
            }
        }
        event_barrier(C::kThreads);                         // every thread has read the request and rescaled its bins
        if (threadIdx.x == 0) {
#pragma unroll
            for (int h = 0; h < R; ++h) {
                ctl->e_cur[h] = e_next[h];
                ctl->total[h] = t_next[h];
                ctl->req_ref[h] = kUnset;
                ctl->req_need[h] = kUnset;
            }
            ctl->want = 0;
        }
        event_barrier(C::kThreads);                         // the new state is visible
    };
    constexpr bool kSplit = C::kHalfRows && R >= 2;      // the two half warps serve different query heads
    const unsigned grp_mask = kSplit ? (lane < 16 ? 0x0000ffffu : 0xffff0000u) : 0xffffffffu;
    const bool grp_leader = kSplit ? (lane & 15) == 0 : lane == 0;
    load_words(kw, kbase, blk0 + (int64_t)warp * C::kBlocksPerIter + qb);

    for (int it = 0; it < n_iters; ++it) {
        const int64_t blk_warp = blk0 + ((int64_t)it * C::kWarps + warp) * C::kBlocksPerIter;
        const int64_t blk = blk_warp + qb;
        load_words(vw, vbase, blk);

        // K side: scores of this quad's 16 tokens for the query heads this lane serves.
        float sc[C::kLaneHeads][16];
#pragma unroll
        for (int k0 = 0; k0 < 16; k0 += kBatch) {
            // All lookups of a batch of tokens are issued before the first MMA needs one.  The row
            // index of a code is formed once and serves every head (the planes are 128 bytes apart).
            uint32_t a[kBatch][C::kLaneHeads][C::kSlots];
#pragma unroll
            for (int kk = 0; kk < kBatch; ++kk)
#pragma unroll
                for (int m = 0; m < C::kSlots; ++m) {
                    const uint32_t idx = row_index(kw[m], k0 + kk, lane_off[m]);
#pragma unroll
                    for (int u = 0; u < C::kLaneHeads; ++u)
                        a[kk][u][m] = *reinterpret_cast<const volatile uint32_t*>(smem + u * 128 + idx);
                }
            // two tokens per MMA chain: fragment rows r and r + 8; two code words per MMA
#pragma unroll
            for (int kk = 0; kk < kBatch; kk += 2)
#pragma unroll
                for (int u = 0; u < C::kLaneHeads; ++u) {
                    float d[4];
                    mma_rowsum_first(d, a[kk][u][0], a[kk + 1][u][0], a[kk][u][1], a[kk + 1][u][1]);
#pragma unroll
                    for (int m = 2; m < C::kSlots; m += 2)
                        mma_rowsum_acc(d, a[kk][u][m], a[kk + 1][u][m], a[kk][u][m + 1], a[kk + 1][u][m + 1]);
                    sc[u][k0 + kk] = d[0];
                    sc[u][k0 + kk + 1] = d[2];
                }
        }

        if (C::kHalfGroups) {            // the other half warp summed the other 32 groups of the same tokens
#pragma unroll
            for (int k = 0; k < 16; ++k) sc[0][k] += __shfl_xor_sync(0xffffffffu, sc[0][k], 16);
        }
        // tokens past the end of the context get -inf (only the warp that holds the ragged end pays)
        if ((blk_warp + C::kBlocksPerIter) * kTokenBlock > t_end) {
            const int64_t tok0 = blk * kTokenBlock;
#pragma unroll
            for (int k = 0; k < 16; ++k)
#pragma unroll
                for (int u = 0; u < C::kLaneHeads; ++u)
                    if (tok0 + k >= t_end) sc[u][k] = -INFINITY;
        }
        // Per head: reference exponent ref = ceil(largest score of this (half) warp).  The four lanes
        // of a quad hold the same 16 scores; lane p turns tokens p, p+4, p+8, p+12 into weights
        // 2^(score - ref) <= 1 (exponentials are the scarce resource here), and the integer weights
        // are handed round the quad by shuffles just before the bins are updated.
        int ref[C::kLaneHeads];
        float wown[C::kLaneHeads][4], zsum[C::kLaneHeads];
        bool any_tokens = false;
#pragma unroll
        for (int u = 0; u < C::kLaneHeads; ++u) {
            float mx = -INFINITY;
#pragma unroll
            for (int k = 0; k < 16; ++k) mx = fmaxf(mx, sc[u][k]);
            const float gm = dec_float(__reduce_max_sync(grp_mask, enc_float(mx * lut_scale)));
            const bool any = gm > -INFINITY;
            any_tokens = any_tokens || any;
            ref[u] = any ? (int)fminf(fmaxf(ceilf(gm), -1.0e9f), 1.0e9f) : kUnset;
            const float fref = any ? (float)ref[u] : 0.f;
            float z = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float s01 = (p & 1) ? sc[u][4 * j + 1] : sc[u][4 * j];
                const float s23 = (p & 1) ? sc[u][4 * j + 3] : sc[u][4 * j + 2];
                const float own = (p & 2) ? s23 : s01;                    // score of token 4 j + p
                wown[u][j] = ex2(fmaf(own, lut_scale, -fref));
                z += wown[u][j];
            }
#pragma unroll
            // (with 64 groups both half warps hold the same tokens: each counts them once)
            for (int o = (kSplit || C::kHalfGroups) ? 8 : 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            zsum[u] = z;
        }
        any_tokens = __any_sync(0xffffffffu, any_tokens);

        // Reserve room for this warp's weights, or ask for a coarser unit.  Bounded: every event
        // coarsens the refused head by at least two bits.
        int eu[C::kLaneHeads];
        for (int attempt = 0; attempt < 64; ++attempt) {
            if (*reinterpret_cast<volatile int*>(&ctl->want) != 0) {
                // someone needs a coarser unit: tell the event what this warp will need, then join it
                if (grp_leader)
#pragma unroll
                    for (int u = 0; u < C::kLaneHeads; ++u)
                        if (ref[u] != kUnset) {
                            atomicMax(&ctl->req_ref[C::lane_head(u, r)], ref[u]);
                            atomicMax(&ctl->req_need[C::lane_head(u, r)], ref[u] + ilogbf(fmaxf(zsum[u], 1e-30f)) + 1);
                        }
                event_barrier(C::kThreads);
                coarsen();
                continue;
            }
            if (!any_tokens) break;
            bool ok = true;
            unsigned int mine[C::kLaneHeads];
#pragma unroll
            for (int u = 0; u < C::kLaneHeads; ++u) {
                const int h = C::lane_head(u, r);
                eu[u] = *reinterpret_cast<volatile int*>(&ctl->e_cur[h]);
                mine[u] = 0u;
                if (ref[u] == kUnset) continue;
                if (eu[u] == kUnset || ref[u] - eu[u] > kMaxWeightBits) { ok = false; continue; }
                // this (half) warp's weights in the current unit, rounded up, in units of 256
                const float cw = (zsum[u] * pow2i(ref[u] - eu[u]) * 1.00002f + (float)(16 * C::kBlocksPerIter)) * (1.f / 256.f) + 1.f;
                const unsigned int ci = (unsigned int)fminf(cw, 6.7e7f);
                unsigned int old = 0u;
                if (grp_leader) old = atomicAdd(&ctl->total[h], ci);
                // (group mask: with two heads per warp the other half warp may have left this iteration)
                old = __shfl_sync(grp_mask, old, kSplit ? (lane & 16) : 0);
                mine[u] = ci;
                if (old + ci >= kBinLimit256) ok = false;
            }
            ok = __all_sync(0xffffffffu, ok);
            if (ok) break;
            // give the reservations back, publish what is needed, raise the request, join the event
            if (grp_leader) {
#pragma unroll
                for (int u = 0; u < C::kLaneHeads; ++u) {
                    const int h = C::lane_head(u, r);
                    if (mine[u]) atomicSub(&ctl->total[h], mine[u]);
                    if (ref[u] != kUnset) {
                        atomicMax(&ctl->req_ref[h], ref[u]);
                        atomicMax(&ctl->req_need[h], ref[u] + ilogbf(fmaxf(zsum[u], 1e-30f)) + 1);
                    }
                }
                atomicExch(&ctl->want, 1);
            }
            event_barrier(C::kThreads);
            coarsen();
        }

        // the next iteration's K words travel while the V side runs
        load_words(kw, kbase, blk + (int64_t)C::kWarps * C::kBlocksPerIter);

        if (!any_tokens) continue;

        // V side: integer weights (own tokens), handed round the quad, into the bins of this lane's groups
        uint32_t wint[C::kLaneHeads][4];
#pragma unroll
        for (int u = 0; u < C::kLaneHeads; ++u) {
            const float f = ref[u] == kUnset ? 0.f : pow2i(ref[u] - eu[u]);      // power of two <= 2^kMaxWeightBits
#pragma unroll
            for (int j = 0; j < 4; ++j) wint[u][j] = __float2uint_rn(wown[u][j] * f);
        }
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            uint32_t wk[C::kLaneHeads];
#pragma unroll
            for (int u = 0; u < C::kLaneHeads; ++u) wk[u] = __shfl_sync(0xffffffffu, wint[u][k >> 2], (lane & ~3) | (k & 3));
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m) {
                const uint32_t idx = row_index(vw[m], k, lane_off[m]);
#pragma unroll
                for (int u = 0; u < C::kLaneHeads; ++u)
                    atomicAdd(reinterpret_cast<unsigned int*>(smem + C::kVOffset + u * 128 + idx), wk[u]);
            }
        }
    }
    // Warps that are done keep joining coarsening events until every warp is done.
    load_unit(cva, vcb, 0);                       // the first V centroids travel meanwhile
    for (int guard = 0; guard < 4096; ++guard) {
        event_barrier(C::kThreads);
        if (*reinterpret_cast<volatile int*>(&ctl->want) == 0) break;
        coarsen();
    }
    __syncthreads();

    // ---------------------------------------------------------------- epilogue: bins x V centroids
    // Same ownership as the table build: a warp owns whole groups, lanes walk the code values.
    // Rows are first rotated by their index so that a column read is bank-conflict free.
#pragma unroll 1
    for (int i0 = 0; i0 < kOwnRowPlanes; i0 += 8) {
        uint32_t v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = warp + (i0 + k) / C::kPlanes * C::kWarps;
            const uint8_t* row = smem + C::kVOffset + j * kRowBytes + (i0 + k) % C::kPlanes * 128;
            v[k] = *reinterpret_cast<const uint32_t*>(row + lane * 4);
        }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = warp + (i0 + k) / C::kPlanes * C::kWarps;
            uint8_t* row = smem + C::kVOffset + j * kRowBytes + (i0 + k) % C::kPlanes * 128;
            *reinterpret_cast<uint32_t*>(row + ((lane + j) & 31) * 4) = v[k];
        }
    }
    __syncthreads();
    float acc[R][kC];
    float lsum[R];                            // sum of the bins of group 0 (the normaliser)
#pragma unroll
    for (int h = 0; h < R; ++h) lsum[h] = 0.f;
    auto use_unit = [&](const float (&cv)[kJb][kC], int u) {
        const int gi = u / kUnitsPerGroup, g = warp * C::kGroupsPerWarp + gi;
        if (u % kUnitsPerGroup == 0) {
#pragma unroll
            for (int h = 0; h < R; ++h)
#pragma unroll
                for (int i = 0; i < kC; ++i) acc[h][i] = 0.f;
        }
#pragma unroll
        for (int jb = 0; jb < kJb; ++jb) {
            const int j = ((u % kUnitsPerGroup) * kJb + jb) * 32 + lane;
#pragma unroll
            for (int h = 0; h < R; ++h) {
                const uint8_t* row = smem + C::kVOffset + j * kRowBytes + C::plane_of(g, h) * 128;
                uint32_t bi = *reinterpret_cast<const uint32_t*>(row + ((C::word_of(g, h) + j) & 31) * 4);
                if (C::kReplica) bi += *reinterpret_cast<const uint32_t*>(row + ((16 + g + j) & 31) * 4);
                const float bv = (float)bi;
                if (gi == 0) lsum[h] += bv;
#pragma unroll
                for (int i = 0; i < kC; ++i) acc[h][i] = fmaf(bv, cv[jb][i], acc[h][i]);
            }
        }
        if (u % kUnitsPerGroup != kUnitsPerGroup - 1) return;
        // Sum over the 32 lanes.  The kC channel sums are folded while they are exchanged: after
        // the steps with lane masks 16, 8 (and 4 for kC = 8) a lane holds one channel, the
        // remaining steps finish that channel.
#pragma unroll
        for (int h = 0; h < R; ++h) {
            if constexpr (kC == 2) {
                // one exchange gives each half warp one of the two channels, four more steps finish it
                const bool up = (lane & 16) != 0;
                float v = (up ? acc[h][1] : acc[h][0]) + __shfl_xor_sync(0xffffffffu, up ? acc[h][0] : acc[h][1], 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if ((lane & 15) == 0) part_base[(int64_t)h * n_parts * stride + 2 + g * kC + (up ? 1 : 0)] = v;
            } else {
                float v = fold_channels<kC>(acc[h], lane);
                // lane holds channel fold_channel_of<kC>(lane) summed over the lanes that share it
                const int ch = fold_channel_of<kC>(lane);
                if ((lane & (kC == 8 ? 3 : 7)) == 0) part_base[(int64_t)h * n_parts * stride + 2 + g * kC + ch] = v;
            }
        }
        if (g == 0) {
#pragma unroll
            for (int h = 0; h < R; ++h) {
                float l = lsum[h];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                if (lane == 0) {
                    part_base[(int64_t)h * n_parts * stride + 0] = (float)ctl->e_cur[h];   // reference exponent (log2 domain)
                    part_base[(int64_t)h * n_parts * stride + 1] = l;            // normaliser, in the same unit
                }
            }
        }
    };
#pragma unroll 1
    for (int u = 0; u < kUnits; u += 2) {
        load_unit(cvb, vcb, u + 1);
        use_unit(cva, u);
        if (u + 2 < kUnits) load_unit(cva, vcb, u + 2);
        use_unit(cvb, u + 1);
    }
    if (out) {
        __syncthreads();
        for (int i = threadIdx.x; i < R * 128; i += C::kThreads) {
            const int h = i >> 7, d = i & 127;
            const float* ph = part_base + (int64_t)h * n_parts * stride;
            const float l = ph[1];
            out[(s * sh.n_q_heads + (int64_t)head_group * R + h) * 128 + d] = l > 0.f ? ph[2 + d] / l : 0.f;
        }
    }
}


// ---------------------------------------------------------------------------------------------
// CQ-8c10b (Section 4 of the paper: groups of 8 channels, 1024 centroids per group, 1.25 bytes per
// code).  The formulation and the weight-unit protocol are those of decode_tuned_kernel; what
// changes is the size of the tables.  One CTA of 16 warps serves one QUERY head (query heads that
// share a KV head read the same codes again, from L2):
//   K table: row j (128 bytes) holds the 16 groups' entries of code value j twice, words g and
//            16 + g, so that the two half warps of a lookup use different banks (128 KiB);
//   V bins:  row j (64 bytes) holds the 16 groups' bins of code value j (64 KiB): bins of even and
//            odd code values fall into different halves of the banks, so a bin update of a warp
//            takes two wavefronts when two of its lanes meet, one otherwise.
// Code words: the low bytes of a (block, group) are one 16-byte word as for b = 8; the upper two
// bits of its 16 tokens are one 32-bit word, 256 bytes into the block.
// ---------------------------------------------------------------------------------------------
struct WideCfg {
    static constexpr int kC = 8, kG = 16, kRows = 1024;
    static constexpr int kWarps = 16, kThreads = kWarps * 32;
    static constexpr int kSlots = 4, kBlocksPerIter = 8;
    static constexpr int kRoundTokens = kWarps * kBlocksPerIter * 16;
    static constexpr int kKRowBytes = 128, kVRowBytes = 64;
    static constexpr int kVOffset = kRows * kKRowBytes;
    static constexpr int kTableBytes = kVOffset + kRows * kVRowBytes;
    static constexpr int kSmemBytes = kTableBytes + 128 + 128 * 4;      // tables, control block, scaled query
    static constexpr int kBlockBytes = kG * (16 + 4);
    static constexpr int kLog2Groups = 4;
    __device__ static __forceinline__ int word(int r, int p, int m) { return 16 * (r >> 2) + 4 * ((r + m) & 3) + p; }
};

__device__ __forceinline__ uint32_t ldg_u32(const uint8_t* p)
{
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// table byte offset (code << row_shift) + lane_off for token k of a code word: low byte from `w`,
// upper two bits from `hw`
__device__ __forceinline__ uint32_t wide_index(const uint4& w, uint32_t hw, int k, uint32_t lane_off, int row_shift)
{
    const uint32_t low = __byte_perm(word32(w, k), 0u, 0x4440u | (uint32_t)(k & 3));
    const uint32_t hi = (hw >> (2 * k)) & 3u;
    return (low << row_shift) + (hi << (row_shift + 8)) + lane_off;
}

__global__ void __launch_bounds__(WideCfg::kThreads, 1)
decode_wide_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                   const float* __restrict__ kcb, const float* __restrict__ vcb,
                   const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int chunk_tokens, int n_parts,
                   int tail_first, int cb_aligned32, float* __restrict__ partials)
{
    using C = WideCfg;
    constexpr int kC = C::kC;
    extern __shared__ __align__(1024) uint8_t smem[];
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + C::kTableBytes);
    float* qs = reinterpret_cast<float*>(smem + C::kTableBytes + 128);     // [128], scaled by scale*log2(e)

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, p = lane & 3;

    // work item: (context part, sequence, query head), with the same tail rule as decode_tuned_kernel
    const int n_items = (int)(sh.n_q_heads * sh.n_seq);
    int item = blockIdx.x % n_items;
    int part = (int)(blockIdx.x / n_items);
    bool whole = false;
    if (tail_first >= 0) {
        whole = (int)blockIdx.x < tail_first;
        item = whole ? blockIdx.x : tail_first + (blockIdx.x - tail_first) / n_parts;
        part = whole ? 0 : (blockIdx.x - tail_first) % n_parts;
    }
    const int hq = item % sh.n_q_heads;
    const int64_t s = seq_by_rank(seq_lens, (int)sh.n_seq, sh.max_tokens, item / sh.n_q_heads);
    const int hkv = hq / sh.R;

    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int64_t t_begin = (int64_t)part * chunk_tokens;
    const int64_t t_end = (whole || t_begin + chunk_tokens >= n) ? n : t_begin + chunk_tokens;
    const int stride = partial_stride(128);
    float* part_base = partials + ((s * sh.n_q_heads + hq) * n_parts + part) * stride;
    if (whole)
        for (int i = threadIdx.x; i < (n_parts - 1) * stride; i += C::kThreads)
            part_base[stride + i] = i % stride == 0 ? -INFINITY : 0.f;
    if (t_begin >= t_end) {
        for (int i = threadIdx.x; i < stride; i += C::kThreads) part_base[i] = i == 0 ? -INFINITY : 0.f;
        return;
    }

    // ---------------------------------------------------------------- addresses; the first centroids travel during the set-up
    const int64_t blk0 = t_begin / kTokenBlock;
    const int64_t blk_lim = (t_end + kTokenBlock - 1) / kTokenBlock;
    const int n_iters = (int)((t_end - t_begin + C::kRoundTokens - 1) / C::kRoundTokens);
    uint32_t lane_off[C::kSlots];      // byte offset of this lane's word inside a K row, per code word
#pragma unroll
    for (int m = 0; m < C::kSlots; ++m) lane_off[m] = 4u * C::word(r, p, m);
    const uint8_t* kbase = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint8_t* vbase = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);

    uint4 kw[C::kSlots], vw[C::kSlots];
    uint32_t kh[C::kSlots], vh[C::kSlots];
    auto load_words = [&](uint4 (&dst)[C::kSlots], uint32_t (&dsth)[C::kSlots], const uint8_t* base, int64_t blk) {
        if (blk < blk_lim) {
            const uint8_t* bp = base + blk * C::kBlockBytes;
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m) {
                const int gm = (lane_off[m] >> 2) & 15;
                dst[m] = ldg_codes(reinterpret_cast<const uint4*>(bp + gm * kTokenBlock));
                dsth[m] = ldg_u32(bp + C::kG * kTokenBlock + gm * 4);
            }
        } else {
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m) {
                dst[m] = make_uint4(0u, 0u, 0u, 0u);
                dsth[m] = 0u;
            }
        }
    };

    // Codebooks: warp g owns group g; its lanes walk the code values in units of 4 x 32 centroids
    // (32 registers per lane), the next unit loaded while the current one is used.
    constexpr int kJb = 4;
    constexpr int kUnits = C::kRows / 32 / kJb;
    const int g = warp;
    auto load_unit = [&](float (&cv)[kJb][kC], const float* cb, int u) {
        const float* cg = cb + (((int64_t)hkv * C::kG + g) * C::kRows + u * kJb * 32 + lane) * kC;
#pragma unroll
        for (int jb = 0; jb < kJb; ++jb) load_centroid<kC>(cg + jb * 32 * kC, cv[jb], cb_aligned32 != 0);
    };
    float cva[kJb][kC], cvb[kJb][kC];
    load_unit(cva, kcb, 0);

    // ---------------------------------------------------------------- set-up: query, LUT, bins
    if (threadIdx.x < 4) {
        ctl->e_cur[threadIdx.x] = kUnset;
        ctl->total[threadIdx.x] = 0u;
        ctl->req_ref[threadIdx.x] = kUnset;
        ctl->req_need[threadIdx.x] = kUnset;
    }
    if (threadIdx.x == 4) { ctl->want = 0; ctl->lut_absmax = 0.f; }
    if (threadIdx.x < 128)
        qs[threadIdx.x] = __half2float(q[(s * sh.n_q_heads + hq) * 128 + threadIdx.x]) * scale_log2e;
    for (int i = threadIdx.x; i < C::kRows * C::kVRowBytes / 16; i += C::kThreads)
        *reinterpret_cast<uint4*>(smem + C::kVOffset + i * 16) = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();

    // K table: row j is written rotated by j words (a column would fall into one bank), both copies,
    // then every row is un-rotated.  Entries are half2 (hi, lo) of LUT * 2^-kexp as in decode_tuned_kernel.
    float lut_scale = 1.f;
    for (int attempt = 0; attempt < 2; ++attempt) {
        const float inv = 1.f / lut_scale;
        float absmax = 0.f;
        float qreg[kC];
#pragma unroll
        for (int i = 0; i < kC; ++i) qreg[i] = qs[g * kC + i] * inv;
        auto build_unit = [&](const float (&cv)[kJb][kC], int u) {
#pragma unroll
            for (int jb = 0; jb < kJb; ++jb) {
                const int j = (u * kJb + jb) * 32 + lane;
                float dot = 0.f;
#pragma unroll
                for (int i = 0; i < kC; ++i) dot = fmaf(qreg[i], cv[jb][i], dot);
                absmax = fmaxf(absmax, fabsf(dot));
                const uint32_t e = pack_hi_lo(dot);
                uint8_t* row = smem + j * C::kKRowBytes;
                *reinterpret_cast<uint32_t*>(row + ((g + j) & 31) * 4) = e;
                *reinterpret_cast<uint32_t*>(row + ((16 + g + j) & 31) * 4) = e;
            }
        };
        if (attempt == 1) load_unit(cva, kcb, 0);
#pragma unroll 1
        for (int u = 0; u < kUnits; u += 2) {
            load_unit(cvb, kcb, u + 1);
            build_unit(cva, u);
            if (u + 2 < kUnits) load_unit(cva, kcb, u + 2);
            build_unit(cvb, u + 1);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) absmax = fmaxf(absmax, __shfl_xor_sync(0xffffffffu, absmax, o));
        if (lane == 0) atomicMax(reinterpret_cast<int*>(&ctl->lut_absmax), __float_as_int(absmax));
        __syncthreads();
        const float amax = ctl->lut_absmax;
        if (attempt == 1 || amax < 32768.f) break;       // same decision in every thread
        int ex;
        frexpf(amax, &ex);
        lut_scale = exp2f((float)(ex - 15));
        __syncthreads();
        if (threadIdx.x == 0) ctl->lut_absmax = 0.f;
        __syncthreads();
    }
#pragma unroll 1
    for (int i0 = 0; i0 < C::kRows / C::kWarps; i0 += 8) {
        uint32_t e[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = warp + (i0 + k) * C::kWarps;
            e[k] = *reinterpret_cast<const uint32_t*>(smem + j * C::kKRowBytes + ((lane + j) & 31) * 4);
        }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int j = warp + (i0 + k) * C::kWarps;
            *reinterpret_cast<uint32_t*>(smem + j * C::kKRowBytes + lane * 4) = e[k];
        }
    }
    __syncthreads();

    // ---------------------------------------------------------------- main loop over the chunk
    constexpr int kBatch = 4;
    auto coarsen = [&]() {                       // entered by every thread, right after the event's first barrier
        const int e = ctl->e_cur[0], cmr = ctl->req_ref[0], need = ctl->req_need[0];
        const unsigned int tot = ctl->total[0];
        int e_new = e, shift = 0;
        unsigned int t_next = tot;
        if (cmr != kUnset) {
            if (e == kUnset || cmr - e > kMaxWeightBits) e_new = cmr - kUnitBits;
            const int room = need + C::kLog2Groups - 31;
            if (need != kUnset && room > e_new) e_new = room;
        }
        if (e != kUnset) {
            for (int tries = 0; tries < 24; ++tries) {              // 2 bits per try: bounded
                const int k = e_new - e;
                if ((k >= 32 ? 0u : tot >> k) < kBinLimit256 / 16u) break;
                e_new += 2;
            }
            shift = e_new - e;
            t_next = (shift >= 32 ? 0u : tot >> shift) + 1u;
        }
        if (shift > 0) {
            for (int i = threadIdx.x; i < C::kRows * C::kVRowBytes / 4; i += C::kThreads) {
                uint32_t* bp = reinterpret_cast<uint32_t*>(smem + C::kVOffset) + i;
                const uint32_t v = *bp;
                *bp = shift >= 32 ? 0u : (v >> shift) + ((v >> (shift - 1)) & 1u);
            }
        }
        event_barrier(C::kThreads);                         // every thread has read the request and rescaled its bins
        if (threadIdx.x == 0) {
            ctl->e_cur[0] = e_new;
            ctl->total[0] = t_next;
            ctl->req_ref[0] = kUnset;
            ctl->req_need[0] = kUnset;
            ctl->want = 0;
        }
        event_barrier(C::kThreads);                         // the new state is visible
    };
    load_words(kw, kh, kbase, blk0 + (int64_t)warp * C::kBlocksPerIter + r);

    for (int it = 0; it < n_iters; ++it) {
        const int64_t blk_warp = blk0 + ((int64_t)it * C::kWarps + warp) * C::kBlocksPerIter;
        const int64_t blk = blk_warp + r;
        load_words(vw, vh, vbase, blk);

        // K side: scores of this quad's 16 tokens
        float sc[16];
#pragma unroll
        for (int k0 = 0; k0 < 16; k0 += kBatch) {
            uint32_t a[kBatch][C::kSlots];
#pragma unroll
            for (int kk = 0; kk < kBatch; ++kk)
#pragma unroll
                for (int m = 0; m < C::kSlots; ++m)
                    a[kk][m] = *reinterpret_cast<const volatile uint32_t*>(smem + wide_index(kw[m], kh[m], k0 + kk, lane_off[m], 7));
#pragma unroll
            for (int kk = 0; kk < kBatch; kk += 2) {
                float d[4];
                mma_rowsum_first(d, a[kk][0], a[kk + 1][0], a[kk][1], a[kk + 1][1]);
                mma_rowsum_acc(d, a[kk][2], a[kk + 1][2], a[kk][3], a[kk + 1][3]);
                sc[k0 + kk] = d[0];
                sc[k0 + kk + 1] = d[2];
            }
        }
        if ((blk_warp + C::kBlocksPerIter) * kTokenBlock > t_end) {
            const int64_t tok0 = blk * kTokenBlock;
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if (tok0 + k >= t_end) sc[k] = -INFINITY;
        }
        // reference exponent of the warp, weights of this lane's own four tokens (see decode_tuned_kernel)
        float mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < 16; ++k) mx = fmaxf(mx, sc[k]);
        const float gm = dec_float(__reduce_max_sync(0xffffffffu, enc_float(mx * lut_scale)));
        const bool any_tokens = gm > -INFINITY;
        const int ref = any_tokens ? (int)fminf(fmaxf(ceilf(gm), -1.0e9f), 1.0e9f) : kUnset;
        const float fref = any_tokens ? (float)ref : 0.f;
        float wown[4], zsum = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float s01 = (p & 1) ? sc[4 * j + 1] : sc[4 * j];
            const float s23 = (p & 1) ? sc[4 * j + 3] : sc[4 * j + 2];
            const float own = (p & 2) ? s23 : s01;
            wown[j] = ex2(fmaf(own, lut_scale, -fref));
            zsum += wown[j];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zsum += __shfl_xor_sync(0xffffffffu, zsum, o);

        // reserve room for this warp's weights, or ask for a coarser unit (bounded: see decode_tuned_kernel)
        int eu = kUnset;
        for (int attempt = 0; attempt < 64; ++attempt) {
            if (*reinterpret_cast<volatile int*>(&ctl->want) != 0) {
                if (lane == 0 && ref != kUnset) {
                    atomicMax(&ctl->req_ref[0], ref);
                    atomicMax(&ctl->req_need[0], ref + ilogbf(fmaxf(zsum, 1e-30f)) + 1);
                }
                event_barrier(C::kThreads);
                coarsen();
                continue;
            }
            if (!any_tokens) break;
            bool ok = true;
            unsigned int mine = 0u;
            eu = *reinterpret_cast<volatile int*>(&ctl->e_cur[0]);
            if (eu == kUnset || ref - eu > kMaxWeightBits) {
                ok = false;
            } else {
                const float cw = (zsum * pow2i(ref - eu) * 1.00002f + (float)(16 * C::kBlocksPerIter)) * (1.f / 256.f) + 1.f;
                const unsigned int ci = (unsigned int)fminf(cw, 6.7e7f);
                unsigned int old = 0u;
                if (lane == 0) old = atomicAdd(&ctl->total[0], ci);
                old = __shfl_sync(0xffffffffu, old, 0);
                mine = ci;
                if (old + ci >= kBinLimit256) ok = false;
            }
            if (ok) break;
            if (lane == 0) {
                if (mine) atomicSub(&ctl->total[0], mine);
                atomicMax(&ctl->req_ref[0], ref);
                atomicMax(&ctl->req_need[0], ref + ilogbf(fmaxf(zsum, 1e-30f)) + 1);
                atomicExch(&ctl->want, 1);
            }
            event_barrier(C::kThreads);
            coarsen();
        }

        load_words(kw, kh, kbase, blk + (int64_t)C::kWarps * C::kBlocksPerIter);
        if (!any_tokens) continue;

        // V side: integer weights, handed round the quad, into the bins of this lane's groups
        uint32_t wint[4];
        {
            const float f = pow2i(ref - eu);
#pragma unroll
            for (int j = 0; j < 4; ++j) wint[j] = __float2uint_rn(wown[j] * f);
        }
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const uint32_t wk = __shfl_sync(0xffffffffu, wint[k >> 2], (lane & ~3) | (k & 3));
#pragma unroll
            for (int m = 0; m < C::kSlots; ++m)
                atomicAdd(reinterpret_cast<unsigned int*>(smem + C::kVOffset + wide_index(vw[m], vh[m], k, lane_off[m] & 63u, 6)), wk);
        }
    }
    load_unit(cva, vcb, 0);                       // the first V centroids travel meanwhile
    for (int guard = 0; guard < 4096; ++guard) {
        event_barrier(C::kThreads);
        if (*reinterpret_cast<volatile int*>(&ctl->want) == 0) break;
        coarsen();
    }
    __syncthreads();

    // ---------------------------------------------------------------- epilogue: bins x V centroids
    // The bins are 512 rows of 32 words (two code values per row); each is rotated by its index so
    // that the column read of a warp (its group, 32 consecutive code values) is conflict-free.
#pragma unroll 1
    for (int i0 = 0; i0 < C::kRows / 2 / C::kWarps; i0 += 8) {
        uint32_t v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int rho = warp + (i0 + k) * C::kWarps;
            v[k] = *reinterpret_cast<const uint32_t*>(smem + C::kVOffset + rho * 128 + lane * 4);
        }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int rho = warp + (i0 + k) * C::kWarps;
            *reinterpret_cast<uint32_t*>(smem + C::kVOffset + rho * 128 + ((lane + rho) & 31) * 4) = v[k];
        }
    }
    __syncthreads();
    float acc[kC];
#pragma unroll
    for (int i = 0; i < kC; ++i) acc[i] = 0.f;
    float lsum = 0.f;
#pragma unroll 1
    for (int u = 0; u < kUnits; u += 2) {
        load_unit(cvb, vcb, u + 1);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            if (half == 1 && u + 2 < kUnits) load_unit(cva, vcb, u + 2);
#pragma unroll
            for (int jb = 0; jb < kJb; ++jb) {
                const int j = ((u + half) * kJb + jb) * 32 + lane;
                const int rho = j >> 1;
                const uint32_t bi = *reinterpret_cast<const uint32_t*>(smem + C::kVOffset + rho * 128 + ((16 * (j & 1) + g + rho) & 31) * 4);
                const float bv = (float)bi;
                lsum += bv;
#pragma unroll
                for (int i = 0; i < kC; ++i) acc[i] = fmaf(bv, half == 0 ? cva[jb][i] : cvb[jb][i], acc[i]);
            }
        }
    }
    {
        const float v = fold_channels<kC>(acc, lane);
        const int ch = fold_channel_of<kC>(lane);
        if ((lane & 3) == 0) part_base[2 + g * kC + ch] = v;
    }
    if (g == 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
        if (lane == 0) {
            part_base[0] = (float)ctl->e_cur[0];      // reference exponent (log2 domain)
            part_base[1] = lsum;                      // normaliser, in the same unit
        }
    }
}

int aligned32(const float* a, const float* b)
{
    return ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) & 31u) == 0 ? 1 : 0;
}

// Launch plan of one call: context chunk per CTA, partial slots per (sequence, query head), and
// the first item of the tail (-1: none).
struct Plan {
    int chunk;
    int n_parts;
    int tail_first;
    unsigned grid;
};

// The table build and the bins x centroids product are paid once per CTA, so chunks are long (up
// to 65536 tokens); they are halved only while the grid would not give the CTA slots of the
// SMs one and a half CTAs each, and never below 2048 tokens.  When every context fits one chunk
// and the last wave of CTAs would fill at most half of the slots, the items of that wave are
// spread over 2 to 4 CTAs each instead, which shortens the wave by that factor.  This applies
// where one CTA fills an SM; with two CTAs per SM a CTA whose neighbour has finished already runs
// faster, and the split was measured to gain nothing.
Plan plan_from(const Shape& sh, int64_t round, int min_blocks, int64_t items)
{
    Plan pl;
    const int64_t slots = (int64_t)device_sm_count() * min_blocks;
    int64_t chunk = (sh.max_tokens + round - 1) / round * round;
    if (chunk > 65536) chunk = 65536;
    while (chunk > 2048 && 2 * items * ((sh.max_tokens + chunk - 1) / chunk) < 3 * slots)
        chunk = (chunk / 2 + round - 1) / round * round;
    pl.chunk = (int)chunk;
    pl.n_parts = (int)((sh.max_tokens + chunk - 1) / chunk);
    pl.tail_first = -1;
    pl.grid = (unsigned)(items * pl.n_parts);
    const int64_t rest = items % slots;               // CTAs of the last wave
    if (min_blocks == 1 && pl.n_parts == 1 && items > slots && rest > 0 && 2 * rest <= slots && chunk >= 2 * 2048) {
        int64_t k = slots / rest;
        if (k > 4) k = 4;
        const int64_t part_chunk = ((chunk + k - 1) / k + round - 1) / round * round;
        pl.chunk = (int)part_chunk;
        pl.n_parts = (int)((sh.max_tokens + part_chunk - 1) / part_chunk);
        pl.tail_first = (int)(items - rest);
        pl.grid = (unsigned)(pl.tail_first + rest * pl.n_parts);
    }
    return pl;
}

template <int G, int R>
Plan plan_for(const Shape& sh)
{
    return plan_from(sh, Cfg<G, R>::kRoundTokens, Cfg<G, R>::kMinBlocks, sh.n_seq * sh.n_kv_heads * (sh.R / R));
}

template <int G, int R>
cudaError_t launch_cfg(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                       const int32_t* seq_lens, float scale, const Shape& sh, const Plan& pl, float* partials,
                       cudaStream_t st, float* out, const AppendArgs& app)
{
    using C = Cfg<G, R>;
    const int kv_share = sh.R / R;
    // call-site slots of ensure_dynamic_smem: 1 is the wide kernel, 2 ... 13 the template instances
    constexpr int kSlot = 2 + 2 * ((G == 16 ? 0 : G == 32 ? 3 : 5) + (R == 1 ? 0 : R == 2 ? 1 : 2));
    const bool append = app.k_new != nullptr;
    // one launch per (shared KV head or not, appending or not) instance; smem call-site slots kSlot, kSlot + 1 and 64 + those
#define CQ_LAUNCH_TUNED(SHARED, APPEND, SLOT)                                                                                   \
    do {                                                                                                                        \
        cudaError_t e_ = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_tuned_kernel<G, R, SHARED, APPEND>),           \
                                             C::kSmemBytes, SLOT);                                                              \
        if (e_ != cudaSuccess) return e_;                                                                                       \
        decode_tuned_kernel<G, R, SHARED, APPEND><<<pl.grid, C::kThreads, C::kSmemBytes, st>>>(                                  \
            q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, pl.chunk, pl.n_parts, pl.tail_first, aligned32(kcb, vcb),         \
            kv_share, partials, pl.n_parts == 1 ? out : nullptr, app);                                                          \
    } while (0)
    if (kv_share > 1) {
        if (append) CQ_LAUNCH_TUNED(true, true, 62 + kSlot);
        else CQ_LAUNCH_TUNED(true, false, kSlot);
    } else {
        if (append) CQ_LAUNCH_TUNED(false, true, 62 + kSlot + 1);
        else CQ_LAUNCH_TUNED(false, false, kSlot + 1);
    }
#undef CQ_LAUNCH_TUNED
    return cudaGetLastError();
}

bool wide_shape(const Shape& sh) { return sh.head_dim == 128 && sh.c == 8 && sh.b == 10; }

// Query heads one CTA of decode_tuned_kernel serves for this shape: the largest built width that divides
// the number of query heads per KV head (16 groups: 4, 2, 1; 32 groups: 2, 1; 64 groups: 1).
int heads_per_cta(const Shape& sh)
{
    if (sh.G == 16) return sh.R % 4 == 0 ? 4 : (sh.R % 2 == 0 ? 2 : 1);
    if (sh.G == 32) return sh.R % 2 == 0 ? 2 : 1;
    return 1;
}

Plan plan_dispatch(const Shape& sh)
{
    if (wide_shape(sh)) return plan_from(sh, WideCfg::kRoundTokens, 1, sh.n_seq * sh.n_q_heads);
    const int w = heads_per_cta(sh);
    if (sh.G == 16 && w == 1) return plan_for<16, 1>(sh);
    if (sh.G == 16 && w == 2) return plan_for<16, 2>(sh);
    if (sh.G == 16 && w == 4) return plan_for<16, 4>(sh);
    if (sh.G == 32 && w == 1) return plan_for<32, 1>(sh);
    if (sh.G == 32 && w == 2) return plan_for<32, 2>(sh);
    if (sh.G == 64) return plan_for<64, 1>(sh);
    return Plan{0, 1, -1, 0u};
}

}  // namespace

bool decode_tuned_supported(const Shape& sh)
{
    if (sh.max_tokens > ((int64_t)1 << 30)) return false;
    if (wide_shape(sh)) return true;
    if (sh.head_dim != 128 || sh.b != 8) return false;
    return sh.G == 16 || sh.G == 32 || sh.G == 64;      // any number of query heads per KV head
}

int decode_tuned_parts(const Shape& sh)
{
    // (either kernel may be asked for: the workspace holds the larger of the two plans)
    const int own = plan_dispatch(sh).n_parts;
    if (!decode_pair_supported(sh)) return own;
    const int pair = decode_pair_plan(sh).n_parts;
    return pair > own ? pair : own;
}

bool decode_fused_append_supported(const Shape& sh) { return decode_tuned_supported(sh) && !wide_shape(sh); }

int decode_step_fused_launches(const Shape& sh)
{
    if (decode_pair_supported(sh)) return decode_pair_plan(sh).n_parts == 1 ? 1 : 2;
    return plan_dispatch(sh).n_parts == 1 ? 1 : 2;
}

cudaError_t launch_decode_step_fused(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                     const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh,
                                     float* out, float* partials, const AppendArgs& app, cudaStream_t st)
{
    if (!decode_fused_append_supported(sh)) return cudaErrorNotSupported;
    return launch_decode_tuned(q, kc, vc, kcb, vcb, seq_lens, scale, sh, out, partials, st, false, app);
}

cudaError_t launch_decode_tuned(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                const float* vcb, const int32_t* seq_lens, float scale, const Shape& sh, float* out,
                                float* partials, cudaStream_t st, bool per_head_tables, const AppendArgs& app)
{
    if (!per_head_tables && decode_pair_supported(sh)) {
        const DecodePlan pp = decode_pair_plan(sh);
        const cudaError_t ep = launch_decode_pair(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pp, partials, st, app, out);
        if (ep != cudaSuccess || pp.n_parts == 1) return ep;      // one part per item: the kernel wrote the output itself
        return launch_merge(partials, pp.n_parts, sh, out, st);
    }
    const Plan pl = plan_dispatch(sh);
    if (pl.chunk <= 0) return cudaErrorNotSupported;
    cudaError_t e = cudaErrorNotSupported;
    if (wide_shape(sh)) {
        if (app.k_new) return cudaErrorNotSupported;          // this kernel does not append
        e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_wide_kernel), WideCfg::kSmemBytes, 1);
        if (e != cudaSuccess) return e;
        decode_wide_kernel<<<pl.grid, WideCfg::kThreads, WideCfg::kSmemBytes, st>>>(
            q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, pl.chunk, pl.n_parts, pl.tail_first, aligned32(kcb, vcb),
            partials);
        e = cudaGetLastError();
    }
    else if (sh.G == 16 && heads_per_cta(sh) == 1) e = launch_cfg<16, 1>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pl, partials, st, out, app);
    else if (sh.G == 16 && heads_per_cta(sh) == 2) e = launch_cfg<16, 2>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pl, partials, st, out, app);
    else if (sh.G == 16 && heads_per_cta(sh) == 4) e = launch_cfg<16, 4>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pl, partials, st, out, app);
    else if (sh.G == 32 && heads_per_cta(sh) == 1) e = launch_cfg<32, 1>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pl, partials, st, out, app);
    else if (sh.G == 32 && heads_per_cta(sh) == 2) e = launch_cfg<32, 2>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pl, partials, st, out, app);
    else if (sh.G == 64) e = launch_cfg<64, 1>(q, kc, vc, kcb, vcb, seq_lens, scale, sh, pl, partials, st, out, app);
    if (e != cudaSuccess) return e;
    if (pl.n_parts == 1 && !wide_shape(sh)) return e;           // one part per item: the kernel wrote the output itself
    return launch_merge(partials, pl.n_parts, sh, out, st);
}

}  // namespace cq
