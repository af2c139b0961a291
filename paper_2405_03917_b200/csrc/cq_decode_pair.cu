// Decode attention over CQ-8c8b codes for KV heads shared by four query heads (head_dim 128,
// 16 groups of 8 channels, one byte per code): the kernel for grouped-query attention.
//
// Same re-association of Eq. 1 of the paper (K and V replaced by their CQ reconstructions,
// Section 3.2) as decode_tuned_kernel:
//   LUT[h][g][j]  = scale*log2(e) * <q_h,g , Ck[g][j]>
//   s_t[h]        = sum_g LUT[h][g][kcode[t][g]]
//   w_t[h]        = round(2^(s_t[h] - e_h))                      integer weight, unit 2^e_h
//   bins[h][g][j] += w_t[h]   for j = vcode[t][g]
//   acc[h][g*8+i] = sum_j bins[h][g][j] * Cv[g][j][i],  l[h] = sum_j bins[h][0][j]
// Measured on sm_100a, what limits this path with four heads per KV head is the number of warp
// instructions issued per token (the instruction issue slots of the four schedulers of an SM),
// before the shared-memory pipe and long before HBM.  The kernel is built around that:
//
// * K side, four query heads per lookup.  Per (head, group) the smallest entry is taken out
//   (softmax does not see a constant added to every score of a head) and the rest is stored as a
//   16-bit fixed-point number in units of delta_h = (largest entry range of the head's groups) /
//   65535.  A 32-bit word holds the entries of heads 2i and 2i+1 and the words of the two head
//   pairs of a (code value, group) are neighbours, so ONE 64-bit lookup serves the four heads: 16
//   lookup instructions per token instead of 64.  A looked-up word is one register of an
//   m16n8k32 u8 A fragment; the B operand selects byte position n mod 4 into column n, so the
//   integer MMA returns, exactly, the sums of the low bytes and of the high bytes of one head in
//   the two accumulator columns of a lane: lanes 0 and 2 of a quad get the first head of a
//   pair, lanes 1 and 3 the second.  score = low + 256 * high, an exact integer.
// * A lane therefore holds the scores of its quad's tokens for TWO heads (one of each pair),
//   turns them into weights itself and adds them to those heads' bins for 8 of the 16 groups, one
//   index computation per two adds; no weight crosses lanes.
// * Tables of 32 KiB (K) + 64 KiB (bins) let two CTAs share an SM, so one CTA's table build and
//   bins x centroids product overlap the other's main loop.
// * Code words reach the lanes through shared memory: a warp's four blocks are 1 KiB of
//   contiguous codes per tensor, which one bulk asynchronous copy (no tensor map, no multicast)
//   puts into the warp's staging tile while the previous tile is in use; the lanes then take their
//   8-byte half words with 64-bit loads.  (Direct 16-byte global loads of this access pattern
//   were measured 10 % slower.)
//
// Lane roles: lane = (r, p) = (lane / 4, lane % 4).  Quad r owns the tokens 8 (r % 2) ... + 7 of
// block r / 2 of the warp's four 16-token blocks.  With hb = p % 2 and pu = p / 2:
//   K row j (128 bytes): bytes 8 g ... 8 g + 7 = (pair 0 word, pair 1 word) of group g.  The
//     lane's m-th K code word: group 4 ((r' ^ m) % 4) + p with r' = r with its two low bits swapped
//     (16 lanes, 16 groups: distinct banks).
//   bins row j (256 bytes): word 32 (h / 2) + 16 (h % 2) + g.  The lane serves heads hb and
//     2 + hb; its m-th V code word: group 8 pu + ((r + 4 pu) % 8 ^ m), so that for every m the 32
//     lanes touch 32 distinct banks (and the 64-bit reads of the staging tile do not collide).
//   The eight bins offsets of a lane are bytes of two registers, and one PRMT builds
//   code * 256 + offset from a code byte and an offset byte (every offset is below 128, so the
//   byte's replicated sign supplies the zero upper bytes).
//
// The integer weight units, the reservation of bin room and the coarsening events are those of
// decode_tuned_kernel (see there).  In the usual case (no request pending, the lane's scores fit
// the unit, its sum is small and the total is far from its limit) a lane decides by itself, from
// a control record it read at the top of the iteration, and adds its sum to the head's total
// without waiting for the old value; no value crosses lanes.  Everything else - the first tokens
// of a head, a large sum, a full total, a pending request - takes reserve_slow(), where the
// sixteen lanes of a warp with the same hb act as one group.  That code and the coarsening are
// kept out of line: inlined into the loop they cost a quarter of the kernel's time in
// instruction fetches alone.
#include <utility>

#include "cq_bulk_copy.cuh"
#include "cq_decode_util.cuh"

namespace cq {

namespace {

struct PairCfg {
    static constexpr int kHeads = 4;                  // query heads per CTA
    static constexpr int kWarps = 8, kThreads = kWarps * 32;
    static constexpr int kBlocksPerIter = 4;          // 16-token blocks per warp iteration
    static constexpr int kRoundTokens = kWarps * kBlocksPerIter * 16;
    static constexpr int kKRowBytes = 128, kVRowBytes = 256;
    static constexpr int kKBytes = kRows * kKRowBytes;          // 32 KiB
    static constexpr int kVOffset = kKBytes;
    static constexpr int kVBytes = kRows * kVRowBytes;          // 64 KiB; also the fp32 staging area of the table build
    static constexpr int kCtlOffset = kVOffset + kVBytes;
    static constexpr int kCtlBytes = 768;                       // keeps the tiles 256-byte aligned (their words are addressed with XOR)
    static constexpr int kStageOffset = kCtlOffset + kCtlBytes; // per warp: K tile (4 blocks x 256 bytes), then V tile
    static constexpr int kTileBytes = kBlocksPerIter * 16 * 16;
    static constexpr int kSmemBytes = kStageOffset + kWarps * 2 * kTileBytes;   // 112.75 KiB: two CTAs per SM
    static constexpr int kQOffset = 0;                          // scaled query [4][128] fp32, in the K table's place until the table is written
    static constexpr int kLog2Groups = 3;             // log2 of the warps that add to a head's bins per round
    static_assert(kStageOffset % 256 == 0, "tile alignment");
};

struct PairCtl {
    // Per query head, one 16-byte record that a lane reads with one load at the top of an iteration:
    // e_cur = log2 of the weight unit of the head's bins (kUnset before the first tokens); total = bound,
    // in units of 256, on the weights added since the last coarsening; want_hint = copy of `want`.
    struct Head { int e_cur; unsigned int total; int want_hint; int pad; } head[4];
    int req_ref[4];            // coarsening request: largest score exponent the requesters need to represent
    int req_need[4];           // coarsening request: log2 bound of the largest round sum of one lane group
    int want;                  // non-zero: a warp asks every warp to stop adding and coarsen
    int range_bits[4];         // per head: largest (max - min) over its groups' table entries, as float bits
    float offset[4];           // per head: sum over groups of the entry taken out of each group
    float mins[4][16];         // per (head, group): smallest table entry
    uint64_t bar[PairCfg::kWarps][2];   // per warp: arrival of its K tile and of its V tile
    uint8_t newcode[2][16];    // codes of the token this launch appends (key, value), when its position is in the CTA's range
};
static_assert(sizeof(PairCtl) <= PairCfg::kCtlBytes, "control block");

// D = A * B + C for u8 operands: A holds looked-up table words (four bytes = four k slots), B
// selects byte position n % 4 into column n, so that columns 2p and 2p + 1 of lane p are the sums
// of the low and of the high bytes of one head.  Rows r (a0, a2) and r + 8 (a1, a3) are two tokens.
__device__ __forceinline__ void mma_bytesum_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b, int c_low)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%8}, {%9,%10,%9,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b), "r"(c_low), "r"(0));
}
__device__ __forceinline__ void mma_bytesum_acc(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%8}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b));
}

// byte k (0..7) of an 8-byte code half word
__device__ __forceinline__ uint32_t word32(const uint2& w, int k) { return (k >> 2) == 0 ? w.x : w.y; }
// code * 128 + lane_off as one multiply-add (byte offset into the K table)
__device__ __forceinline__ uint32_t k_row_index(const uint2& w, int k, uint32_t lane_off)
{
    const uint32_t code = __byte_perm(word32(w, k), 0u, 0x4440u | (uint32_t)(k & 3));
    uint32_t idx;
    asm("mad.lo.u32 %0, %1, 128, %2;" : "=r"(idx) : "r"(code), "r"(lane_off));
    return idx;
}
template <typename F, int... I>
__device__ __forceinline__ void static_for_impl(F&& f, std::integer_sequence<int, I...>) { (f(std::integral_constant<int, I>{}), ...); }
// f(integral_constant<int, 0>) ... f(integral_constant<int, N - 1>): a loop whose index is a compile-time constant
template <int N, typename F>
__device__ __forceinline__ void static_for(F&& f) { static_for_impl(f, std::make_integer_sequence<int, N>{}); }

// code * 256 + (byte m % 4 of `offs`): byte offset into the bins.  Result bytes: the offset byte, the code
// byte k of the half word, and twice the replicated sign of the offset byte (zero: offsets are below 128).
template <int K, int M>
__device__ __forceinline__ uint32_t v_row_index(const uint2& w, uint32_t offs)
{
    // (prmt in PTX form: the fourth bit of a selector digit asks for the byte's replicated sign)
    constexpr uint32_t ob = 4u + (uint32_t)(M & 3);
    constexpr uint32_t sel = ob | ((uint32_t)(K & 3) << 4) | ((ob | 8u) << 8) | ((ob | 8u) << 12);
    uint32_t idx;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(idx) : "r"(K < 4 ? w.x : w.y), "r"(offs), "n"(sel));
    return idx;
}

// Coarsening event (see decode_tuned_kernel): entered by every thread of the CTA, right after the
// event's first barrier.  Per head: new unit from the published requests, bins shifted right with
// rounding, total rescaled.  Out of line on purpose.
__device__ __noinline__ void coarsen_bins(uint8_t* smem, PairCtl* ctl)
{
    using C = PairCfg;
    constexpr int R = C::kHeads;
    int shift[R], e_next[R];
    unsigned int t_next[R];
    bool any_shift = false;
#pragma unroll
    for (int h = 0; h < R; ++h) {
        const int e = ctl->head[h].e_cur, cmr = ctl->req_ref[h], need = ctl->req_need[h];
        const unsigned int tot = ctl->head[h].total;
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
        for (int i = threadIdx.x; i < C::kVBytes / 4; i += C::kThreads) {
            const int word = i & 63;                                // word 32 (h / 2) + 16 (h % 2) + g of a bins row
            const int hw_ = 2 * (word >> 5) + ((word >> 4) & 1);
            int k = shift[0];
#pragma unroll
            for (int h = 1; h < R; ++h) k = hw_ == h ? shift[h] : k;
            if (k > 0) {
                uint32_t* bp = reinterpret_cast<uint32_t*>(smem + C::kVOffset) + i;
                const uint32_t v = *bp;
                *bp = k >= 32 ? 0u : (v >> k) + ((v >> (k - 1)) & 1u);
            }
        }
    }
    event_barrier(C::kThreads);                         // every thread has read the request and rescaled its bins
    if (threadIdx.x == 0) {
#pragma unroll
        for (int h = 0; h < R; ++h) {
            ctl->head[h].e_cur = e_next[h];
            ctl->head[h].total = t_next[h];
            ctl->head[h].want_hint = 0;
            ctl->req_ref[h] = kUnset;
            ctl->req_need[h] = kUnset;
        }
        ctl->want = 0;
    }
    event_barrier(C::kThreads);                         // the new state is visible
}

// A lane whose weights (for one head, one iteration) sum to less than kFastLane256 units of 256 adds them to
// the head's total without asking, after a look at the total as it stood at the top of its iteration.  A warp
// adds at most 8 such sums per head and iteration (2^19).  Once the total has passed the soft limit
// kBinLimit256 - 2^19 - kFastSlack256, every later look sends its warp to reserve_slow; until then each of
// the 8 warps can still be inside one iteration that looked earlier, plus the add that crossed the limit: at
// most 9 * 2^19 = kFastSlack256 on top, so the total stays below kBinLimit256 and no bin can wrap.
constexpr unsigned int kFastLane256 = 1u << 16;
constexpr unsigned int kFastSlack256 = 9u << 19;

// Room for a warp's weights when the usual case does not apply (entered by the whole warp).  The
// sixteen lanes with the same hb = lane % 2 form a group that serves heads hb and 2 + hb.  Per
// head: ref_lane = the lane's reference exponent (kUnset without tokens), z_lane = the sum of its
// weights 2^(score - ref_lane).  The group reserves the sum of its weights on the head's total
// with the old value in hand, or asks for a coarser unit and joins the event.  Bounded: every
// event coarsens the refused head by at least two bits.  Returns the units to use for the two heads.
// (Scalars in, scalars out: nothing the caller's loop keeps in registers is forced into memory.)
__device__ __noinline__ int2 reserve_slow(uint8_t* smem, PairCtl* ctl, int ref_lane0, int ref_lane1, float z_lane0, float z_lane1)
{
    const int ref_lane[2] = {ref_lane0, ref_lane1};
    const float z_lane[2] = {z_lane0, z_lane1};
    int eu[2] = {kUnset, kUnset};
    using C = PairCfg;
    const int lane = threadIdx.x & 31, hb = lane & 1;
    const unsigned grp_mask = hb ? 0xaaaaaaaau : 0x55555555u;
    const bool grp_leader = lane == hb;
    int ref[2];
    float zsum[2];
    bool any_tokens = false;                                            // the same in every lane of the warp
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        ref[u] = __reduce_max_sync(grp_mask, ref_lane[u]);
        any_tokens = ref[u] != kUnset;
        const float zrel = ref_lane[u] == kUnset ? 0.f : z_lane[u] * pow2i(ref_lane[u] - ref[u]);
        // sum over the group in 2^-16 steps, rounded up (the lanes p and p + 2 of a quad hold the same
        // tokens, so the group's sum counts every token twice)
        zsum[u] = (float)__reduce_add_sync(grp_mask, __float2uint_ru(zrel * 65536.f)) * (0.5f / 65536.f);
    }
    for (int attempt = 0; attempt < 64; ++attempt) {
        if (*reinterpret_cast<volatile int*>(&ctl->want) != 0) {
            // someone needs a coarser unit: tell the event what this group will need, then join it
            if (grp_leader) {
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    if (ref[u] != kUnset) {
                        atomicMax(&ctl->req_ref[2 * u + hb], ref[u]);
                        atomicMax(&ctl->req_need[2 * u + hb], ref[u] + ilogbf(fmaxf(zsum[u], 1e-30f)) + 1);
                    }
            }
            event_barrier(C::kThreads);
            coarsen_bins(smem, ctl);
            continue;
        }
        if (!any_tokens) break;
        bool ok = true;
        unsigned int mine[2] = {0u, 0u};
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int h = 2 * u + hb;
            eu[u] = *reinterpret_cast<volatile int*>(&ctl->head[h].e_cur);
            if (eu[u] == kUnset || ref[u] - eu[u] > kMaxWeightBits) { ok = false; continue; }
            // this group's weights in the current unit, rounded up, in units of 256
            const float cw = (zsum[u] * pow2i(ref[u] - eu[u]) * 1.00002f + (float)(16 * C::kBlocksPerIter)) * (1.f / 256.f) + 1.f;
            const unsigned int ci = (unsigned int)fminf(cw, 6.7e7f);
            unsigned int old = 0u;
            if (grp_leader) old = atomicAdd(&ctl->head[h].total, ci);
            old = __shfl_sync(grp_mask, old, hb);
            mine[u] = ci;
            // (the sums that other warps add without asking are covered by kFastSlack256)
            if (old + ci + kFastSlack256 >= kBinLimit256) ok = false;
        }
        ok = __all_sync(0xffffffffu, ok);
        if (ok) break;
        // give the reservations back, publish what is needed, raise the request, join the event
        if (grp_leader) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int h = 2 * u + hb;
                if (mine[u]) atomicSub(&ctl->head[h].total, mine[u]);
                atomicMax(&ctl->req_ref[h], ref[u]);
                atomicMax(&ctl->req_need[h], ref[u] + ilogbf(fmaxf(zsum[u], 1e-30f)) + 1);
            }
            atomicExch(&ctl->want, 1);
#pragma unroll
            for (int h = 0; h < C::kHeads; ++h) atomicExch(&ctl->head[h].want_hint, 1);
        }
        event_barrier(C::kThreads);
        coarsen_bins(smem, ctl);
    }
    return make_int2(eu[0], eu[1]);
}

// The value codes of the token that the launch appends (CQ encode, Section 3.2), by the whole CTA: warp w takes
// groups 2 w and 2 w + 1, its lanes walk the centroids; d_j = sum_i (x_i - C_ji)^2 in fp32 in the order of the
// encode kernels, lowest index on ties.  The codes go to the control block and, from the CTA that `writer` names,
// to position `pos` of the cache.  (The key codes come out of the table build, which reads the key centroids anyway.)
__device__ __noinline__ void encode_new_value(PairCtl* ctl, AppendArgs app, const float* __restrict__ vcb, Shape sh,
                                              int64_t s, int hkv, int64_t pos, bool writer, bool aligned32)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll 1
    for (int e = 0; e < 2; ++e) {
        const int g = warp * 2 + e;
        const __half* xp = app.v_new + (s * sh.n_kv_heads + hkv) * 128 + g * 8;
        const float* cg = vcb + ((int64_t)hkv * 16 + g) * kRows * 8;
        float xg[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) xg[i] = __half2float(xp[i]);
        float best = INFINITY;
        int arg = 0;
        float cv[kRows / 32][8];                      // all loads in flight at once
#pragma unroll
        for (int t = 0; t < kRows / 32; ++t) load_centroid<8>(cg + (int64_t)(t * 32 + lane) * 8, cv[t], aligned32);
#pragma unroll
        for (int t = 0; t < kRows / 32; ++t) {
            const int j = t * 32 + lane;
            float d = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float diff = xg[i] - cv[t][i];
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
        if (lane == 0) {
            ctl->newcode[1][g] = (uint8_t)arg;
            if (writer) app.vc_w[code_word_offset(sh, sh.n_kv_heads, s, hkv, pos / kTokenBlock, g) + pos % kTokenBlock] = (uint8_t)arg;
        }
    }
}

// Puts the new token's codes into a 64-bit code word that was loaded straight from global memory: word_off is the
// word's byte offset inside its warp's tile, new_off + 16 g that of the new token's code of group g.
__device__ __noinline__ uint2 patch_word(uint2 w, uint32_t word_off, uint32_t new_off, const uint8_t* newcode)
{
#pragma unroll 1
    for (int g = 0; g < 16; ++g) {
        const uint32_t d = new_off + 16u * g - word_off;
        if (d < 4u)
            w.x = (w.x & ~(0xffu << (8 * d))) | ((uint32_t)newcode[g] << (8 * d));
        else if (d < 8u)
            w.y = (w.y & ~(0xffu << (8 * (d - 4)))) | ((uint32_t)newcode[g] << (8 * (d - 4)));
    }
    return w;
}

__global__ void __launch_bounds__(PairCfg::kThreads, 2)
decode_pair_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                   const float* __restrict__ kcb, const float* __restrict__ vcb,
                   const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int chunk_tokens, int n_parts,
                   int tail_first, int cb_aligned32, float* __restrict__ partials, AppendArgs app, float* __restrict__ out)
{
    using C = PairCfg;
    constexpr int R = C::kHeads;
    extern __shared__ __align__(1024) uint8_t smem[];
    PairCtl* ctl = reinterpret_cast<PairCtl*>(smem + C::kCtlOffset);
    float* qs = reinterpret_cast<float*>(smem + C::kQOffset);
    float* stage = reinterpret_cast<float*>(smem + C::kVOffset);       // [4][16][256] fp32 during the table build

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int p = lane & 3, r = lane >> 2;
    const int hb = p & 1, pu = p >> 1;

    // Work item: (context part, sequence, group of four query heads).  Items before tail_first take
    // their whole context in one CTA; each later item is spread over n_parts CTAs of chunk_tokens
    // (see the launch plan).
    const int n_head_groups = sh.n_q_heads / R;
    const int kv_share = sh.R / R;                    // CTAs (of four query heads) that share one KV head
    const int n_items = (int)(n_head_groups * sh.n_seq);
    int item = blockIdx.x % n_items;
    int part = (int)(blockIdx.x / n_items);
    bool whole = false;
    if (tail_first >= 0) {
        whole = (int)blockIdx.x < tail_first;
        item = whole ? blockIdx.x : tail_first + (blockIdx.x - tail_first) / n_parts;
        part = whole ? 0 : (blockIdx.x - tail_first) % n_parts;
    }
    const int head_group = item % n_head_groups;
    const int hkv = head_group / kv_share;
    const int64_t s = seq_by_rank(seq_lens, (int)sh.n_seq, sh.max_tokens, item / n_head_groups);

    // (the query travels while the context length is looked up)
    const __half* qrow = q + (s * sh.n_q_heads + (int64_t)head_group * R) * 128;
    const __half q_lo = qrow[threadIdx.x], q_hi = qrow[C::kThreads + threadIdx.x];
    static_assert(R * 128 == 2 * C::kThreads, "two query elements per thread");
    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    // With an append, seq_lens counts the tokens cached before this launch: the new token takes position n and
    // the attention covers n + 1 tokens (a sequence at capacity gets no new token).
    const bool has_new = app.k_new != nullptr && n < sh.max_tokens;
    if (has_new) ++n;
    const int64_t t_begin = (int64_t)part * chunk_tokens;
    const int64_t t_end = (whole || t_begin + chunk_tokens >= n) ? n : t_begin + chunk_tokens;
    const int stride = partial_stride(128);
    float* part_base = partials + ((s * sh.n_q_heads + (int64_t)head_group * R) * n_parts + part) * stride;
    // partial of query head head_group*4 + h: part_base + h * n_parts * stride
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
        if (out)            // one part per item and nothing to attend: the zero row of the merge
            for (int i = threadIdx.x; i < R * 128; i += C::kThreads) out[(s * sh.n_q_heads + (int64_t)head_group * R) * 128 + i] = 0.f;
        return;
    }

    const int64_t blk0 = t_begin / kTokenBlock;
    const int n_tok = (int)(t_end - blk0 * kTokenBlock);                   // tokens of this CTA, counted from its first block
    // The new token, when its position is in this CTA's range: which warp's tile of which iteration holds its block.
    // The CTA works its codes out itself (so do the CTAs of the other query heads that share the KV head) and puts
    // them into the staged tile; the CTA of the KV head's first four query heads also writes them to the cache.
    const bool new_here = has_new && t_begin <= n - 1 && n - 1 < t_end;
    const int new_blk = new_here ? (int)((n - 1) / kTokenBlock - blk0) : 0;
    const int new_it = new_blk / (C::kWarps * C::kBlocksPerIter), new_warp = (new_blk / C::kBlocksPerIter) % C::kWarps;
    const uint32_t new_off = (uint32_t)(new_blk % C::kBlocksPerIter) * 256u + (uint32_t)((n - 1) % kTokenBlock);   // + 16 g: byte in the tile
    const int n_iters = (n_tok + C::kRoundTokens - 1) / C::kRoundTokens;
    const uint8_t* kbase = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, blk0, 0);
    const uint8_t* vbase = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, blk0, 0);

    // Codebooks are read in units of 4 x 32 centroids (32 registers per lane): a warp owns two
    // groups, its lanes walk the code values, the next unit is loaded while the current one is used.
    constexpr int kJb = 4;
    constexpr int kUnits = 2 * (kRows / 32 / kJb);          // 4 units per warp
    auto load_unit = [&](float (&cv)[kJb][8], const float* cb, int u) {
        const int g = warp * 2 + (u >> 1);
        const float* cg = cb + (((int64_t)hkv * 16 + g) * kRows + (u & 1) * (kJb * 32) + lane) * 8;
#pragma unroll
        for (int jb = 0; jb < kJb; ++jb) load_centroid<8>(cg + jb * 32 * 8, cv[jb], cb_aligned32 != 0);
    };
    float cva[kJb][8], cvb[kJb][8];
    load_unit(cva, kcb, 0);

    // table offsets of this lane's code words (bytes inside a K row / inside plane 0 of a bins row)
    // m-th K code word: koff0 ^ (32 m).  (The two low bits of r are swapped so that the quads of a half warp,
    // which read the two 8-byte halves of code words in two blocks, also spread over the staging tile's banks.)
    const uint32_t koff0 = 8u * (4 * (((r >> 1) & 1) | ((r & 1) << 1)) + p);
    const int vx = (r + 4 * pu) & 7;
    uint32_t voffs[2] = {0u, 0u};                                        // m-th V code word: byte m % 4 of voffs[m / 4]
#pragma unroll
    for (int m = 0; m < 8; ++m) voffs[m >> 2] |= (4u * (16 * hb + 8 * pu + (vx ^ m))) << (8 * (m & 3));
    const uint32_t bsel = 1u << (8 * (r & 3));                          // B fragment: column n = lane / 4 takes byte n % 4

    // Code tiles.  Tile `it` of this warp = its four blocks of iteration `it`, 1 KiB of contiguous
    // codes per tensor (less at the end of the chunk; blocks past the end are not copied and keep
    // whatever the tile held: any byte is a valid table row, and those tokens are masked).  Lane 0
    // asks for a tensor's next tile as soon as every lane has taken its words of the current one.
    uint8_t* ktile = smem + C::kStageOffset + warp * 2 * C::kTileBytes;
    uint8_t* vtile = ktile + C::kTileBytes;
    // this lane's half word of its first code word in the K tile and in the V tile; word m is 64 m / 16 m bytes
    // away in the XOR sense (the tiles are 128-byte aligned)
    const uint32_t my_ktile = (uint32_t)(C::kStageOffset + warp * 2 * C::kTileBytes + (r >> 1) * 256 + 8 * (r & 1)) + 2u * koff0;
    const uint32_t my_vtile = (uint32_t)(C::kStageOffset + warp * 2 * C::kTileBytes + C::kTileBytes + (r >> 1) * 256 + 8 * (r & 1)) +
                              16u * (8 * pu + vx);
    uint64_t* kbar = &ctl->bar[warp][0];
    uint64_t* vbar = &ctl->bar[warp][1];
    uint32_t kphase = 0u, vphase = 0u;
    bool bulk = true;                       // false after a wait that gave up: plain loads from then on
    bool k_out = false, v_out = false;      // a copy into the tile has been requested and not yet awaited
    const int n_blocks_cta = (n_tok + kTokenBlock - 1) / kTokenBlock;   // blocks holding a valid token
    // bytes of this warp's tile of iteration `it` (per tensor)
    auto tile_bytes = [&](int it) -> uint32_t {
        int nb = n_blocks_cta - (it * C::kWarps + warp) * C::kBlocksPerIter;
        nb = nb < 0 ? 0 : (nb > C::kBlocksPerIter ? C::kBlocksPerIter : nb);
        return (uint32_t)nb * 256u;
    };
    auto request_tile = [&](uint8_t* tile, uint64_t* bar, const uint8_t* base, int it, uint32_t bytes) {      // lane 0 only
        const int64_t off = (int64_t)(it * C::kWarps + warp) * (C::kBlocksPerIter * 256);
        fence_async_smem();
        mbar_expect_tx(bar, bytes);
        bulk_copy_g2s(tile, base + off, bytes, bar);
    };
    uint2 kw[4], vw[8];
    // the K words of tile `it` into registers; then the tile is free for iteration it + 1
    auto take_k = [&](int it) {
        bool have = false;
        const uint32_t bytes = tile_bytes(it);
        if (bulk && bytes != 0u) {
            have = mbar_wait(kbar, kphase);
            have = __all_sync(0xffffffffu, have);
            if (have) { kphase ^= 1u; k_out = false; } else bulk = false;
        }
        const bool patch = new_here && it == new_it && warp == new_warp;
        if (have || bytes == 0u) {
            if (patch) {
                if (lane < 16) ktile[new_off + 16u * lane] = ctl->newcode[0][lane];
                __syncwarp();
            }
#pragma unroll
            for (int m = 0; m < 4; ++m) kw[m] = *reinterpret_cast<const uint2*>(smem + (my_ktile ^ (64u * m)));
        } else {
            const int blk = (it * C::kWarps + warp) * C::kBlocksPerIter + (r >> 1);
            const int64_t off = (int64_t)blk * 256 + 8 * (r & 1);
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                kw[m] = blk < n_blocks_cta ? __ldg(reinterpret_cast<const uint2*>(kbase + off + 2u * (koff0 ^ (32u * m))))
                                           : make_uint2(0u, 0u);
                if (patch) kw[m] = patch_word(kw[m], (uint32_t)((r >> 1) * 256 + 8 * (r & 1)) + 2u * (koff0 ^ (32u * m)), new_off, ctl->newcode[0]);
            }
        }
        __syncwarp();
        const uint32_t next = it + 1 < n_iters ? tile_bytes(it + 1) : 0u;
        if (bulk && next != 0u) {
            k_out = true;
            if (lane == 0) request_tile(ktile, kbar, kbase, it + 1, next);
        }
    };
    auto take_v = [&](int it) {
        bool have = false;
        const uint32_t bytes = tile_bytes(it);
        if (bulk && bytes != 0u) {
            have = mbar_wait(vbar, vphase);
            have = __all_sync(0xffffffffu, have);
            if (have) { vphase ^= 1u; v_out = false; } else bulk = false;
        }
        const bool patch = new_here && it == new_it && warp == new_warp;
        if (have || bytes == 0u) {
            if (patch) {
                if (lane < 16) vtile[new_off + 16u * lane] = ctl->newcode[1][lane];
                __syncwarp();
            }
#pragma unroll
            for (int m = 0; m < 8; ++m) vw[m] = *reinterpret_cast<const uint2*>(smem + (my_vtile ^ (16u * m)));
        } else {
            const int blk = (it * C::kWarps + warp) * C::kBlocksPerIter + (r >> 1);
            const int64_t off = (int64_t)blk * 256 + 8 * (r & 1);
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                vw[m] = blk < n_blocks_cta ? __ldg(reinterpret_cast<const uint2*>(vbase + off + 16u * (8 * pu + (vx ^ m))))
                                           : make_uint2(0u, 0u);
                if (patch) vw[m] = patch_word(vw[m], (uint32_t)((r >> 1) * 256 + 8 * (r & 1)) + 16u * (8 * pu + (vx ^ m)), new_off, ctl->newcode[1]);
            }
        }
        __syncwarp();
        const uint32_t next = it + 1 < n_iters ? tile_bytes(it + 1) : 0u;
        if (bulk && next != 0u) {
            v_out = true;
            if (lane == 0) request_tile(vtile, vbar, vbase, it + 1, next);
        }
    };

    // ---------------------------------------------------------------- set-up: query, control block
    if (threadIdx.x < 4) {
        ctl->head[threadIdx.x].e_cur = kUnset;
        ctl->head[threadIdx.x].total = 0u;
        ctl->head[threadIdx.x].want_hint = 0;
        ctl->req_ref[threadIdx.x] = kUnset;
        ctl->req_need[threadIdx.x] = kUnset;
        ctl->range_bits[threadIdx.x] = 0;
    }
    if (threadIdx.x == 4) ctl->want = 0;
    if (threadIdx.x == 5) {
        for (int w = 0; w < C::kWarps; ++w) {
            mbar_init(&ctl->bar[w][0], 1);
            mbar_init(&ctl->bar[w][1], 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    qs[threadIdx.x] = __half2float(q_lo) * scale_log2e;
    qs[C::kThreads + threadIdx.x] = __half2float(q_hi) * scale_log2e;
    if (new_here) encode_new_value(ctl, app, vcb, sh, s, hkv, n - 1, head_group % kv_share == 0, cb_aligned32 != 0);
    __syncthreads();
    // the first code tiles travel during the table build
    k_out = v_out = tile_bytes(0) != 0u;
    if (lane == 0 && k_out) {
        request_tile(ktile, kbar, kbase, 0, tile_bytes(0));
        request_tile(vtile, vbar, vbase, 0, tile_bytes(0));
    }

    // Table build, first pass: fp32 entries into the staging area (the later bins), entry (h, g, j)
    // at word (h*16 + g)*256 + (j ^ (16*(h/2) + g)): a warp writing 32 consecutive j of one (h, g)
    // and a warp reading one j of the 32 (h/2, g) both touch 32 distinct banks.  Per (head, group)
    // the smallest and the largest entry are kept.
    {
        float qreg[R][8];
        float vmin[R], vmax[R];
        // the new token's key, when this CTA appends it: its code of group g is the centroid nearest to it, found on
        // the way (d_j = sum_i (x_i - C_ji)^2 in fp32 in the order of the encode kernels, lowest index on ties)
        float xnew[8], dnew = INFINITY;
        int jnew = 0;
        auto build_unit = [&](const float (&cv)[kJb][8], int u) {
            const int g = warp * 2 + (u >> 1);
            if ((u & 1) == 0 && new_here) {
                const __half* xp = app.k_new + (s * sh.n_kv_heads + hkv) * 128 + g * 8;
#pragma unroll
                for (int i = 0; i < 8; ++i) xnew[i] = __half2float(xp[i]);
                dnew = INFINITY;
                jnew = 0;
            }
            if ((u & 1) == 0) {
#pragma unroll
                for (int h = 0; h < R; ++h) {
                    vmin[h] = INFINITY;
                    vmax[h] = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 8; ++i) qreg[h][i] = qs[h * 128 + g * 8 + i];
                }
            }
#pragma unroll
            for (int jb = 0; jb < kJb; ++jb) {
                const int j = (u & 1) * (kJb * 32) + jb * 32 + lane;
#pragma unroll
                for (int h = 0; h < R; ++h) {
                    float dot = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) dot = fmaf(qreg[h][i], cv[jb][i], dot);
                    vmin[h] = fminf(vmin[h], dot);
                    vmax[h] = fmaxf(vmax[h], dot);
                    stage[(h * 16 + g) * kRows + (j ^ (16 * (h >> 1) + g))] = dot;
                }
                if (new_here) {
                    float d = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float diff = xnew[i] - cv[jb][i];
                        d = fmaf(diff, diff, d);
                    }
                    if (d < dnew) { dnew = d; jnew = j; }        // a lane's j ascend: strict < keeps the lowest index
                }
            }
            if ((u & 1) == 1 && new_here) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, dnew, o);
                    const int oa = __shfl_xor_sync(0xffffffffu, jnew, o);
                    if (ob < dnew || (ob == dnew && oa < jnew)) { dnew = ob; jnew = oa; }
                }
                if (lane == 0) {
                    ctl->newcode[0][g] = (uint8_t)jnew;
                    if (head_group % kv_share == 0)
                        app.kc_w[code_word_offset(sh, sh.n_kv_heads, s, hkv, (n - 1) / kTokenBlock, g) + (n - 1) % kTokenBlock] = (uint8_t)jnew;
                }
            }
            if ((u & 1) == 1) {
#pragma unroll
                for (int h = 0; h < R; ++h) {
                    const float mn = dec_float(__reduce_min_sync(0xffffffffu, enc_float(vmin[h])));
                    const float mx = dec_float(__reduce_max_sync(0xffffffffu, enc_float(vmax[h])));
                    if (lane == 0) {
                        ctl->mins[h][g] = mn;
                        const float range = mx - mn;                     // >= 0 (or NaN / inf for non-finite inputs)
                        atomicMax(&ctl->range_bits[h], __float_as_int(range >= 0.f ? range : 0.f));
                    }
                }
            }
        };
#pragma unroll 1
        for (int u = 0; u < kUnits; u += 2) {
            load_unit(cvb, kcb, u + 1);
            build_unit(cva, u);
            if (u + 2 < kUnits) load_unit(cva, kcb, u + 2);
            build_unit(cvb, u + 1);
        }
    }
    __syncthreads();

    // Second pass: lane = (head pair hp = lane / 16, group g = lane % 16) writes word 2 g + hp of the
    // rows warp*32 ... +31: a row's 32 words, one per lane.
    {
        const int hp = lane >> 4, g = lane & 15;
        const float r0 = __int_as_float(ctl->range_bits[2 * hp]), r1 = __int_as_float(ctl->range_bits[2 * hp + 1]);
        const float inv0 = r0 > 1e-30f ? 65535.f / r0 : 0.f, inv1 = r1 > 1e-30f ? 65535.f / r1 : 0.f;
        const float m0 = ctl->mins[2 * hp][g], m1 = ctl->mins[2 * hp + 1][g];
        const float* s0 = stage + ((2 * hp) * 16 + g) * kRows;
        const float* s1 = stage + ((2 * hp + 1) * 16 + g) * kRows;
#pragma unroll 8
        for (int i = 0; i < kRows / C::kWarps; ++i) {
            const int j = warp * (kRows / C::kWarps) + i;
            // round to nearest by adding 1.5 * 2^23: the integer is then in the low mantissa bits (no
            // conversion instruction; non-finite inputs end up clamped like everything else)
            const float u0 = fminf(fmaxf((s0[j ^ lane] - m0) * inv0, 0.f), 65535.f) + 12582912.f;
            const float u1 = fminf(fmaxf((s1[j ^ lane] - m1) * inv1, 0.f), 65535.f) + 12582912.f;
            *reinterpret_cast<uint32_t*>(smem + j * C::kKRowBytes + (2 * g + hp) * 4) =
                ((uint32_t)__float_as_int(u0) & 0xffffu) | ((uint32_t)__float_as_int(u1) << 16);
        }
        if (threadIdx.x < R) {
            float o = 0.f;
            for (int gg = 0; gg < 16; ++gg) o += ctl->mins[threadIdx.x][gg];
            ctl->offset[threadIdx.x] = o;
        }
    }
    __syncthreads();
    // bins start at zero
    for (int i = threadIdx.x; i < C::kVBytes / 16; i += C::kThreads)
        *reinterpret_cast<uint4*>(smem + C::kVOffset + i * 16) = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();

    // ---------------------------------------------------------------- main loop over the chunk
    // This lane's heads: hb (pair 0) and 2 + hb (pair 1); index u = 0, 1 below.
    float delta[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const float rng = __int_as_float(ctl->range_bits[2 * u + hb]);
        delta[u] = rng > 1e-30f ? rng * (1.f / 65535.f) : 0.f;
    }
    const uint32_t head_rec = smem_addr(&ctl->head[hb]);                // record of head hb; head 2 + hb is 32 bytes on

    // K side of one token: four 64-bit lookups (one per code word, both head pairs), then one MMA chain:
    // fragment row r takes the words of pair 0, row r + 8 the words of pair 1 (the two halves of a lookup
    // are neighbours in the A fragment), two code words per MMA.  The scores of the lane's two heads come
    // out as exact integers held in floats.
    float sc[2][8];
    auto k_lookup = [&](uint2 (&dst)[4], int k) {
#pragma unroll
        for (int m = 0; m < 4; ++m)
            dst[m] = *reinterpret_cast<const uint2*>(smem + k_row_index(kw[m], k, koff0 ^ (32u * m)));
    };
    auto k_score = [&](const uint2 (&src)[4], int k) {
        int d[4];
        // columns start at 2^23 as float bits (low sums) and 0 (high sums): low + 256 * high < 2^21, so the
        // float with these bits, minus 2^23, is the integer score, exactly
        mma_bytesum_first(d, src[0].x, src[0].y, src[1].x, src[1].y, bsel, 0x4b000000);
        mma_bytesum_acc(d, src[2].x, src[2].y, src[3].x, src[3].y, bsel);
        sc[0][k] = __int_as_float(d[0] + (d[1] << 8)) - 8388608.f;
        sc[1][k] = __int_as_float(d[2] + (d[3] << 8)) - 8388608.f;
    };

    // The loop is software-pipelined: the K side of iteration it + 1 is interleaved, token by token, with the
    // V side of iteration it, so that the lookups' and the MMAs' latencies pass behind the bin updates.
    uint2 a[2][4];
    take_k(0);
    static_for<8>([&](auto kc_) {
        constexpr int k = decltype(kc_)::value;
        k_lookup(a[k & 1], k);
        if (k >= 1) k_score(a[(k - 1) & 1], k - 1);
    });
    k_score(a[1], 7);
    take_v(0);

    for (int it = 0; it < n_iters; ++it) {
        // the heads' control records as they stand now
        int4 seen[2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
            asm volatile("ld.volatile.shared.v4.s32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(seen[u].x), "=r"(seen[u].y), "=r"(seen[u].z), "=r"(seen[u].w) : "r"(head_rec + 32u * u));

        // tokens past the end of the context (only the warp that holds the ragged end pays)
        const int tok0 = ((it * C::kWarps + warp) * C::kBlocksPerIter + (r >> 1)) * kTokenBlock + 8 * (r & 1);
        const bool ragged = ((it * C::kWarps + warp) * C::kBlocksPerIter + C::kBlocksPerIter) * kTokenBlock > n_tok;
        if (ragged) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (tok0 + k >= n_tok) sc[0][k] = sc[1][k] = -1.f;
        }
        // Per head, from this lane's own eight tokens: reference exponent ref >= largest score, weights
        // 2^(score - ref) <= 1 and their sum.  Usual case, decided from the records just read: no request
        // pending, the scores fit the unit, the sum is small and the total far from its limit -> the sum
        // goes to the total without waiting for the old value.  (No event can happen between the read of the
        // records and this warp's bin updates: an event needs this warp.)
        int ref[2], eu[2];
        float y[2][8], zlane[2];
        unsigned int ci[2];
        bool fast = true, have = false;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            float mx = -1.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) mx = fmaxf(mx, sc[u][k]);
            have = mx >= 0.f;                                           // this lane holds a token of the context
            // ref = round(mx * delta) + 1, formed with the 1.5 * 2^23 trick (no conversion instruction)
            const float t = fmaf(mx, delta[u], 12582912.f);
            const float fref = have ? (t - 12582912.f) + 1.f : 0.f;
            ref[u] = have ? (__float_as_int(t) - 0x4b400000) + 1 : kUnset;
            float z = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                y[u][k] = ex2(fmaf(sc[u][k], delta[u], -fref));
                z += y[u][k];
            }
            if (ragged) {
                z = 0.f;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (sc[u][k] < 0.f) y[u][k] = 0.f;
                    z += y[u][k];
                }
            }
            zlane[u] = z;
            eu[u] = seen[u].x;
            ci[u] = 0u;
            bool f = seen[u].z == 0 && eu[u] != kUnset;
            if (f && have) {
                // this lane's weights in the current unit, rounded up, in units of 256
                const float cw = (z * pow2i(ref[u] - eu[u]) * 1.00002f + 8.f) * (1.f / 256.f) + 1.f;
                ci[u] = (unsigned int)fminf(cw, 6.7e7f);
                f = ref[u] - eu[u] <= kMaxWeightBits && cw < (float)kFastLane256 &&
                    (unsigned int)seen[u].y + 8u * kFastLane256 + kFastSlack256 < kBinLimit256;
            }
            fast = fast && f;
        }
        if (__all_sync(0xffffffffu, fast)) {
            // one add per head for the warp: the lanes' sums in steps of 16 (rounded up, below 2^12 each), the two
            // heads with hb = 0 / 1 in the two halves of a word, summed over the warp; lanes 0 ... 3 add one head each
            // (the lanes p and p + 2 of a quad hold the same tokens: only p < 2 counts)
            uint32_t packed[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t c16 = (have && pu == 0) ? (ci[u] + 15u) >> 4 : 0u;
                packed[u] = __reduce_add_sync(0xffffffffu, c16 << (16 * hb));
            }
            if (lane < 4) {
                const uint32_t pk = (lane & 2) ? packed[1] : packed[0];                 // head 2 (lane / 2) + lane % 2
                atomicAdd(&ctl->head[lane].total, ((lane & 1) ? pk >> 16 : pk & 0xffffu) << 4);
            }
        } else {
            const int2 e2 = reserve_slow(smem, ctl, ref[0], ref[1], zlane[0], zlane[1]);
            eu[0] = e2.x;
            eu[1] = e2.y;
        }

        // V side of this iteration (the lane's integer weights into the bins of its two heads, for its
        // eight groups; a lane without tokens adds zeros) interleaved with the K side of the next one
        // (past the last iteration it runs on whatever the tile holds; nothing uses those scores).
        const float f0 = have ? pow2i(ref[0] - eu[0]) : 0.f;            // powers of two <= 2^kMaxWeightBits
        const float f1 = have ? pow2i(ref[1] - eu[1]) : 0.f;
        if (it + 1 < n_iters) take_k(it + 1);
        static_for<8>([&](auto kc_) {
            constexpr int k = decltype(kc_)::value;
            k_lookup(a[k & 1], k);
            const uint32_t w0 = __float2uint_rn(y[0][k] * f0), w1 = __float2uint_rn(y[1][k] * f1);
            static_for<8>([&](auto mc_) {
                constexpr int m = decltype(mc_)::value;
                unsigned int* bin = reinterpret_cast<unsigned int*>(smem + C::kVOffset + v_row_index<k, m>(vw[m], voffs[m >> 2]));
                atomicAdd(bin, w0);
                atomicAdd(bin + 32, w1);
            });
            if (k >= 1) k_score(a[(k - 1) & 1], k - 1);
        });
        k_score(a[1], 7);
        if (it + 1 < n_iters) take_v(it + 1);
    }
    // (after a wait that gave up, a requested copy may still be on its way: it must land before the CTA ends)
    if (!bulk) {
        if (k_out) mbar_wait(kbar, kphase);
        if (v_out) mbar_wait(vbar, vphase);
    }
    // Warps that are done keep joining coarsening events until every warp is done.
    for (int guard = 0; guard < 4096; ++guard) {
        event_barrier(C::kThreads);
        if (*reinterpret_cast<volatile int*>(&ctl->want) == 0) break;
        coarsen_bins(smem, ctl);
    }
    __syncthreads();

    // ---------------------------------------------------------------- epilogue: bins x V centroids
    // Lane = (hb', g) reads words `lane` of both planes of row j (heads hb' and 2 + hb', group g): a
    // conflict-free row read; the centroid (g, j) is one 32-byte load.  A warp takes 32 rows; the
    // eight warps' partial sums meet in shared memory (the K table is no longer needed).
    {
        const int g = lane & 15;
        float acc0[8], acc1[8], l0 = 0.f, l1 = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc0[i] = acc1[i] = 0.f;
        const float* cg = vcb + (((int64_t)hkv * 16 + g) * kRows + warp * (kRows / C::kWarps)) * 8;
        const uint8_t* brow = smem + C::kVOffset + warp * (kRows / C::kWarps) * C::kVRowBytes + lane * 4;
#pragma unroll 1
        for (int i0 = 0; i0 < kRows / C::kWarps; i0 += 8) {
            float cv[8][8];                       // eight centroids in flight per lane (the loop's registers are free now)
#pragma unroll
            for (int i = 0; i < 8; ++i) load_centroid<8>(cg + (i0 + i) * 8, cv[i], cb_aligned32 != 0);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float b0 = (float)*reinterpret_cast<const uint32_t*>(brow + (i0 + i) * C::kVRowBytes);
                const float b1 = (float)*reinterpret_cast<const uint32_t*>(brow + (i0 + i) * C::kVRowBytes + 128);
                l0 += b0;
                l1 += b1;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    acc0[c] = fmaf(b0, cv[i][c], acc0[c]);
                    acc1[c] = fmaf(b1, cv[i][c], acc1[c]);
                }
            }
        }
        float* red = reinterpret_cast<float*>(smem);                      // [warp][18][32]
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            red[(warp * 18 + c) * 32 + lane] = acc0[c];
            red[(warp * 18 + 8 + c) * 32 + lane] = acc1[c];
        }
        red[(warp * 18 + 16) * 32 + lane] = l0;
        red[(warp * 18 + 17) * 32 + lane] = l1;
        __syncthreads();
        // 18 x 32 sums of eight terms: slot k < 16 of lane (hb', g) is channel g*8 + k%8 of head 2 (k/8) + hb';
        // slots 16, 17 of the lanes with g = 0 are the normalisers (sum of the bins of group 0)
        for (int o = threadIdx.x; o < 18 * 32; o += C::kThreads) {
            const int slot = o >> 5, ln = o & 31;
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < C::kWarps; ++w) v += red[(w * 18 + slot) * 32 + ln];
            const int hb2 = ln >> 4, g2 = ln & 15;
            if (slot < 16) {
                const int h = 2 * (slot >> 3) + hb2;
                part_base[(int64_t)h * n_parts * stride + 2 + g2 * 8 + (slot & 7)] = v;
            } else if (g2 == 0) {
                const int h = 2 * (slot - 16) + hb2;
                part_base[(int64_t)h * n_parts * stride + 0] = (float)ctl->head[h].e_cur + ctl->offset[h];   // reference exponent (log2 domain)
                part_base[(int64_t)h * n_parts * stride + 1] = v;                                            // normaliser, in the same unit
            }
        }
        // One part per item (out != null only then): the partial is the whole sum, so the CTA normalises it itself
        // and no merge launch follows.
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
}

}  // namespace

bool decode_pair_supported(const Shape& sh)
{
    return sh.head_dim == 128 && sh.b == 8 && sh.G == 16 && sh.R % PairCfg::kHeads == 0 &&
           sh.max_tokens <= ((int64_t)1 << 30);
}

// Launch plan.  Two CTAs share an SM.  The table build and the bins x centroids product are paid
// once per CTA, so a CTA takes its whole context (up to 65536 tokens) unless the grid would leave
// CTA slots idle.  When every context fits one CTA, the items beyond the last full wave of CTAs may be
// spread over k <= 4 CTAs each (see below).
DecodePlan decode_pair_plan(const Shape& sh)
{
    using C = PairCfg;
    DecodePlan pl;
    const int64_t items = sh.n_seq * (sh.n_q_heads / C::kHeads);
    const int64_t slots = 2 * (int64_t)device_sm_count();
    const int64_t round = C::kRoundTokens;
    int64_t chunk = (sh.max_tokens + round - 1) / round * round;
    if (chunk > 65536) chunk = 65536;
    // (split only until every SM has one and a half CTAs: a CTA that has an SM to itself still runs at
    // more than half of the SM's rate, and every split pays another table build)
    while (chunk > 2048 && 4 * items * ((sh.max_tokens + chunk - 1) / chunk) < 3 * slots)
        chunk = (chunk / 2 + round - 1) / round * round;
    pl.chunk = (int)chunk;
    pl.n_parts = (int)((sh.max_tokens + chunk - 1) / chunk);
    pl.tail_first = -1;
    pl.grid = (unsigned)(items * pl.n_parts);
    // Last wave.  Splitting an item over k CTAs shortens it, but every CTA pays the table build and
    // the bins x centroids product, which cost about as much as seven loop iterations (measured), and
    // a CTA that has an SM to itself runs at about 1 / 0.62 of the rate of two that share one.  Take
    // the k <= 4 with the smallest estimated duration of the wave.
    const int64_t rest = items % slots;
    if (pl.n_parts == 1 && items > slots && rest > 0) {
        const double iters = (double)chunk / (double)round, fixed = 7.4;
        int best_k = 1;
        double best = 1e30;
        for (int k = 1; k <= 4; ++k) {
            if (k > 1 && chunk / k < 2048) break;
            const int64_t ctas = rest * k;
            const double waves = (double)((ctas + slots - 1) / slots);
            const double cost = waves * (fixed + iters / k) / (fixed + iters) * (2 * ctas <= slots ? 0.62 : 1.0);
            if (cost < best - 1e-9) { best = cost; best_k = k; }
        }
        if (best_k > 1) {
            const int64_t part_chunk = ((chunk + best_k - 1) / best_k + round - 1) / round * round;
            pl.chunk = (int)part_chunk;
            pl.n_parts = (int)((sh.max_tokens + part_chunk - 1) / part_chunk);
            pl.tail_first = (int)(items - rest);
            pl.grid = (unsigned)(pl.tail_first + rest * pl.n_parts);
        }
    }
    return pl;
}

cudaError_t launch_decode_pair(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                               const int32_t* seq_lens, float scale, const Shape& sh, const DecodePlan& pl,
                               float* partials, cudaStream_t st, const AppendArgs& app, float* out)
{
    using C = PairCfg;
    const cudaError_t attr = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_pair_kernel), C::kSmemBytes, 0);
    if (attr != cudaSuccess) return attr;
    const int aligned = ((reinterpret_cast<uintptr_t>(kcb) | reinterpret_cast<uintptr_t>(vcb)) & 31u) == 0 ? 1 : 0;
    decode_pair_kernel<<<pl.grid, C::kThreads, C::kSmemBytes, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, pl.chunk,
                                                                    pl.n_parts, pl.tail_first, aligned, partials, app,
                                                                    pl.n_parts == 1 ? out : nullptr);
    return cudaGetLastError();
}

}  // namespace cq
