// Tuned decode attention over codes of keys that were quantised BEFORE the rotary position embedding
// (last sentence of Section 3.2), for head_dim 128, b = 8, c in {4, 8} and the pairing (i, i + 64).
//
// The key of Eq. 1 is the reconstruction rotated by its position, K_a = k_a cos - k_b sin,
// K_b = k_b cos + k_a sin for the channel pair (a, b) = (i, i + 64), so a score is a dot product of
// the query with a dequantised, rotated key: there is no table of per-code score terms.  What the
// kernel does instead:
//   - A CTA serves up to 8 query heads of one KV head (what the bins leave room for) over a range of
//     the context; the KV head's key centroids sit in shared memory as fp16 (64 KiB), code-major
//     ([code][group][channel]), so that the 32 lanes of a gather - each in its own group's columns -
//     touch 32 different banks whatever the codes are.  The bins are code-major for the same reason.
//   - Lane l of a warp owns the pairs i = 2l, 2l + 1.  For a batch of 32 / heads consecutive tokens it
//     gathers the two half2 words of its channels per token, rotates them and multiplies by its slice
//     of every head's query: 32 partial scores per lane, which a five-stage exchange between the
//     lanes sums so that lane (head, token) ends up with that score.
//   - The cosines and sines of a batch are read from the tables once, for its first token; the next
//     tokens' values follow by the angle-addition rule with the step (cos, sin) taken from the
//     tables' first two rows.  At the end of the batch the result is compared with the table row of
//     the token after the batch; if it differs (tables that are not of the form cos / sin of
//     position x frequency + phase) the batch is done again with every row read from the tables, and
//     so are the warp's later batches.
//   - Scores of a chunk of the range are kept in shared memory; the chunk's largest score per head
//     fixes the reference exponent (the bins are rescaled when it grows), then the weights
//     2^(score - reference) are added to fp32 bins per (head, group, value code), lane = group, and
//     bins x value centroids closes the partial.  Partials and their merge are those of the other
//     decode kernels.
#include "cq_common.cuh"
#include "cq_decode_util.cuh"
#include <type_traits>

namespace cq {

namespace {

constexpr int kRtThreads = 512;
constexpr int kRtWarps = kRtThreads / 32;
constexpr int kRtScoreBytes = 32 * 1024;

struct RtCtl {
    float m_run[8];                    // per head: reference exponent of the bins (log2 domain)
    float factor[8];                   // per head: 2^(old reference - new reference) of the current chunk
    float warp_max[kRtWarps][8];       // per warp and head: largest score of the current chunk
    float l_part[kRtWarps][8];         // per warp and head: sum of weights (final reduction)
};

template <int kC, int kHeads>
struct RtCfg {
    static constexpr int G = 128 / kC;
    static constexpr int kT = 32 / kHeads;                        // tokens of a warp's batch
    static constexpr int kChunk = kRtScoreBytes / 4 / kHeads;     // tokens whose scores are kept at a time
    static constexpr int kBookOff = 0;                            // fp16 [256][G][kC]
    static constexpr int kBinsOff = 128 * 256 * 2;                // fp32 [kHeads][256][G]
    static constexpr int kScoreOff = kBinsOff + kHeads * G * 256 * 4;      // fp32 [kHeads][kChunk]
    static constexpr int kCtlOff = kScoreOff + kRtScoreBytes;
    static constexpr int kSmemBytes = kCtlOff + 2048;
    static_assert(sizeof(RtCtl) <= 2048, "control block");
    static_assert(kSmemBytes <= 227 * 1024, "shared memory");
    static_assert(kChunk % 32 == 0 && kT >= 4, "batches of whole words");
};

// byte j of a run of code bytes held in 32-bit words (little endian)
template <int kWords>
__device__ __forceinline__ uint32_t rt_code(const uint32_t (&w)[kWords], int j)
{
    return (w[j >> 2] >> (8 * (j & 3))) & 0xffu;
}

template <int kC, int kHeads>
__global__ void __launch_bounds__(kRtThreads, 1)
decode_rope_tuned_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                         const float* __restrict__ kcb, const float* __restrict__ vcb, const int32_t* __restrict__ seq_lens,
                         const float* __restrict__ rope_cos, const float* __restrict__ rope_sin, float scale_log2e, Shape sh,
                         int n_splits, int split_tokens, float* __restrict__ partials)
{
    using C = RtCfg<kC, kHeads>;
    constexpr int G = C::G, kT = C::kT, kWords = kT / 4;
    extern __shared__ __align__(16) unsigned char rt_smem[];
    const uint32_t* book = reinterpret_cast<const uint32_t*>(rt_smem + C::kBookOff);
    float* bins = reinterpret_cast<float*>(rt_smem + C::kBinsOff);
    float* scores = reinterpret_cast<float*>(rt_smem + C::kScoreOff);
    RtCtl* ctl = reinterpret_cast<RtCtl*>(rt_smem + C::kCtlOff);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_hgroups = sh.n_q_heads / kHeads;
    const int split = blockIdx.x % n_splits;
    const int hg = (blockIdx.x / n_splits) % n_hgroups;
    const int64_t s = seq_by_rank(seq_lens, (int)sh.n_seq, sh.max_tokens, (int)(blockIdx.x / (n_splits * n_hgroups)));   // longest first
    const int hq0 = hg * kHeads, hkv = hq0 / sh.R;
    const int stride = partial_stride(128);

    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int64_t t_begin = (int64_t)split * split_tokens;
    const int64_t t_end = t_begin + split_tokens < n ? t_begin + split_tokens : n;
    float* part0 = partials + ((s * sh.n_q_heads + hq0) * n_splits + split) * (int64_t)stride;      // head h: + h * n_splits * stride
    if (t_end <= t_begin) {          // empty range: neutral element of the merge
        for (int i = threadIdx.x; i < kHeads * stride; i += kRtThreads) {
            const int h = i / stride, d = i % stride;
            part0[(int64_t)h * n_splits * stride + d] = d == 0 ? -INFINITY : 0.f;
        }
        return;
    }

    // ------------------------------------------------------------------ set-up
    // key centroids of the KV head as fp16, bins at zero
    {
        const float4* src = reinterpret_cast<const float4*>(kcb + (int64_t)hkv * 128 * 256);
        uint2* dst = reinterpret_cast<uint2*>(rt_smem + C::kBookOff);
        for (int i = threadIdx.x; i < 128 * 256 / 4; i += kRtThreads) {
            // four channels of centroid (g, j): piece i of the global [g][j][c] order goes to the [j][g][c] order
            const int per = kC / 4, g = i / (256 * per), j = (i / per) % 256, w4 = i % per;
            const float4 v = ldg_f4(reinterpret_cast<const float*>(src + i));
            const __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
            dst[(j * G + g) * per + w4] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
        }
        for (int i = threadIdx.x; i < kHeads * G * 256 / 4; i += kRtThreads)
            reinterpret_cast<float4*>(bins)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (threadIdx.x < 8) ctl->m_run[threadIdx.x] = -INFINITY;
    }
    // this lane's channels: a = 2 lane, 2 lane + 1 and b = a + 64; its slice of every head's query
    float qa[kHeads][2], qb[kHeads][2];
#pragma unroll
    for (int h = 0; h < kHeads; ++h) {
        const __half* qh = q + (s * sh.n_q_heads + hq0 + h) * 128;
        qa[h][0] = __half2float(qh[2 * lane]) * scale_log2e;
        qa[h][1] = __half2float(qh[2 * lane + 1]) * scale_log2e;
        qb[h][0] = __half2float(qh[64 + 2 * lane]) * scale_log2e;
        qb[h][1] = __half2float(qh[64 + 2 * lane + 1]) * scale_log2e;
    }
    // rotation from one position to the next, from the tables' first two rows: row1 x conj(row0) / |row0|^2
    float2 st_re = make_float2(1.f, 1.f), st_im = make_float2(0.f, 0.f);
    bool exact = sh.max_tokens < 2;              // true: every token's row is read from the tables
    if (!exact) {
        const float2 c0 = *reinterpret_cast<const float2*>(rope_cos + 2 * lane), s0 = *reinterpret_cast<const float2*>(rope_sin + 2 * lane);
        const float2 c1 = *reinterpret_cast<const float2*>(rope_cos + 64 + 2 * lane), s1 = *reinterpret_cast<const float2*>(rope_sin + 64 + 2 * lane);
        const float nx = c0.x * c0.x + s0.x * s0.x, ny = c0.y * c0.y + s0.y * s0.y;
        if (!(nx > 1e-12f) || !(ny > 1e-12f)) exact = true;
        st_re.x = (c1.x * c0.x + s1.x * s0.x) / nx;
        st_im.x = (s1.x * c0.x - c1.x * s0.x) / nx;
        st_re.y = (c1.y * c0.y + s1.y * s0.y) / ny;
        st_im.y = (s1.y * c0.y - c1.y * s0.y) / ny;
        exact = __any_sync(0xffffffffu, exact);
    }
    // words of the lane's two channels inside a centroid, and its two groups
    const int gA = (2 * lane) / kC, gB = gA + G / 2;
    // word of the lane's channels a in the centroid row of a code: code * (64 words) + colA; channels b: + 32 words
    const uint32_t colA = (uint32_t)(gA * kC + (2 * lane) % kC) / 2u, colB = colA + 32u;
    static_assert(128 / 2 == 64, "64 words of fp16 pairs per code");
    const uint8_t* kseq = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint8_t* vseq = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    float l_thr[kHeads];
#pragma unroll
    for (int h = 0; h < kHeads; ++h) l_thr[h] = 0.f;
    __syncthreads();

    for (int64_t chunk_begin = t_begin; chunk_begin < t_end; chunk_begin += C::kChunk) {
        const int chunk_len = (int)(t_end - chunk_begin < C::kChunk ? t_end - chunk_begin : C::kChunk);

        // -------------------------------------------------------------- scores of the chunk
        float lane_max = -INFINITY;                  // over the scores of this lane's head
        // a batch's key codes of the lane's two groups and the table rows of its first token
        auto load_batch = [&](int64_t t0, uint32_t (&ca)[kWords], uint32_t (&cbw)[kWords], float2& cs0, float2& sn0) {
            const uint8_t* pa = kseq + (t0 / kTokenBlock) * sh.block_bytes + (t0 % kTokenBlock);
            if (kT == 32) {
                const bool two = t0 + 16 < t_end;
                const uint4 a0 = *reinterpret_cast<const uint4*>(pa + gA * kTokenBlock), b0w = *reinterpret_cast<const uint4*>(pa + gB * kTokenBlock);
                const uint4 a1 = two ? *reinterpret_cast<const uint4*>(pa + sh.block_bytes + gA * kTokenBlock) : make_uint4(0u, 0u, 0u, 0u);
                const uint4 b1 = two ? *reinterpret_cast<const uint4*>(pa + sh.block_bytes + gB * kTokenBlock) : make_uint4(0u, 0u, 0u, 0u);
                ca[0] = a0.x; ca[1 % kWords] = a0.y; ca[2 % kWords] = a0.z; ca[3 % kWords] = a0.w;
                ca[4 % kWords] = a1.x; ca[5 % kWords] = a1.y; ca[6 % kWords] = a1.z; ca[7 % kWords] = a1.w;
                cbw[0] = b0w.x; cbw[1 % kWords] = b0w.y; cbw[2 % kWords] = b0w.z; cbw[3 % kWords] = b0w.w;
                cbw[4 % kWords] = b1.x; cbw[5 % kWords] = b1.y; cbw[6 % kWords] = b1.z; cbw[7 % kWords] = b1.w;
            } else if (kT == 16) {
                const uint4 a0 = *reinterpret_cast<const uint4*>(pa + gA * kTokenBlock), b0w = *reinterpret_cast<const uint4*>(pa + gB * kTokenBlock);
                ca[0] = a0.x; ca[1 % kWords] = a0.y; ca[2 % kWords] = a0.z; ca[3 % kWords] = a0.w;
                cbw[0] = b0w.x; cbw[1 % kWords] = b0w.y; cbw[2 % kWords] = b0w.z; cbw[3 % kWords] = b0w.w;
            } else if (kT == 8) {
                const uint2 a0 = *reinterpret_cast<const uint2*>(pa + gA * kTokenBlock), b0w = *reinterpret_cast<const uint2*>(pa + gB * kTokenBlock);
                ca[0] = a0.x; ca[1 % kWords] = a0.y;
                cbw[0] = b0w.x; cbw[1 % kWords] = b0w.y;
            } else {
                ca[0] = *reinterpret_cast<const uint32_t*>(pa + gA * kTokenBlock);
                cbw[0] = *reinterpret_cast<const uint32_t*>(pa + gB * kTokenBlock);
            }
            cs0 = *reinterpret_cast<const float2*>(rope_cos + t0 * 64 + 2 * lane);
            sn0 = *reinterpret_cast<const float2*>(rope_sin + t0 * 64 + 2 * lane);
        };
        uint32_t ca[kWords], cbw[kWords];
        float2 cs0 = make_float2(1.f, 1.f), sn0 = make_float2(0.f, 0.f);
        if (warp * kT < chunk_len) load_batch(chunk_begin + warp * kT, ca, cbw, cs0, sn0);
        for (int b0 = warp * kT; b0 < chunk_len; b0 += kRtWarps * kT) {
            const int64_t t0 = chunk_begin + b0;
            float p[32];
            // The partial scores of the batch; from_tables: every token's row is read from the tables, else the rows
            // after the first follow by the step rotation.  Returns false when the stepped rows leave the tables.
            // With one head per CTA the query is rotated instead of the key (by the opposite angle): the rotated
            // query u = q_a cos + q_b sin, v = q_b cos - q_a sin steps like the angle does, and the score term of a
            // pair is k_a u + k_b v.
            auto batch = [&](auto from_tables) -> bool {
                constexpr bool kFromTables = decltype(from_tables)::value;
                float2 cs = cs0, sn = sn0;
                float2 u = make_float2(0.f, 0.f), v = make_float2(0.f, 0.f);
                if (kHeads == 1) {
                    u = make_float2(fmaf(qa[0][0], cs.x, qb[0][0] * sn.x), fmaf(qa[0][1], cs.y, qb[0][1] * sn.y));
                    v = make_float2(fmaf(qb[0][0], cs.x, -qa[0][0] * sn.x), fmaf(qb[0][1], cs.y, -qa[0][1] * sn.y));
                }
#pragma unroll
                for (int j = 0; j < kT; ++j) {
                    const uint32_t wa = book[rt_code<kWords>(ca, j) * 64u + colA];
                    const uint32_t wb = book[rt_code<kWords>(cbw, j) * 64u + colB];
                    const float2 ka = __half22float2(*reinterpret_cast<const __half2*>(&wa));
                    const float2 kb = __half22float2(*reinterpret_cast<const __half2*>(&wb));
                    if (kHeads == 1) {
                        p[j] = fmaf(ka.x, u.x, fmaf(kb.x, v.x, fmaf(ka.y, u.y, kb.y * v.y)));
                    } else {
                        // the rotated key of the lane's four channels
                        const float ra0 = ka.x * cs.x - kb.x * sn.x, rb0 = kb.x * cs.x + ka.x * sn.x;
                        const float ra1 = ka.y * cs.y - kb.y * sn.y, rb1 = kb.y * cs.y + ka.y * sn.y;
#pragma unroll
                        for (int h = 0; h < kHeads; ++h)
                            p[h * kT + j] = fmaf(qa[h][0], ra0, fmaf(qb[h][0], rb0, fmaf(qa[h][1], ra1, qb[h][1] * rb1)));
                    }
                    // the next position
                    if (kFromTables) {
                        if (j + 1 < kT) {
                            const int64_t tn = t0 + j + 1 < sh.max_tokens ? t0 + j + 1 : t0 + j;
                            cs = *reinterpret_cast<const float2*>(rope_cos + tn * 64 + 2 * lane);
                            sn = *reinterpret_cast<const float2*>(rope_sin + tn * 64 + 2 * lane);
                            if (kHeads == 1) {
                                u = make_float2(fmaf(qa[0][0], cs.x, qb[0][0] * sn.x), fmaf(qa[0][1], cs.y, qb[0][1] * sn.y));
                                v = make_float2(fmaf(qb[0][0], cs.x, -qa[0][0] * sn.x), fmaf(qb[0][1], cs.y, -qa[0][1] * sn.y));
                            }
                        }
                    } else if (kHeads == 1) {
                        const float ux = fmaf(u.x, st_re.x, v.x * st_im.x), vx = fmaf(v.x, st_re.x, -u.x * st_im.x);
                        const float uy = fmaf(u.y, st_re.y, v.y * st_im.y), vy = fmaf(v.y, st_re.y, -u.y * st_im.y);
                        u = make_float2(ux, uy);
                        v = make_float2(vx, vy);
                    } else {
                        const float cx = cs.x * st_re.x - sn.x * st_im.x, sx = sn.x * st_re.x + cs.x * st_im.x;
                        const float cy = cs.y * st_re.y - sn.y * st_im.y, sy = sn.y * st_re.y + cs.y * st_im.y;
                        cs = make_float2(cx, cy);
                        sn = make_float2(sx, sy);
                    }
                }
                if (kFromTables) return true;
                // what was stepped to is the prediction for position t0 + kT: it must be what the tables hold there
                bool off = false;
                if (t0 + kT < sh.max_tokens) {
                    const float2 ct = *reinterpret_cast<const float2*>(rope_cos + (t0 + kT) * 64 + 2 * lane);
                    const float2 stt = *reinterpret_cast<const float2*>(rope_sin + (t0 + kT) * 64 + 2 * lane);
                    const float tol = 2e-5f;
                    if (kHeads == 1) {
                        const float ux = fmaf(qa[0][0], ct.x, qb[0][0] * stt.x), uy = fmaf(qa[0][1], ct.y, qb[0][1] * stt.y);
                        const float vx = fmaf(qb[0][0], ct.x, -qa[0][0] * stt.x), vy = fmaf(qb[0][1], ct.y, -qa[0][1] * stt.y);
                        const float bx = tol * (fabsf(qa[0][0]) + fabsf(qb[0][0])) * (1.f + fabsf(ct.x) + fabsf(stt.x));
                        const float by = tol * (fabsf(qa[0][1]) + fabsf(qb[0][1])) * (1.f + fabsf(ct.y) + fabsf(stt.y));
                        off = !(fabsf(ux - u.x) <= bx) || !(fabsf(vx - v.x) <= bx) || !(fabsf(uy - u.y) <= by) || !(fabsf(vy - v.y) <= by);
                    } else {
                        off = !(fabsf(ct.x - cs.x) <= tol * (1.f + fabsf(ct.x))) || !(fabsf(ct.y - cs.y) <= tol * (1.f + fabsf(ct.y))) ||
                              !(fabsf(stt.x - sn.x) <= tol * (1.f + fabsf(stt.x))) || !(fabsf(stt.y - sn.y) <= tol * (1.f + fabsf(stt.y)));
                    }
                }
                return !__any_sync(0xffffffffu, off);
            };
            if (exact || !batch(std::false_type())) {
                exact = true;                            // this batch, and every later one of the warp, from the tables
                batch(std::true_type());
            }
            // the next batch's words travel during the exchange
            {
                const int nb = b0 + kRtWarps * kT;
                if (nb < chunk_len) load_batch(chunk_begin + nb, ca, cbw, cs0, sn0);
            }
            // Sum over the lanes: after the stage with offset o a lane keeps the half of its slots whose index has
            // bit o like its own lane number; after five stages lane L holds slot L = (head L / kT, token L % kT).
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                const bool upper = (lane & o) != 0;
#pragma unroll
                for (int i = 0; i < o; ++i) {
                    const float send = upper ? p[i] : p[i + o];
                    const float keep = upper ? p[i + o] : p[i];
                    p[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
            }
            const int h = lane / kT, j = lane % kT;
            const bool valid = t0 + j < t_end;
            const float sc = valid ? p[0] : -INFINITY;
            scores[h * C::kChunk + b0 + j] = sc;
            lane_max = fmaxf(lane_max, sc);
        }
        // largest score per head: over the lanes of a head, then over the warps
#pragma unroll
        for (int o = 1; o < kT; o <<= 1) lane_max = fmaxf(lane_max, __shfl_xor_sync(0xffffffffu, lane_max, o));
        if (lane % kT == 0) ctl->warp_max[warp][lane / kT] = lane_max;
        __syncthreads();
        if (threadIdx.x < kHeads) {
            float m = ctl->m_run[threadIdx.x];
            const float old = m;
            for (int w = 0; w < kRtWarps; ++w) m = fmaxf(m, ctl->warp_max[w][threadIdx.x]);
            ctl->factor[threadIdx.x] = old == m ? 1.f : exp2f(old - m);      // 0 when there was no reference yet
            ctl->m_run[threadIdx.x] = m;
        }
        __syncthreads();
        // the bins follow the reference; weights of the chunk
#pragma unroll
        for (int h = 0; h < kHeads; ++h) {
            const float f = ctl->factor[h], m = ctl->m_run[h];
            if (f != 1.f) {
                for (int i = threadIdx.x; i < G * 256; i += kRtThreads) bins[h * G * 256 + i] *= f;
                l_thr[h] *= f;
            }
            for (int i = threadIdx.x; i < chunk_len; i += kRtThreads) {
                const float w = exp2f(scores[h * C::kChunk + i] - m);
                scores[h * C::kChunk + i] = w;
                l_thr[h] += w;
            }
        }
        __syncthreads();
        // -------------------------------------------------------------- value side: weights into the bins
        // a warp per block of 16 tokens; lane = (group, run of tokens of the block)
        {
            constexpr int kLanesPerGroup = 32 / G;                  // 2 for c = 8, 1 for c = 4
            constexpr int kRun = 16 / kLanesPerGroup;               // tokens of the block per lane
            const int g = lane % G, run = lane / G;
            const int n_blk = (chunk_len + kTokenBlock - 1) / kTokenBlock;
            for (int blk = warp; blk < n_blk; blk += kRtWarps) {
                const uint8_t* pv = vseq + ((chunk_begin / kTokenBlock) + blk) * sh.block_bytes + g * kTokenBlock + run * kRun;
                uint32_t cw[kRun / 4];
                if (kRun == 16) {
                    const uint4 v4 = *reinterpret_cast<const uint4*>(pv);
                    cw[0] = v4.x; cw[1 % (kRun / 4)] = v4.y; cw[2 % (kRun / 4)] = v4.z; cw[3 % (kRun / 4)] = v4.w;
                } else {
                    const uint2 v2 = *reinterpret_cast<const uint2*>(pv);
                    cw[0] = v2.x; cw[1 % (kRun / 4)] = v2.y;
                }
#pragma unroll
                for (int k = 0; k < kRun; ++k) {
                    const int tl = blk * kTokenBlock + run * kRun + k;
                    const uint32_t code = rt_code<kRun / 4>(cw, k);
#pragma unroll
                    for (int h = 0; h < kHeads; ++h) {
                        const float w = tl < chunk_len ? scores[h * C::kChunk + tl] : 0.f;      // (adding zero changes nothing)
                        atomicAdd(&bins[(h * 256 + code) * G + g], w);
                    }
                }
            }
        }
        __syncthreads();
    }

    // ------------------------------------------------------------------ partial: reference, normaliser, bins x value centroids
#pragma unroll
    for (int h = 0; h < kHeads; ++h) {
        float l = l_thr[h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        if (lane == 0) ctl->l_part[warp][h] = l;
    }
    __syncthreads();
    if (threadIdx.x < kHeads) {
        float l = 0.f;
        for (int w = 0; w < kRtWarps; ++w) l += ctl->l_part[w][threadIdx.x];
        part0[(int64_t)threadIdx.x * n_splits * stride + 0] = ctl->m_run[threadIdx.x];
        part0[(int64_t)threadIdx.x * n_splits * stride + 1] = l;
    }
    // bins x value centroids: lane = group (two lanes per group for c = 8, one for the even and one for the odd codes),
    // a warp per 16 codes, the warps' sums added through shared memory (the score area is free now)
    {
        constexpr int kLanesPerGroup = 32 / G;
        const int g = lane % G, sub = lane / G;
        float* red = scores;                                     // [warps][128]
#pragma unroll 1
        for (int h = 0; h < kHeads; ++h) {
            float acc[kC];
#pragma unroll
            for (int k = 0; k < kC; ++k) acc[k] = 0.f;
#pragma unroll 4
            for (int i = 0; i < 16 / kLanesPerGroup; ++i) {
                const int j = warp * 16 + kLanesPerGroup * i + sub;
                const float w = bins[(h * 256 + j) * G + g];
                float cv[kC];
                load_centroid<kC>(vcb + (((int64_t)hkv * G + g) * 256 + j) * kC, cv, false);
#pragma unroll
                for (int k = 0; k < kC; ++k) acc[k] = fmaf(w, cv[k], acc[k]);
            }
            if (kLanesPerGroup == 2) {
#pragma unroll
                for (int k = 0; k < kC; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], 16);
            }
            if (sub == 0) {
#pragma unroll
                for (int k = 0; k < kC; ++k) red[warp * 128 + g * kC + k] = acc[k];
            }
            __syncthreads();
            if (threadIdx.x < 128) {
                float v = 0.f;
#pragma unroll
                for (int w = 0; w < kRtWarps; ++w) v += red[w * 128 + threadIdx.x];
                part0[(int64_t)h * n_splits * stride + 2 + threadIdx.x] = v;
            }
            __syncthreads();
        }
    }
}

template <int kC, int kHeads>
cudaError_t launch_rt(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                      const int32_t* seq_lens, const float* rope_cos, const float* rope_sin, float scale, const Shape& sh,
                      int n_splits, int split_tokens, float* partials, cudaStream_t st)
{
    using C = RtCfg<kC, kHeads>;
    constexpr int kSlot = 48 + (kC == 8 ? 0 : 4) + (kHeads == 1 ? 0 : kHeads == 2 ? 1 : kHeads == 4 ? 2 : 3);    // 48 ... 55
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(decode_rope_tuned_kernel<kC, kHeads>), C::kSmemBytes, kSlot);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(sh.n_seq * (sh.n_q_heads / kHeads) * n_splits);
    decode_rope_tuned_kernel<kC, kHeads><<<grid, kRtThreads, C::kSmemBytes, st>>>(q, kc, vc, kcb, vcb, seq_lens, rope_cos, rope_sin,
                                                                                  scale * kLog2e, sh, n_splits, split_tokens, partials);
    return cudaGetLastError();
}

int rope_heads_per_cta(const Shape& sh)
{
    const int most = sh.c == 8 ? 8 : 4;              // what the bins leave room for
    int h = 1;
    while (h * 2 <= most && sh.R % (h * 2) == 0) h *= 2;
    return h;
}

}  // namespace

bool decode_rope_tuned_supported(const Shape& sh, int pairing)
{
    return pairing == 0 && sh.head_dim == 128 && sh.b == 8 && (sh.c == 4 || sh.c == 8);
}

cudaError_t launch_decode_rope_tuned(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb,
                                     const float* vcb, const int32_t* seq_lens, const float* rope_cos, const float* rope_sin,
                                     float scale, const Shape& sh, float* out, float* partials, cudaStream_t st)
{
    const int heads = rope_heads_per_cta(sh);
    // ranges of the context: enough CTAs for two per SM... one CTA fills an SM, so two waves; never more partial slots
    // than the workspace holds (those of decode_generic_splits), ranges of whole 256 tokens
    const int64_t items = sh.n_seq * (sh.n_q_heads / heads);
    int64_t want = (2 * (int64_t)device_sm_count() + items - 1) / items;
    const int64_t cap = (sh.max_tokens + 1023) / 1024;
    if (want > cap) want = cap;
    const int most = decode_generic_splits(sh);
    if (want > most) want = most;
    if (want < 1) want = 1;
    int64_t split_tokens = (sh.max_tokens + want - 1) / want;
    split_tokens = (split_tokens + 255) / 256 * 256;
    const int n_splits = (int)((sh.max_tokens + split_tokens - 1) / split_tokens);
    cudaError_t e = cudaErrorNotSupported;
#define CQ_RT(C_, H_) e = launch_rt<C_, H_>(q, kc, vc, kcb, vcb, seq_lens, rope_cos, rope_sin, scale, sh, n_splits, (int)split_tokens, partials, st)
    if (sh.c == 8) {
        switch (heads) { case 1: CQ_RT(8, 1); break; case 2: CQ_RT(8, 2); break; case 4: CQ_RT(8, 4); break; case 8: CQ_RT(8, 8); break; default: break; }
    } else {
        switch (heads) { case 1: CQ_RT(4, 1); break; case 2: CQ_RT(4, 2); break; case 4: CQ_RT(4, 4); break; default: break; }
    }
#undef CQ_RT
    if (e != cudaSuccess) return e;
    return launch_merge(partials, n_splits, sh, out, st);
}

}  // namespace cq
