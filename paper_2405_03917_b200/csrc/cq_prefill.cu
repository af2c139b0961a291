// Causal attention of a run of new tokens over the CQ-coded cache (a prompt, or a chunk of one).
//
// Section 2.1 of the paper: Eq. 1 gives the output of "the current token" from the keys and values
// of all tokens up to and including it; here it is applied to each of the n_q newest cached tokens,
// with K and V replaced by their CQ reconstructions (Section 3.2).  Query i of sequence s sits at
// position seq_lens[s] - n_q + i and attends the cached tokens 0 ... that position.
//
// With many queries per cached token the per-query lookup tables of the decode kernels no longer
// pay (one table per query); the codes are turned back into vectors instead and the two
// contractions run on the tensor cores:
//   prefill_mma_kernel (head_dim 128, one byte per code, c = 2, 4 or 8): one CTA per (sequence,
//     KV head, tile of 128 (query, head of the KV head's group) rows).  Both codebooks are kept
//     in shared memory as fp16, code-major, so that the lanes of a gather (one group each) meet
//     in no bank whatever the codes are; per tile of 64 cached tokens the K and V codes are gathered into
//     fp16 tiles, S = Q Khat^T and O += P Vhat are m16n8k16 MMAs with fp32 accumulators, and the
//     softmax is the usual running-maximum form in the log2 domain.  Four producer warps do the
//     gathering into two tile buffers while eight warps (16 rows each) multiply; named barriers
//     hand a buffer back and forth, and the producers give most of their registers to the others.
//     The multiplying warps hold their query fragments in registers; a tile wholly below the
//     causal limit of a warp's rows skips the mask and folds the scale into the exponent.
//   prefill_generic_kernel: any supported shape, one CTA per (sequence, query, head), plain loops.
#include "cq_common.cuh"

namespace cq {

namespace {

// ------------------------------------------------------------------------------------------
// generic kernel
// ------------------------------------------------------------------------------------------
constexpr int kGenWarps = 4;
constexpr int kMaxLaneCh = 8;          // head_dim <= 256: up to 8 channels per lane

__global__ void __launch_bounds__(kGenWarps * 32)
prefill_generic_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                       const float* __restrict__ kcb, const float* __restrict__ vcb,
                       const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int n_q, float* __restrict__ out)
{
    __shared__ float red_m[kGenWarps], red_l[kGenWarps];
    __shared__ float red_acc[kGenWarps][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hq = blockIdx.x % sh.n_q_heads;
    const int qi = (blockIdx.x / sh.n_q_heads) % n_q;
    const int64_t s = blockIdx.x / ((int64_t)sh.n_q_heads * n_q);
    const int hkv = hq / sh.R;
    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int64_t n_att = n - n_q + qi + 1;                              // tokens 0 .. position of the query
    const int64_t row = (s * n_q + qi) * sh.n_q_heads + hq;
    float* o = out + row * sh.head_dim;
    if (n_att <= 0) {
        for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) o[d] = 0.f;
        return;
    }
    float qd[kMaxLaneCh], acc[kMaxLaneCh];
#pragma unroll
    for (int j = 0; j < kMaxLaneCh; ++j) {
        const int d = lane + 32 * j;
        qd[j] = d < sh.head_dim ? __half2float(q[row * sh.head_dim + d]) * scale_log2e : 0.f;
        acc[j] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    for (int64_t t = warp; t < n_att; t += kGenWarps) {
        const uint8_t* kblk = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, t / kTokenBlock, 0);
        const uint8_t* vblk = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, t / kTokenBlock, 0);
        const int k = (int)(t % kTokenBlock);
        float dot = 0.f, vv[kMaxLaneCh];
#pragma unroll
        for (int j = 0; j < kMaxLaneCh; ++j) {
            const int d = lane + 32 * j;
            vv[j] = 0.f;
            if (d < sh.head_dim) {
                const int g = d / sh.c, i = d % sh.c;
                dot = fmaf(qd[j], kcb[(((int64_t)hkv * sh.G + g) * sh.K + read_code(kblk, sh, g, k)) * sh.c + i], dot);
                vv[j] = vcb[(((int64_t)hkv * sh.G + g) * sh.K + read_code(vblk, sh, g, k)) * sh.c + i];
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        const float m_new = fmaxf(m, dot);
        const float corr = exp2f(m - m_new), p = exp2f(dot - m_new);
        l = l * corr + p;
#pragma unroll
        for (int j = 0; j < kMaxLaneCh; ++j) acc[j] = fmaf(p, vv[j], acc[j] * corr);
        m = m_new;
    }
    if (lane == 0) { red_m[warp] = m; red_l[warp] = l; }
#pragma unroll
    for (int j = 0; j < kMaxLaneCh; ++j) red_acc[warp][lane + 32 * j] = acc[j];
    __syncthreads();
    float M = -INFINITY;
    for (int w = 0; w < kGenWarps; ++w) M = fmaxf(M, red_m[w]);
    float L = 0.f;
    for (int w = 0; w < kGenWarps; ++w) L += red_m[w] == -INFINITY ? 0.f : exp2f(red_m[w] - M) * red_l[w];
    for (int d = threadIdx.x; d < sh.head_dim; d += blockDim.x) {
        float a = 0.f;
        for (int w = 0; w < kGenWarps; ++w)
            if (red_m[w] != -INFINITY) a = fmaf(exp2f(red_m[w] - M), red_acc[w][d], a);
        o[d] = a / L;
    }
}

// ------------------------------------------------------------------------------------------
// tensor-core kernel
// ------------------------------------------------------------------------------------------
struct PfCfg {
    static constexpr int kWarps = 8;                                    // warps that multiply (16 rows each)
    static constexpr int kProducerWarps = 4;                            // warps that dequantise the tiles
    static constexpr int kThreads = (kWarps + kProducerWarps) * 32;
    // Registers: the CTA is launched with 168 per thread (the most 384 threads can have); the producers go down to
    // 40, the multiplying warps up to 232.  The registers the producers give back must cover what the others ask
    // for, or the increase waits for ever (48 for the producers does: 4 x 120 < 8 x 64).
    static constexpr int kLaunchRegs = 168, kProducerRegs = 40, kMultiplierRegs = 232;
    static_assert((kLaunchRegs - kProducerRegs) * kProducerWarps >= (kMultiplierRegs - kLaunchRegs) * kWarps,
                  "setmaxnreg: the producers must release what the multiplying warps take");
    static constexpr int kRows = 128;             // (query, head) rows per CTA: 16 per warp
    static constexpr int kTile = 64;              // cached tokens per step
    static constexpr int kRowBytes = 256;         // 128 fp16 channels
    static constexpr int kCbBytes = 128 * 256 * 2;                     // one codebook as fp16: [G][256][c]
    static constexpr int kKcbOffset = 0, kVcbOffset = kCbBytes;
    static constexpr int kQOffset = 2 * kCbBytes;
    static constexpr int kKtOffset = kQOffset + kRows * kRowBytes;     // K tiles, two buffers
    static constexpr int kVtOffset = kKtOffset + 2 * kTile * kRowBytes; // V tiles, two buffers
    static constexpr int kTileBytes = kTile * kRowBytes;
    static constexpr int kSmemBytes = kVtOffset + 2 * kTile * kRowBytes;   // 224 KiB
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of 16-byte chunk `chunk` (0..15) of row `row` in a tile of 256-byte rows; the chunk index is
// XOR-ed with the low row bits so that eight consecutive rows of one chunk column fall into different banks
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// 2^x by the special-function unit (two units in the last place; P is rounded to fp16 afterwards)
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int kC>
__global__ void __launch_bounds__(PfCfg::kThreads, 1)
prefill_mma_kernel(const __half* __restrict__ q, const uint8_t* __restrict__ kc, const uint8_t* __restrict__ vc,
                   const float* __restrict__ kcb, const float* __restrict__ vcb,
                   const int32_t* __restrict__ seq_lens, float scale_log2e, Shape sh, int n_q, int row_tiles,
                   float* __restrict__ out)
{
    using C = PfCfg;
    constexpr int G = 128 / kC;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, p = lane & 3;
    const int R = sh.R;
    const int q_per_tile = C::kRows / R;                                 // query tokens of one row tile

    const int tile = row_tiles - 1 - blockIdx.x % row_tiles;               // later queries attend more tokens: they start first
    const int hkv = (blockIdx.x / row_tiles) % sh.n_kv_heads;
    const int64_t s = blockIdx.x / ((int64_t)row_tiles * sh.n_kv_heads);
    int64_t n = seq_lens[s];
    n = n < 0 ? 0 : (n > sh.max_tokens ? sh.max_tokens : n);
    const int qi0 = tile * q_per_tile;
    // row rho of the CTA: query qi0 + rho / R, head hkv * R + rho % R, position n - n_q + query
    const int64_t pos0 = n - n_q + qi0;                                  // position of the tile's first query (may be negative)
    int q_last = qi0 + q_per_tile - 1;
    if (q_last > n_q - 1) q_last = n_q - 1;
    const int64_t pos_last = n - n_q + q_last;                           // largest position of the tile

    // ---- codebooks as fp16, the query tile
    for (int i = threadIdx.x; i < 128 * 256 / 2; i += C::kThreads) {
        const float2 a = *reinterpret_cast<const float2*>(kcb + (int64_t)hkv * 128 * 256 + 2 * i);
        const float2 b = *reinterpret_cast<const float2*>(vcb + (int64_t)hkv * 128 * 256 + 2 * i);
        // code-major ([code][group][channel]): the lanes of a gather take different groups, so they meet in no bank
        // whatever the codes are.  For c = 2 (one word per centroid, a lane gathers the groups 4 chunk + i) group g
        // sits in column 16 (g mod 4) + g / 4, so that the 16 chunks of one gather fall into 16 different banks.
        int w;
        {
            const int g = (2 * i) / (256 * kC), code = ((2 * i) / kC) % 256, ch = (2 * i) % kC;
            w = kC == 2 ? code * G + 16 * (g & 3) + (g >> 2) : ((code * G + g) * kC + ch) / 2;
        }
        *reinterpret_cast<uint32_t*>(smem + C::kKcbOffset + 4 * w) = pack_half2(a.x, a.y);
        *reinterpret_cast<uint32_t*>(smem + C::kVcbOffset + 4 * w) = pack_half2(b.x, b.y);
    }
    for (int i = threadIdx.x; i < C::kRows * 16; i += C::kThreads) {
        const int rho = i >> 4, chunk = i & 15;
        const int qi = qi0 + rho / R, h = hkv * R + rho % R;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (qi < n_q) v = *reinterpret_cast<const uint4*>(q + (((s * n_q + qi) * sh.n_q_heads + h) * 128 + chunk * 8));
        *reinterpret_cast<uint4*>(smem + C::kQOffset + tile_off(rho, chunk)) = v;
    }
    __syncthreads();

    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int j = 0; j < 4; ++j) o[nt][j] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};     // rows r and r + 8 of the warp
    // positions of this thread's two rows
    const int rho_a = warp * 16 + r, rho_b = rho_a + 8;
    const int64_t pos_a = pos0 + rho_a / R, pos_b = pos0 + rho_b / R;
    const int64_t pos_warp = pos0 + (warp * 16) / R;                      // smallest position among the warp's rows

    const int64_t n_tiles = pos_last < 0 ? 0 : pos_last / C::kTile + 1;
    const uint8_t* kbase = kc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint8_t* vbase = vc + code_word_offset(sh, sh.n_kv_heads, s, hkv, 0, 0);
    const uint32_t q_s = smem_u32(smem + C::kQOffset), kt_s = smem_u32(smem + C::kKtOffset), vt_s = smem_u32(smem + C::kVtOffset);

    // codes -> fp16 tiles of the 64 tokens from j0 on, into buffer `buf`, by the 128 producer threads: a work item
    // is (8 tokens, one group), 8 G items per tile (one per thread for c = 8, two for c = 4)
    auto dequantise_groups = [&](int64_t j0, int buf) {
        for (int item = threadIdx.x - C::kWarps * 32; item < 8 * G; item += C::kProducerWarps * 32) {
            const int g = item % G, oct = item / G;                      // tokens 8 oct .. 8 oct + 7 of the tile
            const int64_t blk = j0 / kTokenBlock + (oct >> 1);
            uint2 kw = make_uint2(0u, 0u), vw = make_uint2(0u, 0u);
            if (blk < sh.n_blocks) {
                kw = *reinterpret_cast<const uint2*>(kbase + blk * (G * kTokenBlock) + g * kTokenBlock + 8 * (oct & 1));
                vw = *reinterpret_cast<const uint2*>(vbase + blk * (G * kTokenBlock) + g * kTokenBlock + 8 * (oct & 1));
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t kcode = ((k < 4 ? kw.x : kw.y) >> (8 * (k & 3))) & 0xffu;
                const uint32_t vcode = ((k < 4 ? vw.x : vw.y) >> (8 * (k & 3))) & 0xffu;
                const int tok = 8 * oct + k;
                const uint32_t dst = tile_off(tok, (g * kC) >> 3) + (uint32_t)((g * kC) & 7) * 2u;
                if (kC == 8) {
                    *reinterpret_cast<uint4*>(smem + C::kKtOffset + buf * C::kTileBytes + dst) = *reinterpret_cast<const uint4*>(smem + C::kKcbOffset + (kcode * G + g) * 16);
                    *reinterpret_cast<uint4*>(smem + C::kVtOffset + buf * C::kTileBytes + dst) = *reinterpret_cast<const uint4*>(smem + C::kVcbOffset + (vcode * G + g) * 16);
                } else if (kC == 4) {
                    *reinterpret_cast<uint2*>(smem + C::kKtOffset + buf * C::kTileBytes + dst) = *reinterpret_cast<const uint2*>(smem + C::kKcbOffset + (kcode * G + g) * 8);
                    *reinterpret_cast<uint2*>(smem + C::kVtOffset + buf * C::kTileBytes + dst) = *reinterpret_cast<const uint2*>(smem + C::kVcbOffset + (vcode * G + g) * 8);
                } else {
                    *reinterpret_cast<uint32_t*>(smem + C::kKtOffset + buf * C::kTileBytes + dst) = *reinterpret_cast<const uint32_t*>(smem + C::kKcbOffset + (g * 256 + kcode) * 4);
                    *reinterpret_cast<uint32_t*>(smem + C::kVtOffset + buf * C::kTileBytes + dst) = *reinterpret_cast<const uint32_t*>(smem + C::kVcbOffset + (g * 256 + vcode) * 4);
                }
            }
        }
    };
    // The same with work items of (8 tokens, one 16-byte chunk of the row = 8 channels = 8 / c groups): 128 items,
    // one per producer thread, which gathers the chunk's centroids per token and stores the 16 bytes at once.
    // Measured (4 x 2048 queries over 8192 tokens, 32 heads on 8 KV heads): c = 2 5.24 -> 3.91 ms, but c = 4 3.55 -> 3.66 and c = 8
    // 3.32 -> 3.56 ms, so only c = 2 takes this form.
    auto dequantise_chunks = [&](int64_t j0, int buf) {
        constexpr int kGpi = 8 / kC;                                     // groups per item
        const int item = threadIdx.x - C::kWarps * 32;
        const int chunk = item & 15, oct = item >> 4;                    // tokens 8 oct .. 8 oct + 7 of the tile
        const int64_t blk = j0 / kTokenBlock + (oct >> 1);
        uint2 kw[kGpi], vw[kGpi];
#pragma unroll
        for (int i = 0; i < kGpi; ++i) {
            kw[i] = make_uint2(0u, 0u);
            vw[i] = make_uint2(0u, 0u);
            if (blk < sh.n_blocks) {
                const int64_t off = blk * (G * kTokenBlock) + (chunk * kGpi + i) * kTokenBlock + 8 * (oct & 1);
                kw[i] = *reinterpret_cast<const uint2*>(kbase + off);
                vw[i] = *reinterpret_cast<const uint2*>(vbase + off);
            }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t kv[4], vv[4];
#pragma unroll
            for (int i = 0; i < kGpi; ++i) {
                const uint32_t kcode = ((k < 4 ? kw[i].x : kw[i].y) >> (8 * (k & 3))) & 0xffu;
                const uint32_t vcode = ((k < 4 ? vw[i].x : vw[i].y) >> (8 * (k & 3))) & 0xffu;
                // (the c = 2 placement of the codebooks; the other sizes do not take this form)
                const uint32_t krow = (kcode * G + 16 * i + chunk) * 4;
                const uint32_t vrow = (vcode * G + 16 * i + chunk) * 4;
                if (kC == 8) {
                    const uint4 a = *reinterpret_cast<const uint4*>(smem + C::kKcbOffset + krow);
                    const uint4 b2 = *reinterpret_cast<const uint4*>(smem + C::kVcbOffset + vrow);
                    kv[0] = a.x; kv[1] = a.y; kv[2] = a.z; kv[3] = a.w;
                    vv[0] = b2.x; vv[1] = b2.y; vv[2] = b2.z; vv[3] = b2.w;
                } else if (kC == 4) {
                    const uint2 a = *reinterpret_cast<const uint2*>(smem + C::kKcbOffset + krow);
                    const uint2 b2 = *reinterpret_cast<const uint2*>(smem + C::kVcbOffset + vrow);
                    kv[(2 * i) & 3] = a.x; kv[(2 * i + 1) & 3] = a.y;
                    vv[(2 * i) & 3] = b2.x; vv[(2 * i + 1) & 3] = b2.y;
                } else {
                    kv[i & 3] = *reinterpret_cast<const uint32_t*>(smem + C::kKcbOffset + krow);
                    vv[i & 3] = *reinterpret_cast<const uint32_t*>(smem + C::kVcbOffset + vrow);
                }
            }
            const uint32_t dst = tile_off(8 * oct + k, chunk);
            *reinterpret_cast<uint4*>(smem + C::kKtOffset + buf * C::kTileBytes + dst) = make_uint4(kv[0], kv[1], kv[2], kv[3]);
            *reinterpret_cast<uint4*>(smem + C::kVtOffset + buf * C::kTileBytes + dst) = make_uint4(vv[0], vv[1], vv[2], vv[3]);
        }
    };
    auto dequantise = [&](int64_t j0, int buf) {
        if (kC == 2) dequantise_chunks(j0, buf);
        else dequantise_groups(j0, buf);
    };
    // Producer warps fill the two tile buffers, the other warps multiply; named barriers 1 + buf ("buffer free") and
    // 3 + buf ("buffer full") hand a buffer back and forth, registers move from the producers to the multipliers.
    constexpr int kAll = C::kThreads;
    if (warp >= C::kWarps) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        for (int64_t jt = 0; jt < n_tiles; ++jt) {
            const int buf = (int)(jt & 1);
            if (jt >= 2) asm volatile("bar.sync %0, %1;" ::"r"(1 + buf), "n"(kAll) : "memory");
            dequantise(jt * C::kTile, buf);
            __threadfence_block();
            asm volatile("bar.arrive %0, %1;" ::"r"(3 + buf), "n"(kAll) : "memory");
        }
        return;
    }
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
    // the warp's query rows as A fragments, kept in registers for the whole context
    uint32_t qf[8][4];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        const int mi = lane >> 3;
        ldmatrix_x4(qf[ks], q_s + tile_off(warp * 16 + (lane & 7) + 8 * (mi & 1), 2 * ks + (mi >> 1)));
    }

    for (int64_t jt = 0; jt < n_tiles; ++jt) {
        const int64_t j0 = jt * C::kTile;
        const int buf = (int)(jt & 1);
        asm volatile("bar.sync %0, %1;" ::"r"(3 + buf), "n"(kAll) : "memory");

        // ---- S = Q Khat^T for the warp's 16 rows and the tile's 64 tokens
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) sc[nt][j] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint32_t (&a)[4] = qf[ks];
#pragma unroll
            for (int ntp = 0; ntp < 4; ++ntp) {
                uint32_t b[4];
                const int mi = lane >> 3;
                ldmatrix_x4(b, kt_s + buf * C::kTileBytes + tile_off(16 * ntp + (lane & 7) + 8 * (mi >> 1), 2 * ks + (mi & 1)));
                mma_f16(sc[2 * ntp], a, b[0], b[1]);
                mma_f16(sc[2 * ntp + 1], a, b[2], b[3]);
            }
        }
        // ---- running maximum and P.  A tile that lies wholly below every row's causal limit needs no mask: the
        // maximum is taken over the raw scores and the scale folded into the exponent's multiply-add.
        float corr[2];
        uint32_t pa[4][4];                                               // P as A fragments: one per 16 tokens
        if (j0 + C::kTile - 1 <= pos_warp && scale_log2e > 0.f) {
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int j = 0; j < 4; ++j) mx[j >> 1] = fmaxf(mx[j >> 1], sc[nt][j]);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
                const float m_new = fmaxf(m_run[h], mx[h] * scale_log2e);      // finite: the tile has no masked score
                corr[h] = exp2f(m_run[h] - m_new);
                m_run[h] = m_new;
                l_run[h] *= corr[h];
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                float pv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    pv[j] = ex2_approx(fmaf(sc[nt][j], scale_log2e, -m_run[j >> 1]));
                    l_run[j >> 1] += pv[j];
                }
                pa[nt >> 1][(nt & 1) * 2 + 0] = pack_half2(pv[0], pv[1]);
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack_half2(pv[2], pv[3]);
            }
        } else {
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t tok = j0 + 8 * nt + 2 * p + (j & 1);
                    const int64_t pos = (j < 2) ? pos_a : pos_b;
                    const float v = tok <= pos ? sc[nt][j] * scale_log2e : -INFINITY;
                    sc[nt][j] = v;
                    mx[j >> 1] = fmaxf(mx[j >> 1], v);
                }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
                const float m_new = fmaxf(m_run[h], mx[h]);
                corr[h] = m_new == -INFINITY ? 1.f : exp2f(m_run[h] - m_new);
                m_run[h] = m_new;
                l_run[h] *= corr[h];
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                float pv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float mrow = m_run[j >> 1];
                    pv[j] = mrow == -INFINITY ? 0.f : exp2f(sc[nt][j] - mrow);
                    l_run[j >> 1] += pv[j];
                }
                pa[nt >> 1][(nt & 1) * 2 + 0] = pack_half2(pv[0], pv[1]);
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack_half2(pv[2], pv[3]);
            }
        }
        if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {   // most tiles leave every maximum as it was
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) {
                o[nt][0] *= corr[0];
                o[nt][1] *= corr[0];
                o[nt][2] *= corr[1];
                o[nt][3] *= corr[1];
            }
        }
        // ---- O += P Vhat
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int ntp = 0; ntp < 8; ++ntp) {
                uint32_t b[4];
                const int mi = lane >> 3;
                ldmatrix_x4_trans(b, vt_s + buf * C::kTileBytes + tile_off(16 * ks + (lane & 7) + 8 * (mi & 1), 2 * ntp + (mi >> 1)));
                mma_f16(o[2 * ntp], pa[ks], b[0], b[1]);
                mma_f16(o[2 * ntp + 1], pa[ks], b[2], b[3]);
            }
        if (jt + 2 < n_tiles) asm volatile("bar.arrive %0, %1;" ::"r"(1 + buf), "n"(kAll) : "memory");   // the buffer is free again
    }

    // ---- normalise and write (l is spread over the quad)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int rho = h == 0 ? rho_a : rho_b;
        const int qi = qi0 + rho / R;
        if (qi >= n_q) continue;
        const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;        // no position: zero row
        float* orow = out + ((s * n_q + qi) * sh.n_q_heads + hkv * R + rho % R) * 128;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
            *reinterpret_cast<float2*>(orow + 8 * nt + 2 * p) = make_float2(o[nt][2 * h] * inv, o[nt][2 * h + 1] * inv);
    }
}

}  // namespace

bool prefill_mma_supported(const Shape& sh)
{
    return sh.head_dim == 128 && sh.b == 8 && (sh.c == 2 || sh.c == 4 || sh.c == 8) && sh.R <= 64 && PfCfg::kRows % sh.R == 0;
}

cudaError_t launch_prefill(const __half* q, const uint8_t* kc, const uint8_t* vc, const float* kcb, const float* vcb,
                           const int32_t* seq_lens, float scale, const Shape& sh, int n_q, float* out, bool generic,
                           cudaStream_t st)
{
    if (!generic && prefill_mma_supported(sh)) {
        using C = PfCfg;
        const int q_per_tile = C::kRows / sh.R;
        const int row_tiles = (n_q + q_per_tile - 1) / q_per_tile;
        const int64_t grid = sh.n_seq * sh.n_kv_heads * row_tiles;
        if (grid > 0x7fffffff) return cudaErrorInvalidConfiguration;
        cudaError_t e = cudaSuccess;
        switch (sh.c) {
            case 8:
                e = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_mma_kernel<8>), C::kSmemBytes, 40);
                if (e != cudaSuccess) return e;
                prefill_mma_kernel<8><<<(unsigned)grid, C::kThreads, C::kSmemBytes, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, n_q, row_tiles, out);
                break;
            case 4:
                e = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_mma_kernel<4>), C::kSmemBytes, 41);
                if (e != cudaSuccess) return e;
                prefill_mma_kernel<4><<<(unsigned)grid, C::kThreads, C::kSmemBytes, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, n_q, row_tiles, out);
                break;
            default:
                e = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_mma_kernel<2>), C::kSmemBytes, 42);
                if (e != cudaSuccess) return e;
                prefill_mma_kernel<2><<<(unsigned)grid, C::kThreads, C::kSmemBytes, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, n_q, row_tiles, out);
                break;
        }
        return cudaGetLastError();
    }
    const int64_t grid = sh.n_seq * (int64_t)n_q * sh.n_q_heads;
    if (grid > 0x7fffffff) return cudaErrorInvalidConfiguration;
    prefill_generic_kernel<<<(unsigned)grid, kGenWarps * 32, 0, st>>>(q, kc, vc, kcb, vcb, seq_lens, scale * kLog2e, sh, n_q, out);
    return cudaGetLastError();
}

}  // namespace cq
