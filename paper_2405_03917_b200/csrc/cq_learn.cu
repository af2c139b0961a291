// Centroid learning (Section 3.2.1 of the paper): k-means++ initialisation and k-means
// iterations, uniform (Eq. 5) or weighted per group vector (Eq. 6), for every (head, group)
// problem of a key or value tensor at once.  The assignment step of an iteration is cq_encode.
//
// k-means++ decides integers (which vector becomes the next centre) from sums of squared
// distances.  Those sums are formed in fp64, in index order, with the same operation order as
// the definition (one multiply and one add per term, no fused multiply-add), so that the
// decision does not depend on the machine: one CTA per problem stages the terms in shared
// memory and one of its threads adds them up in order (two passes per draw), while the distance
// update between draws runs over all (vector, problem) pairs in parallel.  The mean update of an iteration accumulates in fp32 in shared memory.
#include "cq_common.cuh"

namespace cq {

namespace {

// problem p = h * G + g; vector i.  dist[p][i]: squared distance of vector i to its nearest centre
// so far; contrib[p][i] = w_i * dist[p][i], the term of the k-means++ draw.

// One CTA per problem.  The CTA stages tiles of contributions in shared memory (coalesced loads, the next
// tile while the current one is summed); thread 0 adds them up in index order, so the fp64 running sum is
// the sequential one.  The running sum at the end of every tile is kept: it never decreases (the
// contributions are not negative), so the walk that looks for the drawn vector starts at the first tile
// whose end reaches the target, from the sum before that tile - the same additions in the same order as a
// walk from the first vector, without repeating them.
constexpr int kPickThreads = 128;
constexpr int kPickTile = 2048;
constexpr int kPickPrefixes = 1024;              // tile ends that are kept (later tiles are walked one by one)

// sum += v[0] + ... in order, sixteen loads in flight ahead of the chain of additions
__device__ __forceinline__ double pick_sum_tile(const double* tile, int m, double sum)
{
    int e = 0;
    for (; e + 16 <= m; e += 16) {
        double v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = tile[e + j];
#pragma unroll
        for (int j = 0; j < 16; ++j) sum = __dadd_rn(sum, v[j]);
    }
    for (; e < m; ++e) sum = __dadd_rn(sum, tile[e]);
    return sum;
}

__global__ void __launch_bounds__(kPickThreads)
pp_pick_kernel(const __half* __restrict__ x, const double* __restrict__ uniforms, const double* __restrict__ contrib,
               int64_t n_vec, int n_prob, int c, int K, int k, float* __restrict__ codebooks)
{
    __shared__ double tile[2][kPickTile];
    __shared__ double s_prefix[kPickPrefixes];
    __shared__ double s_total;
    __shared__ long long s_pick;
    const int p = blockIdx.x;
    const double u = uniforms[(int64_t)p * K + k];
    const double* cp = contrib + (int64_t)p * n_vec;
    const int64_t n_tiles = (n_vec + kPickTile - 1) / kPickTile;
    auto stage = [&](int64_t t, int buf) {
        const int64_t t0 = t * kPickTile;
        const int m = (int)(n_vec - t0 < kPickTile ? n_vec - t0 : kPickTile);
        // warp 0 does not stage: its first thread is busy with the chain of additions
        for (int e = (int)threadIdx.x - 32; e >= 0 && e < m; e += kPickThreads - 32) tile[buf][e] = cp[t0 + e];
    };
    if (threadIdx.x == 0) s_pick = -1;
    if (k > 0) {
        double total = 0.0;
        stage(0, 0);
        for (int64_t t = 0; t < n_tiles; ++t) {
            __syncthreads();                                  // tile t is staged, the other buffer is free
            if (t + 1 < n_tiles) stage(t + 1, (int)((t + 1) & 1));
            if (threadIdx.x == 0) {
                const int64_t t0 = t * kPickTile;
                const int m = (int)(n_vec - t0 < kPickTile ? n_vec - t0 : kPickTile);
                total = pick_sum_tile(tile[t & 1], m, total);
                if (t < kPickPrefixes) s_prefix[t] = total;
            }
        }
        if (threadIdx.x == 0) s_total = total;
        __syncthreads();
        if (s_total > 0.0) {
            const double target = __dmul_rn(u, s_total);
            // first tile whose end reaches the target (every thread takes the same decision)
            int64_t first = 0;
            const int64_t kept = n_tiles < kPickPrefixes ? n_tiles : kPickPrefixes;
            while (first < kept && !(s_prefix[first] >= target)) ++first;
            if (first == n_tiles) first = n_tiles - 1;      // rounding put the target past the total: the last tile decides
            double run = first > 0 ? s_prefix[first - 1] : 0.0;
            for (int64_t t = first; t < n_tiles; ++t) {
                const int64_t t0 = t * kPickTile;
                const int m = (int)(n_vec - t0 < kPickTile ? n_vec - t0 : kPickTile);
                __syncthreads();
                if (s_pick >= 0) break;                     // same value in every thread: read after the barrier
                for (int e = threadIdx.x; e < m; e += kPickThreads) tile[0][e] = cp[t0 + e];
                __syncthreads();
                if (threadIdx.x == 0)
                    for (int e = 0; e < m; ++e) {
                        run = __dadd_rn(run, tile[0][e]);
                        if (run >= target && tile[0][e] > 0.0) { s_pick = t0 + e; break; }
                    }
            }
            __syncthreads();
            if (threadIdx.x == 0 && s_pick < 0) s_pick = n_vec - 1;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long pick = s_pick;
        if (pick < 0) pick = (long long)__dmul_rn(u, (double)n_vec);       // first centre, or no vector left to draw
        if (pick >= n_vec) pick = n_vec - 1;
        // x row of vector `pick`: all problems of a vector are contiguous (p * c = h * D + g * c)
        const __half* xv = x + pick * (int64_t)n_prob * c + (int64_t)p * c;
        float* cb = codebooks + ((int64_t)p * K + k) * c;
        for (int q = 0; q < c; ++q) cb[q] = __half2float(xv[q]);
    }
}

// Distances to the nearest chosen centre and the contributions w * D, for tiles of 32 vectors x 32 problems.
// x and the weights are vector-major, the distances and contributions problem-major (a draw reads one
// problem's run): the tile is turned in shared memory so that every global access runs along the
// contiguous index.  Thread (tx, ty): tx is the vector when the problem-major arrays are touched and the
// problem when x is read.
constexpr int kDistTile = 32;
__global__ void __launch_bounds__(256)
pp_dist_kernel(const __half* __restrict__ x, const float* __restrict__ weights, const float* __restrict__ codebooks,
               int64_t n_vec, int n_prob, int c, int K, int k, double* __restrict__ dist, double* __restrict__ contrib)
{
    __shared__ double d_s[kDistTile][kDistTile + 1];          // [problem][vector]
    __shared__ double c_s[kDistTile][kDistTile + 1];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t tiles_i = (n_vec + kDistTile - 1) / kDistTile;
    const int64_t tiles_p = (n_prob + kDistTile - 1) / kDistTile;
    for (int64_t tile = blockIdx.x; tile < tiles_i * tiles_p; tile += gridDim.x) {
        const int64_t i0 = (tile % tiles_i) * kDistTile;
        const int p0 = (int)(tile / tiles_i) * kDistTile;
        if (k > 0) {
            for (int pp = ty; pp < kDistTile; pp += 8)
                if (p0 + pp < n_prob && i0 + tx < n_vec) d_s[pp][tx] = dist[(int64_t)(p0 + pp) * n_vec + i0 + tx];
        }
        __syncthreads();
        for (int ii = ty; ii < kDistTile; ii += 8) {
            const int64_t i = i0 + ii;
            const int p = p0 + tx;
            if (i < n_vec && p < n_prob) {
                const __half* xv = x + (i * n_prob + p) * c;
                const float* cb = codebooks + ((int64_t)p * K + k) * c;
                double d = 0.0;
                for (int q = 0; q < c; ++q) {
                    const double diff = __dsub_rn((double)__half2float(xv[q]), (double)cb[q]);
                    d = __dadd_rn(d, __dmul_rn(diff, diff));
                }
                if (k > 0 && !(d < d_s[tx][ii])) d = d_s[tx][ii];
                const double w = weights ? (double)weights[i * n_prob + p] : 1.0;
                d_s[tx][ii] = d;
                c_s[tx][ii] = __dmul_rn(w, d);
            }
        }
        __syncthreads();
        for (int pp = ty; pp < kDistTile; pp += 8)
            if (p0 + pp < n_prob && i0 + tx < n_vec) {
                const int64_t idx = (int64_t)(p0 + pp) * n_vec + i0 + tx;
                dist[idx] = d_s[pp][tx];
                contrib[idx] = c_s[pp][tx];
            }
        __syncthreads();
    }
}

// One CTA per problem: weighted sums of the members of every centroid in shared memory, then the
// new centroids; the objective of the assignment (against the input codebooks) in fp64.
constexpr int kUpdThreads = 256;
__global__ void __launch_bounds__(kUpdThreads)
lloyd_update_kernel(const __half* __restrict__ x, const float* __restrict__ weights, const uint8_t* __restrict__ codes,
                    const float* __restrict__ cb_in, Shape sh, int64_t n_vec, float* __restrict__ cb_out,
                    double* __restrict__ objective)
{
    extern __shared__ float upd_smem[];            // [K][c] sums, [K] weight sums, [K][c] input centroids
    const int p = blockIdx.x, h = p / sh.G, g = p % sh.G, c = sh.c, K = sh.K;
    const int n_prob = sh.n_kv_heads * sh.G;
    float* sums = upd_smem;
    float* wsum = sums + K * c;
    float* cin = wsum + K;
    for (int e = threadIdx.x; e < K * c; e += kUpdThreads) { sums[e] = 0.f; cin[e] = cb_in[(int64_t)p * K * c + e]; }
    for (int e = threadIdx.x; e < K; e += kUpdThreads) wsum[e] = 0.f;
    __syncthreads();
    double obj = 0.0;
    for (int64_t i = threadIdx.x; i < n_vec; i += kUpdThreads) {
        const int code = read_code(codes + code_word_offset(sh, sh.n_kv_heads, 0, h, i / kTokenBlock, 0), sh, g,
                                   (int)(i % kTokenBlock));
        const float w = weights ? weights[i * n_prob + p] : 1.f;
        const __half* xv = x + (i * n_prob + p) * (int64_t)c;
        double d = 0.0;
        for (int q = 0; q < c; ++q) {
            const float xf = __half2float(xv[q]);
            const double diff = (double)xf - (double)cin[code * c + q];
            d += diff * diff;
            atomicAdd(&sums[code * c + q], w * xf);
        }
        atomicAdd(&wsum[code], w);
        obj += (double)w * d;
    }
    // objective: block reduction in fp64
    __shared__ double red[kUpdThreads / 32];
    for (int o = 16; o > 0; o >>= 1) obj += __shfl_xor_sync(0xffffffffu, obj, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = obj;
    __syncthreads();
    if (threadIdx.x == 0 && objective) {
        double t = 0.0;
        for (int wv = 0; wv < kUpdThreads / 32; ++wv) t += red[wv];
        objective[p] = t;
    }
    for (int e = threadIdx.x; e < K * c; e += kUpdThreads) {
        const float ws = wsum[e / c];
        cb_out[(int64_t)p * K * c + e] = ws > 0.f ? sums[e] / ws : cin[e];
    }
}

size_t round256(size_t v) { return (v + 255) / 256 * 256; }

struct LearnLayout {
    size_t codes, dist, tmp_cb, total;
};

LearnLayout learn_layout(const Shape& sh, int64_t n_vec)
{
    LearnLayout l;
    const size_t n_prob = (size_t)sh.n_kv_heads * sh.G;
    l.codes = round256((size_t)sh.n_kv_heads * ((n_vec + kTokenBlock - 1) / kTokenBlock) * sh.block_bytes);
    l.dist = round256((size_t)n_vec * n_prob * sizeof(double));
    l.tmp_cb = round256(n_prob * sh.K * sh.c * sizeof(float));
    l.total = l.codes + 2 * l.dist + l.tmp_cb;      // dist and contrib
    return l;
}

}  // namespace

size_t learn_workspace_bytes(const Shape& sh, int64_t n_vec) { return learn_layout(sh, n_vec).total; }

cudaError_t launch_kmeanspp_init(const __half* x, const float* weights, const double* uniforms, const Shape& sh,
                                 int64_t n_vec, float* codebooks, void* workspace, cudaStream_t st)
{
    const LearnLayout l = learn_layout(sh, n_vec);
    double* dist = reinterpret_cast<double*>(static_cast<char*>(workspace) + l.codes);
    const int n_prob = sh.n_kv_heads * sh.G;
    const int64_t dist_tiles = ((n_vec + kDistTile - 1) / kDistTile) * ((n_prob + kDistTile - 1) / kDistTile);
    const int64_t dist_cap = (int64_t)device_sm_count() * 64;
    const int dist_grid = (int)(dist_tiles < dist_cap ? dist_tiles : dist_cap);
    double* contrib = reinterpret_cast<double*>(static_cast<char*>(workspace) + l.codes + l.dist);
    for (int k = 0; k < sh.K; ++k) {
        pp_pick_kernel<<<n_prob, kPickThreads, 0, st>>>(x, uniforms, contrib, n_vec, n_prob, sh.c, sh.K, k, codebooks);
        pp_dist_kernel<<<dist_grid, 256, 0, st>>>(x, weights, codebooks, n_vec, n_prob, sh.c, sh.K, k, dist, contrib);
    }
    return cudaGetLastError();
}

cudaError_t launch_lloyd_step(const __half* x, const float* weights, const float* cb_in, const Shape& sh, int64_t n_vec,
                              float* cb_out, double* objective, void* workspace, cudaStream_t st)
{
    const LearnLayout l = learn_layout(sh, n_vec);
    uint8_t* codes = static_cast<uint8_t*>(workspace);
    // assignment: the vectors are one sequence of n_vec tokens
    Shape es = sh;
    es.n_seq = 1;
    es.max_tokens = n_vec;
    es.n_blocks = (n_vec + kTokenBlock - 1) / kTokenBlock;
    cudaError_t e = encode_tuned_supported(es) ? launch_encode_tuned(x, cb_in, nullptr, es, n_vec, 0, codes, st)
                                               : launch_encode_generic(x, cb_in, nullptr, es, n_vec, 0, codes, st);
    if (e != cudaSuccess) return e;
    const size_t smem = (size_t)(2 * sh.K * sh.c + sh.K) * sizeof(float);
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(lloyd_update_kernel), (int)smem, 34);
    if (e != cudaSuccess) return e;
    lloyd_update_kernel<<<sh.n_kv_heads * sh.G, kUpdThreads, smem, st>>>(x, weights, codes, cb_in, es, n_vec, cb_out,
                                                                         objective);
    (void)l;
    return cudaGetLastError();
}

cudaError_t launch_learn(const __half* x, const float* weights, const double* uniforms, const Shape& sh, int64_t n_vec,
                         int n_iters, float* codebooks, double* objective, void* workspace, cudaStream_t st)
{
    const LearnLayout l = learn_layout(sh, n_vec);
    float* tmp = reinterpret_cast<float*>(static_cast<char*>(workspace) + l.codes + 2 * l.dist);
    cudaError_t e = launch_kmeanspp_init(x, weights, uniforms, sh, n_vec, codebooks, workspace, st);
    if (e != cudaSuccess) return e;
    float* cur = codebooks;
    float* nxt = tmp;
    for (int it = 0; it < n_iters; ++it) {
        e = launch_lloyd_step(x, weights, cur, sh, n_vec, nxt, objective, workspace, st);
        if (e != cudaSuccess) return e;
        float* t = cur; cur = nxt; nxt = t;
    }
    if (cur != codebooks)
        e = cudaMemcpyAsync(codebooks, cur, (size_t)sh.n_kv_heads * sh.G * sh.K * sh.c * sizeof(float),
                            cudaMemcpyDeviceToDevice, st);
    return e;
}

}  // namespace cq
