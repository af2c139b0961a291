/*
 * CPU oracle for Coupled Quantization (CQ) of LLM KV caches -- TEST INFRASTRUCTURE.
 *
 * Plain, slow, fp64 (encode, decode attention, and the centroid-learning steps of
 * Section 3.2.1).  It exists to check the CUDA library and to be timed as a
 * CPU baseline; it shares no code with the CUDA path and the product never
 * calls it.  Every function states the passage of the paper it follows.
 *
 * Conventions
 *   D  head_dim, c channels per group, G = D / c groups, b bits per code,
 *   K = 2^b centroids per group.
 *   x          fp16 bit patterns, row-major [n_vec][n_heads][D]
 *   codebooks  fp32, row-major [n_heads][G][K][c]
 *   codes      int32, row-major [n_vec][n_heads][G]       (encode)
 *              int32, row-major [n_seq][max_tokens][n_kv_heads][G] (attention)
 * fp16 and fp32 inputs are widened exactly to fp64; all arithmetic is fp64.
 * OpenMP parallelises only over independent items (vectors, or (sequence,
 * query head) pairs); there is no blocking, fusion or reordering inside an item.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE binary16 bit pattern -> double, exact. */
static double half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int mant = h & 0x3ff;
    double v;
    if (expo == 0)
        v = ldexp((double)mant, -24);               /* subnormal or zero */
    else if (expo == 31)
        v = mant ? NAN : INFINITY;
    else
        v = ldexp((double)(mant | 0x400), expo - 25);
    return sign ? -v : v;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * CQ encode (Section 3.2: the channels of a key/value vector are split into
 * equal, non-overlapping groups of c contiguous channels and every group is
 * replaced by the index of its nearest centroid in L2 distance; this is the
 * map CQ(.) inside Eq. 5).
 *
 * d_j = sum_{i<c} (x[g c + i] - C[h][g][j][i])^2, code = argmin_j d_j, lowest
 * index on exact ties.  d_best / d_second (may be NULL) receive the smallest
 * and second smallest distance of each (vector, head, group), which the
 * near-tie acceptance rule of the tests needs (d_second = +inf when K == 1).
 */
void oracle_encode(const uint16_t *x, const float *codebooks, int64_t n_vec,
                   int n_heads, int D, int c, int b, int32_t *codes,
                   double *d_best, double *d_second)
{
    const int G = D / c;
    const int K = 1 << b;
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n_vec; ++v) {
        for (int h = 0; h < n_heads; ++h) {
            const uint16_t *xv = x + (v * n_heads + h) * (int64_t)D;
            for (int g = 0; g < G; ++g) {
                const float *cb = codebooks + ((int64_t)h * G + g) * K * c;
                double best = INFINITY, second = INFINITY;
                int32_t arg = 0;
                for (int j = 0; j < K; ++j) {
                    double d = 0.0;
                    for (int i = 0; i < c; ++i) {
                        double diff = half_to_double(xv[g * c + i]) - (double)cb[j * c + i];
                        d += diff * diff;
                    }
                    if (d < best) {
                        second = best;
                        best = d;
                        arg = j;
                    } else if (d < second) {
                        second = d;
                    }
                }
                int64_t o = (v * n_heads + h) * G + g;
                codes[o] = arg;
                if (d_best) d_best[o] = best;
                if (d_second) d_second[o] = second;
            }
        }
    }
}

/*
 * Squared L2 distance between each group of x and the centroid named by an
 * arbitrary code (same definition of distance as oracle_encode, Section 3.2).
 * Used to judge a code that differs from the oracle's.
 */
void oracle_code_distance(const uint16_t *x, const float *codebooks, const int32_t *codes,
                          int64_t n_vec, int n_heads, int D, int c, int b, double *dist)
{
    const int G = D / c;
    const int K = 1 << b;
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n_vec; ++v)
        for (int h = 0; h < n_heads; ++h)
            for (int g = 0; g < G; ++g) {
                int64_t o = (v * n_heads + h) * G + g;
                const float *cj = codebooks + (((int64_t)h * G + g) * K + codes[o]) * c;
                double d = 0.0;
                for (int i = 0; i < c; ++i) {
                    double diff = half_to_double(x[(v * n_heads + h) * (int64_t)D + g * c + i]) - (double)cj[i];
                    d += diff * diff;
                }
                dist[o] = d;
            }
}

/*
 * Dequantisation CQ(A) (Section 3.2.1: the reconstruction whose error
 * ||A - CQ(A)||_F^2 the centroid objectives measure): channel g c + i of the
 * reconstruction is component i of centroid codes[g] of group g.
 */
void oracle_dequant(const int32_t *codes, const float *codebooks, int64_t n_vec,
                    int n_heads, int D, int c, int b, double *xhat)
{
    const int G = D / c;
    const int K = 1 << b;
    for (int64_t v = 0; v < n_vec; ++v)
        for (int h = 0; h < n_heads; ++h)
            for (int g = 0; g < G; ++g) {
                int32_t j = codes[(v * n_heads + h) * G + g];
                const float *cj = codebooks + (((int64_t)h * G + g) * K + j) * c;
                for (int i = 0; i < c; ++i)
                    xhat[(v * n_heads + h) * (int64_t)D + g * c + i] = (double)cj[i];
            }
}

/*
 * Decode attention over a CQ-coded cache, dense form (Eq. 1 with the cached
 * keys and values replaced by their CQ reconstructions, Section 3.2):
 *   Khat_t = dequant(k_codes[t]), Vhat_t = dequant(v_codes[t])
 *   s_t = scale * <q, Khat_t>,  p = softmax(s_0 .. s_{n-1}),  out = sum_t p_t Vhat_t
 * for the first n = seq_lens[s] cached tokens of sequence s.  Query head hq
 * reads KV head hq / (n_q_heads / n_kv_heads).  n == 0 gives a zero row.
 *
 *   q    fp16 bits [n_seq][n_q_heads][D]
 *   out  fp64      [n_seq][n_q_heads][D]
 */
void oracle_decode_dense(const uint16_t *q, const int32_t *k_codes, const int32_t *v_codes,
                         const float *k_cb, const float *v_cb, const int32_t *seq_lens,
                         double scale, int n_seq, int n_q_heads, int n_kv_heads, int D,
                         int c, int b, int64_t max_tokens, double *out)
{
    const int G = D / c;
    const int K = 1 << b;
    const int R = n_q_heads / n_kv_heads;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < n_seq; ++s) {
        for (int hq = 0; hq < n_q_heads; ++hq) {
            const int hkv = hq / R;
            const int64_t n = seq_lens[s];
            double *o = out + ((int64_t)s * n_q_heads + hq) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (n <= 0) continue;
            double *qd = (double *)malloc(sizeof(double) * D);
            double *score = (double *)malloc(sizeof(double) * n);
            for (int d = 0; d < D; ++d)
                qd[d] = half_to_double(q[((int64_t)s * n_q_heads + hq) * D + d]);
            double smax = -INFINITY;
            for (int64_t t = 0; t < n; ++t) {
                const int32_t *kc = k_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                double dot = 0.0;
                for (int g = 0; g < G; ++g) {
                    const float *cj = k_cb + (((int64_t)hkv * G + g) * K + kc[g]) * c;
                    for (int i = 0; i < c; ++i) dot += qd[g * c + i] * (double)cj[i];
                }
                score[t] = scale * dot;
                if (score[t] > smax) smax = score[t];
            }
            double denom = 0.0;
            for (int64_t t = 0; t < n; ++t) {
                score[t] = exp(score[t] - smax);
                denom += score[t];
            }
            for (int64_t t = 0; t < n; ++t) {
                const int32_t *vc = v_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                double p = score[t] / denom;
                for (int g = 0; g < G; ++g) {
                    const float *cj = v_cb + (((int64_t)hkv * G + g) * K + vc[g]) * c;
                    for (int i = 0; i < c; ++i) o[g * c + i] += p * (double)cj[i];
                }
            }
            free(qd);
            free(score);
        }
    }
}

/*
 * Causal attention of a run of n_q new tokens per sequence over the CQ-coded cache
 * (Section 2.1: Eq. 1 gives the output of "the current token" from the keys and values
 * of all tokens up to and including it; a prompt, or a chunk of one, applies it to each
 * of its tokens in turn, with K and V replaced by their CQ reconstructions, Section 3.2).
 *
 * The cache of sequence s holds seq_lens[s] tokens, the last n_q of which are the new
 * ones.  Query i (0 <= i < n_q) therefore sits at position pos_i = seq_lens[s] - n_q + i
 * and attends the cached tokens 0 .. pos_i:
 *   s_t = scale * <q_i, Khat_t>,  p = softmax(s_0 .. s_{pos_i}),  out_i = sum_t p_t Vhat_t
 * A query whose position is negative (seq_lens[s] < n_q: fewer cached tokens than
 * queries) has nothing to attend and gives a zero row.
 *
 *   q    fp16 bits [n_seq][n_q][n_q_heads][D]
 *   out  fp64      [n_seq][n_q][n_q_heads][D]
 */
void oracle_prefill_dense(const uint16_t *q, const int32_t *k_codes, const int32_t *v_codes,
                          const float *k_cb, const float *v_cb, const int32_t *seq_lens,
                          double scale, int n_seq, int n_q, int n_q_heads, int n_kv_heads, int D,
                          int c, int b, int64_t max_tokens, double *out)
{
    const int G = D / c;
    const int K = 1 << b;
    const int R = n_q_heads / n_kv_heads;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int s = 0; s < n_seq; ++s) {
        for (int i = 0; i < n_q; ++i) {
            for (int hq = 0; hq < n_q_heads; ++hq) {
                const int hkv = hq / R;
                const int64_t n = (int64_t)seq_lens[s] - n_q + i + 1;      /* tokens 0 .. pos_i */
                const int64_t row = ((int64_t)s * n_q + i) * n_q_heads + hq;
                double *o = out + row * D;
                for (int d = 0; d < D; ++d) o[d] = 0.0;
                if (n <= 0) continue;
                double *qd = (double *)malloc(sizeof(double) * D);
                double *score = (double *)malloc(sizeof(double) * n);
                for (int d = 0; d < D; ++d) qd[d] = half_to_double(q[row * D + d]);
                double smax = -INFINITY;
                for (int64_t t = 0; t < n; ++t) {
                    const int32_t *kc = k_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                    double dot = 0.0;
                    for (int g = 0; g < G; ++g) {
                        const float *cj = k_cb + (((int64_t)hkv * G + g) * K + kc[g]) * c;
                        for (int e = 0; e < c; ++e) dot += qd[g * c + e] * (double)cj[e];
                    }
                    score[t] = scale * dot;
                    if (score[t] > smax) smax = score[t];
                }
                double denom = 0.0;
                for (int64_t t = 0; t < n; ++t) {
                    score[t] = exp(score[t] - smax);
                    denom += score[t];
                }
                for (int64_t t = 0; t < n; ++t) {
                    const int32_t *vc = v_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                    const double p = score[t] / denom;
                    for (int g = 0; g < G; ++g) {
                        const float *cj = v_cb + (((int64_t)hkv * G + g) * K + vc[g]) * c;
                        for (int e = 0; e < c; ++e) o[g * c + e] += p * (double)cj[e];
                    }
                }
                free(qd);
                free(score);
            }
        }
    }
}

/*
 * Decode attention when the cache holds codes of the keys as they were BEFORE the
 * rotary position embedding (last sentence of Section 3.2: CQ quantises keys before
 * RoPE; Section 2.1: the key transformation f_K includes the positional encoding).
 * The key that enters Eq. 1 is then the rotated reconstruction:
 *   Khat_t = dequant(k_codes[t]);   K_t = rotate(Khat_t, position t)
 *   s_t = scale * <q, K_t>,  p = softmax(s),  out = sum_t p_t Vhat_t
 * rotate acts on channel pairs (a, b) with the angle of pair i at position t given by
 * its cosine and sine, rope_cos[t][i] and rope_sin[t][i] (fp32 [max_tokens][D/2], as
 * models cache them):
 *   K_a = Khat_a cos - Khat_b sin,   K_b = Khat_b cos + Khat_a sin
 * pairing 0: (a, b) = (i, i + D/2)   ("rotate half", the LLaMA / Mistral convention)
 * pairing 1: (a, b) = (2i, 2i + 1)   (interleaved)
 * The query is taken as given (already rotated for its own position).  Values are
 * not rotated.  The paper states neither the pairing nor how the angles are stored:
 * both are this library's reading.
 */
void oracle_decode_dense_rope(const uint16_t *q, const int32_t *k_codes, const int32_t *v_codes,
                              const float *k_cb, const float *v_cb, const int32_t *seq_lens,
                              const float *rope_cos, const float *rope_sin, int pairing,
                              double scale, int n_seq, int n_q_heads, int n_kv_heads, int D,
                              int c, int b, int64_t max_tokens, double *out)
{
    const int G = D / c;
    const int K = 1 << b;
    const int R = n_q_heads / n_kv_heads;
    const int P = D / 2;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < n_seq; ++s) {
        for (int hq = 0; hq < n_q_heads; ++hq) {
            const int hkv = hq / R;
            const int64_t n = seq_lens[s];
            double *o = out + ((int64_t)s * n_q_heads + hq) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (n <= 0) continue;
            double *qd = (double *)malloc(sizeof(double) * D);
            double *khat = (double *)malloc(sizeof(double) * D);
            double *krot = (double *)malloc(sizeof(double) * D);
            double *score = (double *)malloc(sizeof(double) * n);
            for (int d = 0; d < D; ++d)
                qd[d] = half_to_double(q[((int64_t)s * n_q_heads + hq) * D + d]);
            double smax = -INFINITY;
            for (int64_t t = 0; t < n; ++t) {
                const int32_t *kc = k_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                for (int g = 0; g < G; ++g) {
                    const float *cj = k_cb + (((int64_t)hkv * G + g) * K + kc[g]) * c;
                    for (int i = 0; i < c; ++i) khat[g * c + i] = (double)cj[i];
                }
                for (int i = 0; i < P; ++i) {
                    const int a = pairing == 0 ? i : 2 * i;
                    const int bb = pairing == 0 ? i + P : 2 * i + 1;
                    const double cs = (double)rope_cos[t * P + i], sn = (double)rope_sin[t * P + i];
                    krot[a] = khat[a] * cs - khat[bb] * sn;
                    krot[bb] = khat[bb] * cs + khat[a] * sn;
                }
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += qd[d] * krot[d];
                score[t] = scale * dot;
                if (score[t] > smax) smax = score[t];
            }
            double denom = 0.0;
            for (int64_t t = 0; t < n; ++t) {
                score[t] = exp(score[t] - smax);
                denom += score[t];
            }
            for (int64_t t = 0; t < n; ++t) {
                const int32_t *vc = v_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                double p = score[t] / denom;
                for (int g = 0; g < G; ++g) {
                    const float *cj = v_cb + (((int64_t)hkv * G + g) * K + vc[g]) * c;
                    for (int i = 0; i < c; ++i) o[g * c + i] += p * (double)cj[i];
                }
            }
            free(qd);
            free(khat);
            free(krot);
            free(score);
        }
    }
}

/*
 * The same attention in the lookup-table form the CUDA library is asked to
 * use: a per-query table LUT[g][j] = scale * <q_g, Ck[g][j]>, scores as sums
 * of table entries, softmax online over n_chunks contiguous context chunks,
 * softmax weights binned per V code, bins multiplied by the V centroids, and
 * chunk partials (m, l, acc) merged with the log-sum-exp rule.  It is an exact
 * re-association of Eq. 1 and serves only to cross-check oracle_decode_dense.
 */
void oracle_decode_lut(const uint16_t *q, const int32_t *k_codes, const int32_t *v_codes,
                       const float *k_cb, const float *v_cb, const int32_t *seq_lens,
                       double scale, int n_seq, int n_q_heads, int n_kv_heads, int D,
                       int c, int b, int64_t max_tokens, int n_chunks, double *out)
{
    const int G = D / c;
    const int K = 1 << b;
    const int R = n_q_heads / n_kv_heads;
    if (n_chunks < 1) n_chunks = 1;
    for (int s = 0; s < n_seq; ++s) {
        for (int hq = 0; hq < n_q_heads; ++hq) {
            const int hkv = hq / R;
            const int64_t n = seq_lens[s];
            double *o = out + ((int64_t)s * n_q_heads + hq) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (n <= 0) continue;
            double *lut = (double *)malloc(sizeof(double) * G * K);
            double *bins = (double *)malloc(sizeof(double) * G * K);
            double *acc = (double *)malloc(sizeof(double) * D);
            double *tot = (double *)calloc(D, sizeof(double));
            for (int g = 0; g < G; ++g)
                for (int j = 0; j < K; ++j) {
                    const float *cj = k_cb + (((int64_t)hkv * G + g) * K + j) * c;
                    double dot = 0.0;
                    for (int i = 0; i < c; ++i)
                        dot += half_to_double(q[((int64_t)s * n_q_heads + hq) * D + g * c + i]) * (double)cj[i];
                    lut[g * K + j] = scale * dot;
                }
            double M = -INFINITY, L = 0.0;   /* running max and normaliser of merged chunks */
            for (int ch = 0; ch < n_chunks; ++ch) {
                int64_t t0 = n * ch / n_chunks, t1 = n * (ch + 1) / n_chunks;
                if (t1 <= t0) continue;
                double m = -INFINITY, l = 0.0;
                for (int64_t t = t0; t < t1; ++t) {
                    const int32_t *kc = k_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                    double sc = 0.0;
                    for (int g = 0; g < G; ++g) sc += lut[g * K + kc[g]];
                    if (sc > m) m = sc;
                }
                memset(bins, 0, sizeof(double) * G * K);
                for (int64_t t = t0; t < t1; ++t) {
                    const int32_t *kc = k_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                    const int32_t *vc = v_codes + (((int64_t)s * max_tokens + t) * n_kv_heads + hkv) * G;
                    double sc = 0.0;
                    for (int g = 0; g < G; ++g) sc += lut[g * K + kc[g]];
                    double p = exp(sc - m);
                    l += p;
                    for (int g = 0; g < G; ++g) bins[g * K + vc[g]] += p;
                }
                for (int g = 0; g < G; ++g)
                    for (int i = 0; i < c; ++i) {
                        double a = 0.0;
                        for (int j = 0; j < K; ++j)
                            a += bins[g * K + j] * (double)v_cb[(((int64_t)hkv * G + g) * K + j) * c + i];
                        acc[g * c + i] = a;
                    }
                /* merge partial (m, l, acc) into (M, L, tot) */
                double Mn = m > M ? m : M;
                double wo = (M == -INFINITY) ? 0.0 : exp(M - Mn);
                double wn = exp(m - Mn);
                for (int d = 0; d < D; ++d) tot[d] = tot[d] * wo + acc[d] * wn;
                L = L * wo + l * wn;
                M = Mn;
            }
            for (int d = 0; d < D; ++d) o[d] = tot[d] / L;
            free(lut);
            free(bins);
            free(acc);
            free(tot);
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Centroid learning (Section 3.2.1).  For every (head, group) one independent k-means
 * problem over the n_vec group vectors: Eq. 5 (uniform) or Eq. 6 (every group vector carries
 * a non-negative weight, the paper's g^T g of that group).  The paper runs k-means++
 * initialisation followed by a fixed number of k-means iterations (Section 4.3).
 *   x         fp16 bits [n_vec][n_heads][D]
 *   weights   fp32 [n_vec][n_heads][G], or NULL for all-ones (Eq. 5)
 *   codebooks fp32 [n_heads][G][K][c]
 * ------------------------------------------------------------------------------------------ */

/*
 * k-means++ (Arthur and Vassilvitskii 2007) with the random draws passed in:
 * uniforms [n_heads][G][K], each in [0, 1).  Centre 0 of a problem is vector
 * floor(u_0 * n_vec).  Centre k >= 1 is vector i*, the first index whose running sum
 * sum_{i <= i*} w_i D_i reaches u_k * sum_i w_i D_i, where D_i is the squared distance of
 * vector i to its nearest already chosen centre; sums run in index order, in fp64; if the
 * total is 0 (fewer distinct vectors than centres) the draw falls back to floor(u_k * n_vec).
 * chosen (may be NULL) receives the picked vector indices [n_heads][G][K].
 */
void oracle_kmeanspp_init(const uint16_t *x, const float *weights, const double *uniforms,
                          int64_t n_vec, int n_heads, int D, int c, int b,
                          float *codebooks, int64_t *chosen)
{
    const int G = D / c;
    const int K = 1 << b;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int h = 0; h < n_heads; ++h) {
        for (int g = 0; g < G; ++g) {
            double *dist = (double *)malloc(sizeof(double) * (size_t)n_vec);
            float *cb = codebooks + ((int64_t)h * G + g) * K * c;
            const double *u = uniforms + ((int64_t)h * G + g) * K;
            for (int k = 0; k < K; ++k) {
                int64_t pick;
                if (k == 0) {
                    pick = (int64_t)(u[0] * (double)n_vec);
                } else {
                    double total = 0.0;
                    for (int64_t i = 0; i < n_vec; ++i) {
                        double w = weights ? (double)weights[(i * n_heads + h) * G + g] : 1.0;
                        total += w * dist[i];
                    }
                    if (total > 0.0) {
                        const double target = u[k] * total;
                        double run = 0.0;
                        pick = n_vec - 1;
                        for (int64_t i = 0; i < n_vec; ++i) {
                            double w = weights ? (double)weights[(i * n_heads + h) * G + g] : 1.0;
                            run += w * dist[i];
                            if (run >= target && w * dist[i] > 0.0) { pick = i; break; }
                        }
                    } else {
                        pick = (int64_t)(u[k] * (double)n_vec);
                    }
                }
                if (pick >= n_vec) pick = n_vec - 1;
                if (chosen) chosen[((int64_t)h * G + g) * K + k] = pick;
                for (int i = 0; i < c; ++i)
                    cb[k * c + i] = (float)half_to_double(x[(pick * n_heads + h) * (int64_t)D + g * c + i]);
                for (int64_t i = 0; i < n_vec; ++i) {
                    double d = 0.0;
                    for (int j = 0; j < c; ++j) {
                        double diff = half_to_double(x[(i * n_heads + h) * (int64_t)D + g * c + j]) - (double)cb[k * c + j];
                        d += diff * diff;
                    }
                    if (k == 0 || d < dist[i]) dist[i] = d;
                }
            }
            free(dist);
        }
    }
}

/*
 * One k-means (Lloyd) iteration: assign every group vector to its nearest centroid (the map
 * CQ(.), lowest index on ties), then move every centroid to the weighted mean of its members;
 * a centroid without members (or with zero total weight) stays where it is.
 * codes_out (may be NULL) [n_vec][n_heads][G]; objective_out (may be NULL) [n_heads][G] receives
 * sum_i w_i ||x_i - CQ(x_i)||^2 of the assignment, i.e. the objective of Eq. 5 / Eq. 6 for the
 * INPUT codebooks.
 */
void oracle_lloyd_step(const uint16_t *x, const float *weights, const float *codebooks_in,
                       int64_t n_vec, int n_heads, int D, int c, int b,
                       float *codebooks_out, int32_t *codes_out, double *objective_out)
{
    const int G = D / c;
    const int K = 1 << b;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int h = 0; h < n_heads; ++h) {
        for (int g = 0; g < G; ++g) {
            const float *cb = codebooks_in + ((int64_t)h * G + g) * K * c;
            float *out = codebooks_out + ((int64_t)h * G + g) * K * c;
            double *sum = (double *)calloc((size_t)K * c, sizeof(double));
            double *wsum = (double *)calloc((size_t)K, sizeof(double));
            double obj = 0.0;
            for (int64_t i = 0; i < n_vec; ++i) {
                const uint16_t *xv = x + (i * n_heads + h) * (int64_t)D + g * c;
                double best = INFINITY;
                int arg = 0;
                for (int j = 0; j < K; ++j) {
                    double d = 0.0;
                    for (int q = 0; q < c; ++q) {
                        double diff = half_to_double(xv[q]) - (double)cb[j * c + q];
                        d += diff * diff;
                    }
                    if (d < best) { best = d; arg = j; }
                }
                double w = weights ? (double)weights[(i * n_heads + h) * G + g] : 1.0;
                obj += w * best;
                wsum[arg] += w;
                for (int q = 0; q < c; ++q) sum[arg * c + q] += w * half_to_double(xv[q]);
                if (codes_out) codes_out[(i * n_heads + h) * G + g] = arg;
            }
            for (int j = 0; j < K; ++j)
                for (int q = 0; q < c; ++q)
                    out[j * c + q] = wsum[j] > 0.0 ? (float)(sum[j * c + q] / wsum[j]) : cb[j * c + q];
            if (objective_out) objective_out[h * G + g] = obj;
            free(sum);
            free(wsum);
        }
    }
}
