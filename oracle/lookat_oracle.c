/*
 * CPU oracle for LOOKAT decode attention over product-quantised keys.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the method computes, written from the paper, in fp64.  Only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark may call it.  It
 * shares no code with the CUDA library and the CUDA library never calls it.
 *
 * Pins (checked by the CPU tests): lookup-sum == q . k_hat; exactness when
 * m = d_k and the codebooks list every value; brute-force argmin; Lloyd
 * distortion non-increasing, K = 1 closed form; softmax closed forms.
 * Parity unpinned: the k-means initialisation rule (the paper fixes none).
 *
 * Layouts (row-major, innermost last):
 *   keys       fp16 bits  [B][H_kv][n][d_k]
 *   values     fp16 bits  [B][H_kv][L_max][d_v]
 *   queries    fp16 bits  [B][H_q][d_k]
 *   codebooks  fp32       [H_kv][m][K][d_sub]      d_sub = d_k / m
 *   codes      uint8      [B][H_kv][L_max][m]
 *   lut        fp64       [B][H_q][m][K]
 * Query head hq reads the codes, values and codebooks of KV head hq / g,
 * g = H_q / H_kv.  OpenMP is used only across independent (batch, head,
 * subspace) units; every unit runs the paper's steps in order.
 */
#include <math.h>
#include <omp.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* How many threads the OpenMP loops over independent units use from now on (the benchmark times the oracle with
 * one thread and with all of them); returns the setting in force.  No arithmetic depends on it. */
int oracle_set_num_threads(int n)
{
    if (n > 0) omp_set_num_threads(n);
    return omp_get_max_threads();
}

/* fp16 bit pattern -> double, exact (IEEE binary16: 1 sign, 5 exponent, 10 fraction bits). */
static double half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24);                  /* zero / subnormal */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(f | 0x400), e - 25);
    return sign ? -v : v;
}

/* fp16 bit pattern -> integer multiple of 2^-24 (every finite fp16 is one). */
static int64_t half_to_fixed24(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int64_t f = h & 0x3ff;
    int64_t v = (e == 0) ? f : ((f | 0x400) << (e - 1));
    return sign ? -v : v;
}

void oracle_half_to_double(const uint16_t *src, double *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = half_to_double(src[i]);
}

/* Squared L2 distance of a key sub-vector to one centroid, difference form
 * (Section 3.4: || k^(i) - c ||^2). */
static double sq_dist(const double *x, const float *c, int d_sub)
{
    double acc = 0.0;
    for (int i = 0; i < d_sub; ++i) {
        double t = x[i] - (double)c[i];
        acc += t * t;
    }
    return acc;
}

/* argmin over the K centroids of one codebook; the first minimum wins.
 * Also returns the best and the second-best distance. */
static int nearest_centroid(const double *x, const float *book, int K, int d_sub,
                            double *best_out, double *second_out)
{
    int best_c = 0;
    double best = INFINITY, second = INFINITY;
    for (int c = 0; c < K; ++c) {
        double d = sq_dist(x, book + (size_t)c * d_sub, d_sub);
        if (d < best) {
            second = best;
            best = d;
            best_c = c;
        } else if (d < second) {
            second = d;
        }
    }
    if (best_out) *best_out = best;
    if (second_out) *second_out = second;
    return best_c;
}

/*
 * Encoding (Section 3.4, "Encoding"): each key is replaced by m indices,
 * code[j] = argmin_c || k^(j) - C_j[c] ||^2.
 *
 * keys [B][H_kv][n][d_k]; codes written at token offset pos of a
 * [B][H_kv][L_max][m] array.  rel_gap (optional, [B][H_kv][n][m]) receives
 * (d2 - d1) / d2 for the best and second-best distance (0/0 := 0; K == 1
 * gives +inf): a key whose gap lies in (0, 1e-6) is a "near tie".
 */
void oracle_encode_keys(const uint16_t *keys, int B, int H_kv, int64_t n, int d_k, int m, int K,
                        const float *codebooks, uint8_t *codes, int64_t L_max, int64_t pos,
                        double *rel_gap)
{
    int d_sub = d_k / m;
    int64_t units = (int64_t)B * H_kv;
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < units; ++u) {
        int h = (int)(u % H_kv);
        double *x = (double *)malloc(sizeof(double) * d_k);
        for (int64_t t = 0; t < n; ++t) {
            const uint16_t *row = keys + ((size_t)u * n + t) * d_k;
            for (int i = 0; i < d_k; ++i) x[i] = half_to_double(row[i]);
            for (int j = 0; j < m; ++j) {
                const float *book = codebooks + ((size_t)h * m + j) * K * d_sub;
                double d1, d2;
                int c = nearest_centroid(x + j * d_sub, book, K, d_sub, &d1, &d2);
                codes[((size_t)u * L_max + pos + t) * m + j] = (uint8_t)c;
                if (rel_gap) {
                    double gap;
                    if (K < 2) gap = INFINITY;
                    else if (d2 == 0.0) gap = 0.0;
                    else gap = (d2 - d1) / d2;
                    rel_gap[((size_t)u * n + t) * m + j] = gap;
                }
            }
        }
        free(x);
    }
}

/*
 * Prototype learning (Section 3.4, "Prototype Learning"): per subspace a
 * K-centroid codebook minimising sum_k min_c || k^(i) - c ||^2, by Lloyd's
 * algorithm with a fixed number of iterations.
 *
 * The N = B*n keys of one KV head are pooled, pooled index = b*n + t.
 * init == NULL: centroid c starts at pooled row (off + c*stride) mod N with
 *   off = (seed + 0x9E3779B97F4A7C15 * (h*m + j + 1)) mod 2^64 mod N,
 *   stride = max(1, N / K).
 * Assignment: argmin in fp64, first minimum wins.  Update: the mean of the
 * members, summed exactly (every fp16 is an integer multiple of 2^-24), one
 * fp64 division, rounded once to fp32; an empty cluster keeps its centroid.
 * distortion (optional) [H_kv][m][iters+1]: the objective before each
 * update and after the last one.
 * Returns 0, or -1 if N is too large for exact 64-bit sums.
 */
int oracle_fit_codebooks(const uint16_t *keys, int B, int H_kv, int64_t n, int d_k, int m, int K,
                         int iters, uint64_t seed, const float *init, float *codebooks,
                         double *distortion)
{
    int d_sub = d_k / m;
    int64_t N = (int64_t)B * n;
    if (N > ((int64_t)1 << 22)) return -1;           /* |x * 2^24| < 2^40, 2^22 terms < 2^62 */
    int problems = H_kv * m;
#pragma omp parallel for schedule(dynamic)
    for (int p = 0; p < problems; ++p) {
        int h = p / m, j = p % m;
        float *book = codebooks + (size_t)p * K * d_sub;
        double *X = (double *)malloc(sizeof(double) * N * d_sub);
        int64_t *Xfix = (int64_t *)malloc(sizeof(int64_t) * N * d_sub);
        int *assign = (int *)malloc(sizeof(int) * N);
        int64_t *sum = (int64_t *)malloc(sizeof(int64_t) * K * d_sub);
        int64_t *cnt = (int64_t *)malloc(sizeof(int64_t) * K);
        for (int b = 0; b < B; ++b)
            for (int64_t t = 0; t < n; ++t) {
                const uint16_t *row = keys + (((size_t)b * H_kv + h) * n + t) * d_k + j * d_sub;
                for (int i = 0; i < d_sub; ++i) {
                    X[((size_t)b * n + t) * d_sub + i] = half_to_double(row[i]);
                    Xfix[((size_t)b * n + t) * d_sub + i] = half_to_fixed24(row[i]);
                }
            }
        if (init) {
            memcpy(book, init + (size_t)p * K * d_sub, sizeof(float) * K * d_sub);
        } else {
            uint64_t off = (seed + 0x9E3779B97F4A7C15ull * (uint64_t)(h * m + j + 1)) % (uint64_t)N;
            uint64_t stride = (uint64_t)(N / K) > 0 ? (uint64_t)(N / K) : 1;
            for (int c = 0; c < K; ++c) {
                uint64_t r = (off + (uint64_t)c * stride) % (uint64_t)N;
                for (int i = 0; i < d_sub; ++i) book[(size_t)c * d_sub + i] = (float)X[r * d_sub + i];
            }
        }
        for (int it = 0; it <= iters; ++it) {
            double D = 0.0;
            for (int64_t r = 0; r < N; ++r) {
                double best;
                assign[r] = nearest_centroid(X + r * d_sub, book, K, d_sub, &best, NULL);
                D += best;
            }
            if (distortion) distortion[(size_t)p * (iters + 1) + it] = D;
            if (it == iters) break;
            memset(sum, 0, sizeof(int64_t) * K * d_sub);
            memset(cnt, 0, sizeof(int64_t) * K);
            for (int64_t r = 0; r < N; ++r) {
                int c = assign[r];
                cnt[c] += 1;
                for (int i = 0; i < d_sub; ++i) sum[(size_t)c * d_sub + i] += Xfix[r * d_sub + i];
            }
            for (int c = 0; c < K; ++c) {
                if (cnt[c] == 0) continue;
                for (int i = 0; i < d_sub; ++i) {
                    double mean = ldexp((double)sum[(size_t)c * d_sub + i], -24) / (double)cnt[c];
                    book[(size_t)c * d_sub + i] = (float)mean;
                }
            }
        }
        free(X); free(Xfix); free(assign); free(sum); free(cnt);
    }
    return 0;
}

/*
 * Lookup tables (Section 3.5, "Precomputation Lookup Tables"; Algorithm 1,
 * first loop):  LUT_j[c] = q^(j) . C_j[c],  unscaled, in fp64.
 */
void oracle_build_lut(const uint16_t *q, int B, int H_q, int H_kv, int d_k, int m, int K,
                      const float *codebooks, double *lut)
{
    int d_sub = d_k / m;
    int g = H_q / H_kv;
    int64_t units = (int64_t)B * H_q;
#pragma omp parallel for schedule(static)
    for (int64_t u = 0; u < units; ++u) {
        int hq = (int)(u % H_q);
        int h = hq / g;
        for (int j = 0; j < m; ++j)
            for (int c = 0; c < K; ++c) {
                const float *cen = codebooks + (((size_t)h * m + j) * K + c) * d_sub;
                double acc = 0.0;
                for (int i = 0; i < d_sub; ++i)
                    acc += half_to_double(q[(size_t)u * d_k + j * d_sub + i]) * (double)cen[i];
                lut[((size_t)u * m + j) * K + c] = acc;
            }
    }
}

/*
 * Algorithm 1, second loop and continuation: s_l = sum_j LUT_j[code_l[j]],
 * alpha = softmax(s * scale) over l < seq_len, o = sum_l alpha_l v_l.
 * seq_lens == NULL means every row uses L_max tokens; a row with no token
 * gives o = 0.  scores / alpha (optional) are [B][H_q][L_max]; entries at or
 * beyond seq_len are left untouched.
 */
void oracle_attend(const double *lut, const uint8_t *codes, const uint16_t *v, int B, int H_q,
                   int H_kv, int64_t L_max, const int32_t *seq_lens, int d_v, int m, int K,
                   double scale, double *out, double *scores, double *alpha)
{
    int g = H_q / H_kv;
    int64_t units = (int64_t)B * H_q;
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < units; ++u) {
        int b = (int)(u / H_q), hq = (int)(u % H_q);
        int h = hq / g;
        int64_t L = seq_lens ? seq_lens[b] : L_max;
        const double *T = lut + (size_t)u * m * K;
        const uint8_t *cd = codes + ((size_t)b * H_kv + h) * L_max * m;
        const uint16_t *vv = v + ((size_t)b * H_kv + h) * L_max * d_v;
        double *o = out + (size_t)u * d_v;
        for (int i = 0; i < d_v; ++i) o[i] = 0.0;
        if (L <= 0) continue;
        double *s = (double *)malloc(sizeof(double) * L);
        double M = -INFINITY;
        for (int64_t l = 0; l < L; ++l) {
            double acc = 0.0;
            for (int j = 0; j < m; ++j) acc += T[(size_t)j * K + cd[l * m + j]];
            s[l] = acc;
            if (scores) scores[(size_t)u * L_max + l] = acc;
            if (acc * scale > M) M = acc * scale;
        }
        double Z = 0.0;
        for (int64_t l = 0; l < L; ++l) {
            s[l] = exp(s[l] * scale - M);
            Z += s[l];
        }
        for (int64_t l = 0; l < L; ++l) {
            double a = s[l] / Z;
            if (alpha) alpha[(size_t)u * L_max + l] = a;
            for (int i = 0; i < d_v; ++i) o[i] += a * half_to_double(vv[l * d_v + i]);
        }
        free(s);
    }
}

/*
 * Exact attention of Section 3.1 for one decode query per head:
 * softmax(q K^T * scale) V on the fp16 keys, fp64.  Used only to check that
 * LOOKAT reduces to it when the codebooks reproduce the keys exactly.
 */
void oracle_exact_attention(const uint16_t *q, const uint16_t *keys, const uint16_t *v, int B,
                            int H_q, int H_kv, int64_t L_max, const int32_t *seq_lens, int d_k,
                            int d_v, double scale, double *out, double *scores)
{
    int g = H_q / H_kv;
    int64_t units = (int64_t)B * H_q;
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < units; ++u) {
        int b = (int)(u / H_q), hq = (int)(u % H_q);
        int h = hq / g;
        int64_t L = seq_lens ? seq_lens[b] : L_max;
        const uint16_t *kk = keys + ((size_t)b * H_kv + h) * L_max * d_k;
        const uint16_t *vv = v + ((size_t)b * H_kv + h) * L_max * d_v;
        double *o = out + (size_t)u * d_v;
        for (int i = 0; i < d_v; ++i) o[i] = 0.0;
        if (L <= 0) continue;
        double *s = (double *)malloc(sizeof(double) * L);
        double M = -INFINITY;
        for (int64_t l = 0; l < L; ++l) {
            double acc = 0.0;
            for (int i = 0; i < d_k; ++i)
                acc += half_to_double(q[(size_t)u * d_k + i]) * half_to_double(kk[l * d_k + i]);
            s[l] = acc;
            if (scores) scores[(size_t)u * L_max + l] = acc;
            if (acc * scale > M) M = acc * scale;
        }
        double Z = 0.0;
        for (int64_t l = 0; l < L; ++l) {
            s[l] = exp(s[l] * scale - M);
            Z += s[l];
        }
        for (int64_t l = 0; l < L; ++l) {
            double a = s[l] / Z;
            for (int i = 0; i < d_v; ++i) o[i] += a * half_to_double(vv[l * d_v + i]);
        }
        free(s);
    }
}

/*
 * PQ reconstruction k_hat = concat_j C_j[code[j]] (the vector that the
 * lookup-sum of Section 3.5 scores without ever forming it).  The method
 * never does this; the oracle does, to check the lookup-sum identity.
 * k_hat fp64 [B][H_kv][L_max][d_k].
 */
void oracle_reconstruct_keys(const uint8_t *codes, int B, int H_kv, int64_t L_max, int d_k, int m,
                             int K, const float *codebooks, double *k_hat)
{
    int d_sub = d_k / m;
    for (int64_t u = 0; u < (int64_t)B * H_kv; ++u) {
        int h = (int)(u % H_kv);
        for (int64_t l = 0; l < L_max; ++l)
            for (int j = 0; j < m; ++j) {
                int c = codes[((size_t)u * L_max + l) * m + j];
                const float *cen = codebooks + (((size_t)h * m + j) * K + c) * d_sub;
                for (int i = 0; i < d_sub; ++i)
                    k_hat[((size_t)u * L_max + l) * d_k + j * d_sub + i] = (double)cen[i];
            }
    }
}

/*
 * Multi-query causal attention over the compressed keys (prefill): Algorithm 1 applied to each of
 * L_q queries per head, query i standing at position q_pos0 + i and attending tokens 0..q_pos0+i.
 * q fp16 [B][H_q][L_q][d_k]; out fp64 [B][H_q][L_q][d_v]; scores (optional) fp64
 * [B][H_q][L_q][L_max], entries beyond a query's position untouched.
 */
void oracle_attend_prefill(const uint16_t *q, const float *codebooks, const uint8_t *codes, const uint16_t *v,
                           int B, int H_q, int H_kv, int64_t L_q, int64_t L_max, int64_t q_pos0, int d_k,
                           int d_v, int m, int K, double scale, double *out, double *scores)
{
    int g = H_q / H_kv, d_sub = d_k / m;
    int64_t units = (int64_t)B * H_q * L_q;
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t u = 0; u < units; ++u) {
        int64_t i = u % L_q;
        int hq = (int)((u / L_q) % H_q), b = (int)(u / (L_q * H_q));
        int h = hq / g;
        int64_t L = q_pos0 + i + 1;
        const uint16_t *qi = q + (size_t)u * d_k;
        const uint8_t *cd = codes + ((size_t)b * H_kv + h) * L_max * m;
        const uint16_t *vv = v + ((size_t)b * H_kv + h) * L_max * d_v;
        double *o = out + (size_t)u * d_v;
        double *T = (double *)malloc(sizeof(double) * m * K);
        double *s = (double *)malloc(sizeof(double) * L);
        /* first loop of Algorithm 1: the tables of this query */
        for (int j = 0; j < m; ++j)
            for (int c = 0; c < K; ++c) {
                const float *cen = codebooks + (((size_t)h * m + j) * K + c) * d_sub;
                double acc = 0.0;
                for (int t = 0; t < d_sub; ++t) acc += half_to_double(qi[j * d_sub + t]) * (double)cen[t];
                T[j * K + c] = acc;
            }
        /* second loop and continuation */
        double M = -INFINITY;
        for (int64_t l = 0; l < L; ++l) {
            double acc = 0.0;
            for (int j = 0; j < m; ++j) acc += T[(size_t)j * K + cd[l * m + j]];
            s[l] = acc;
            if (scores) scores[(size_t)u * L_max + l] = acc;
            if (acc * scale > M) M = acc * scale;
        }
        double Z = 0.0;
        for (int64_t l = 0; l < L; ++l) {
            s[l] = exp(s[l] * scale - M);
            Z += s[l];
        }
        for (int t = 0; t < d_v; ++t) o[t] = 0.0;
        for (int64_t l = 0; l < L; ++l) {
            double a = s[l] / Z;
            for (int t = 0; t < d_v; ++t) o[t] += a * half_to_double(vv[l * d_v + t]);
        }
        free(T);
        free(s);
    }
}
