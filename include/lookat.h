/*
 * lookat.h - C ABI of the B200 (sm_100a) LOOKAT library: decode-time attention
 * whose keys are stored only as product-quantisation codes.
 *
 * The four operations follow the paper's statement of the method:
 *   lookat_fit_codebooks  Section 3.4 "Prototype Learning" (k-means per subspace)
 *   lookat_encode_keys    Section 3.4 "Encoding" (nearest centroid per subspace)
 *   lookat_build_lut      Section 3.5 "Precomputation Lookup Tables", Algorithm 1 loop 1
 *   lookat_attend         Section 3.5 "Lookup and Sum", Algorithm 1 loop 2 + softmax + value sum
 *
 * Symbols: B batch, H_q query heads, H_kv KV heads, g = H_q / H_kv, L cached
 * tokens, d_k / d_v head dims, m subspaces, d_sub = d_k / m, K centroids (<= 256).
 * Query head hq uses the codebooks, codes and values of KV head hq / g.
 *
 * Memory: every data pointer is DEVICE memory owned by the caller unless its
 * comment says host; the library reads or writes it in stream order on the
 * context's stream and keeps no reference after the call's work completes.
 * Arrays are dense, row-major, innermost dimension last.  Pointers must be
 * aligned to 16 bytes (what cudaMalloc and torch allocations give).
 * The context owns scratch (chunk partials, a table buffer, k-means sums);
 * it grows on demand, which allocates: call once at full size before timing.
 *
 * Errors: every call returns a lookat_status and launches nothing when it
 * rejects its arguments.  Calls do not synchronise; asynchronous CUDA errors
 * surface at the caller's next synchronisation.  There is no CPU fallback.
 */
#ifndef LOOKAT_H
#define LOOKAT_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lookat_ctx lookat_ctx;

typedef enum {
    LOOKAT_OK = 0,
    LOOKAT_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, bad shape, out-of-range size */
    LOOKAT_ERR_UNSUPPORTED = 2,   /* valid but not implemented for this shape */
    LOOKAT_ERR_CUDA = 3,          /* a CUDA runtime call failed; see lookat_last_error */
    LOOKAT_ERR_NOMEM = 4,         /* scratch allocation failed */
    LOOKAT_ERR_TIMEOUT = 5        /* a bounded device-side wait expired (reported by the next lookat_attend_prefill) */
} lookat_status;

typedef struct {
    int32_t n_q_heads;   /* H_q */
    int32_t n_kv_heads;  /* H_kv, divides H_q */
    int32_t d_k;         /* key / query head dim */
    int32_t d_v;         /* value head dim */
    int32_t m;           /* subspaces, divides d_k */
    int32_t K;           /* centroids per subspace, 1..256 (codes are uint8) */
    float scale;         /* softmax scale; 0 selects 1/sqrt(d_k) (Algorithm 1) */
} lookat_config;

/* Creates a context bound to CUDA device `device` and to `cuda_stream` (a
 * cudaStream_t passed as void*; NULL = the default stream).  *out is set only
 * on success.  Destroy frees the scratch; NULL is accepted. */
lookat_status lookat_create(const lookat_config *cfg, int device, void *cuda_stream, lookat_ctx **out);
void lookat_destroy(lookat_ctx *ctx);

/* Host string describing the last error this context returned ("" if none).  In the debug build of the library
 * (compiled with -DLOOKAT_DEBUG, liblookat_debug.so) the attend kernels check every code they read from a cache:
 * a code >= K is clamped to K - 1 before it is used as an index and the finding is recorded in a status word of the
 * context; after the caller has synchronised the stream, this call reports it once.  The normal build does not
 * check: a code >= K there is the caller's error (the streaming kernels then read garbage inside their tables, the
 * any-shape kernel reads past the table). */
const char *lookat_last_error(const lookat_ctx *ctx);

/* 1 in the debug build of the library, 0 otherwise. */
int32_t lookat_is_debug_build(void);

/* One environment variable is read, for tests: with LOOKAT_NO_TENSOR_MAPS set, the long-row attend kernel fetches its
 * tiles by 16-byte cp.async pieces instead of tiled bulk copies -- the path it otherwise takes only where the driver has
 * no tensor-map entry point or the caches have 2^31 rows or more.  Same results, slower. */

/*
 * Section 3.4, Prototype Learning: for every KV head h and subspace j, a
 * K-centroid codebook minimising  sum_k min_c || k^(j) - c ||^2  over the
 * given keys, by `iters` Lloyd iterations (no early stop).
 *
 *   keys        fp16 [B][H_kv][n][d_k]; the N = B*n keys of a head are pooled,
 *               pooled index = b*n + t.  N <= 2^22.
 *   init        NULL, or fp32 [H_kv][m][K][d_sub] starting centroids.
 *               NULL: centroid c starts at pooled row (off + c*stride) mod N,
 *               off = (seed + 0x9E3779B97F4A7C15*(h*m+j+1)) mod 2^64 mod N,
 *               stride = max(1, N/K).  (The paper fixes no initialisation.)
 *   codebooks   out, fp32 [H_kv][m][K][d_sub].
 *   distortion  NULL, or out fp64 [H_kv][m][iters+1]: the objective before
 *               each update and after the last.
 * Assignment takes the lowest index among equal minima.  The update is the
 * exact mean (64-bit fixed-point sums, one fp64 division, rounded to fp32);
 * an empty cluster keeps its centroid.
 */
lookat_status lookat_fit_codebooks(lookat_ctx *ctx, const void *keys, int32_t B, int64_t n,
                                   int32_t iters, uint64_t seed, const float *init,
                                   float *codebooks, double *distortion);

/*
 * Section 3.4, Encoding: code[t][j] = argmin_c || k_t^(j) - C_j[c] ||^2,
 * lowest index on ties, for n new keys per (batch, KV head), written at token
 * offset pos of the code cache.
 *
 *   keys       fp16 [B][H_kv][n][d_k]
 *   codebooks  fp32 [H_kv][m][K][d_sub]
 *   codes      in/out, uint8 [B][H_kv][L_max][m]; rows pos..pos+n-1 are written
 *   near_ties  NULL, or in/out uint64[1]: incremented once per (key, subspace)
 *              whose best and second-best distance differ by a relative gap in
 *              (0, 1e-6) as evaluated in fp64.
 * Codes equal the fp64 argmin of the difference-form distance.  Bulk calls
 * (d_sub 8, 16 or 32) search on the tensor cores (fp16 planes, fp32
 * accumulation) and accept a winner only beyond a proven error margin; every
 * other key, and every shape the tensor-core search does not cover (searched in
 * fp32, accepted beyond a 1e-4 relative margin), is re-decided in fp64.
 * Requires pos >= 0, pos + n <= L_max.
 */
lookat_status lookat_encode_keys(lookat_ctx *ctx, const void *keys, int32_t B, int64_t n,
                                 const float *codebooks, uint8_t *codes, int64_t L_max, int64_t pos,
                                 unsigned long long *near_ties);

/*
 * Section 3.5, Precomputation Lookup Tables (Algorithm 1, first loop):
 *   lut[b][hq][j][c] = sum_i q[b][hq][j*d_sub+i] * C[hq/g][j][c][i]     (unscaled)
 *
 *   q    fp16 [B][H_q][d_k]
 *   lut  out, fp32 [B][H_q][m][K]; products are accumulated in fp64 and
 *        rounded once.
 */
lookat_status lookat_build_lut(lookat_ctx *ctx, const void *q, int32_t B, const float *codebooks,
                               float *lut);

/*
 * Section 3.5, Lookup and Sum, and the continuation of Algorithm 1:
 *   s_t = sum_j lut[j][code[t][j]],  alpha = softmax(s * scale),  o = sum_t alpha_t v_t
 * over t < seq_len, computed per sequence chunk with a running maximum and a
 * final merge of the chunk partials.  Keys are never reconstructed.
 *
 * Exactly one of `lut` or (`q`, `codebooks`) is given; with lut == NULL the
 * tables are built first into context scratch.
 *   codes       uint8 [B][H_kv][L_max][m], every code < K (not checked)
 *   v           fp16 [B][H_kv][L_max][d_v]
 *   seq_lens    NULL (all rows use L_max tokens) or int32 [B], 0..L_max
 *   n_splits    chunks per sequence; 0 = chosen by the library
 *   out         fp32 [B][H_q][d_v]; a row with seq_len 0 gives zeros
 *   scores_out  NULL, or fp32 [B][H_q][L_max] raw unscaled s_t for t < seq_len
 *               (for validation; costs extra writes)
 */
lookat_status lookat_attend(lookat_ctx *ctx, const float *lut, const void *q, const float *codebooks,
                            const uint8_t *codes, const void *v, int32_t B, int64_t L_max,
                            const int32_t *seq_lens, int32_t n_splits, float *out, float *scores_out);

/*
 * lookat_attend without any allocation.  (The paper has no counterpart: it is
 * an interface variant of lookat_attend, same arguments, same results.)
 *
 * For callers that cannot let a library call cudaMalloc / cudaFree: a serving
 * process whose own pool owns all device memory, or a decode loop that cannot
 * afford the device-wide synchronisation those calls imply.  The partial
 * results and the per-unit counters of the attend kernel live in a fixed
 * device array inside the library (2 MiB + 64 KiB + 16 KiB, held by every GPU
 * that loads the library until the process exits) instead of context scratch.
 *
 * Limits: (CTAs launched + B*H_kv*ceil(g/4)) * 4 * d_v floats of partials must
 * fit in 2 MiB (524,288 floats) and B*H_kv*ceil(g/4) <= 4096; with the
 * library's own chunking (n_splits = 0) the CTA count is at most a few per SM.
 * A problem beyond that returns LOOKAT_ERR_UNSUPPORTED and launches nothing,
 * as does a shape whose tables cannot be built inside the kernel when lut is
 * NULL (pass ready tables then).
 *
 * The first call on a device looks up the device address of the array; make
 * that first call before starting a stream capture.  The array and the kernel
 * images take their device memory when the CUDA runtime loads the library's
 * module on that device, which under the default lazy loading can be as late
 * as this first call: a process that hands the whole device to its own pool
 * must make one warm-up call (or run with CUDA_MODULE_LOADING=EAGER) BEFORE the
 * pool takes the memory, else that first call can return LOOKAT_ERR_CUDA.
 * All calls share the array: two calls whose kernels overlap on the GPU
 * (different streams or contexts, same device) race on it and give wrong
 * results; calls on one stream are safe.  The counters are cleared at every
 * call, so a call cut short by an error leaves nothing behind.
 */
lookat_status lookat_attend_static(lookat_ctx *ctx, const float *lut, const void *q, const float *codebooks,
                                   const uint8_t *codes, const void *v, int32_t B, int64_t L_max,
                                   const int32_t *seq_lens, int32_t n_splits, float *out, float *scores_out);

/*
 * Multi-query causal attention over the compressed keys (prefill): Algorithm
 * 1 for each of L_q consecutive queries per head.  Query i stands at position
 * q_pos0 + i and attends tokens 0 .. q_pos0 + i of the cache (its own
 * quantised key included, so the keys up to q_pos0 + L_q - 1 must have been
 * encoded).  The tables of a tile of queries are built on chip.
 *
 *   q           fp16 [B][H_q][L_q][d_k]
 *   codes       uint8 [B][H_kv][L_max][m]
 *   v           fp16 [B][H_kv][L_max][d_v]
 *   out         fp32 [B][H_q][L_q][d_v]
 *   scores_out  NULL, or fp32 [B][H_q][L_q][L_max]: raw unscaled s for the
 *               visible (query, token) pairs (validation only)
 * Requires 0 <= q_pos0, q_pos0 + L_q <= L_max.  d_v must be a multiple of 32
 * (of 16 where tables of 16 queries fit in shared memory) and at most 256;
 * otherwise LOOKAT_ERR_UNSUPPORTED.
 */
lookat_status lookat_attend_prefill(lookat_ctx *ctx, const void *q, const float *codebooks, const uint8_t *codes,
                                    const void *v, int32_t B, int64_t L_q, int64_t L_max, int64_t q_pos0,
                                    float *out, float *scores_out);

/*
 * One decode step on device buffers: append and attend.  The new key of every
 * (batch row, KV head) is encoded at token `pos` of the code cache (Section
 * 3.4, Encoding), then Algorithm 1 runs over tokens 0..pos with tables built
 * from q and the codebooks.  Same results as lookat_encode_keys(n = 1, pos)
 * followed by lookat_attend with every row at pos+1 tokens; where the
 * streaming attend kernel covers the shape, both happen in one launch (the
 * warp that is about to read the tile holding token `pos` encodes the key
 * first).  The value row of token `pos` must already be in the V cache.
 *
 *   q          fp16 [B][H_q][d_k]
 *   k_new      fp16 [B][H_kv][d_k]
 *   codes      in/out, uint8 [B][H_kv][L_max][m]; row pos is written
 *   v          fp16 [B][H_kv][L_max][d_v]
 *   out        fp32 [B][H_q][d_v]
 * Requires 0 <= pos < L_max.
 */
lookat_status lookat_decode_step(lookat_ctx *ctx, const void *q, const void *k_new, const float *codebooks,
                                 uint8_t *codes, const void *v, int32_t B, int64_t L_max, int64_t pos,
                                 int32_t n_splits, float *out);

/*
 * One decode step driven from HOST buffers (what a serving loop that keeps
 * its activations on the host calls): copies the step's query, new key and
 * new value rows to the device, encodes the new key at token `pos`
 * (Section 3.4), stores the value row there, attends over tokens 0..pos
 * (Algorithm 1) and copies the output back.  All on the context's stream;
 * the call returns after the output has arrived (it synchronises the stream).
 *
 *   q_host      host fp16 [B][H_q][d_k]          (pinned memory for speed: when
 *               q_host, k_new_host and out_host are pinned, 16-byte aligned and
 *               addressable by the device, the kernel reads and writes them in
 *               place and only the value rows are copied)
 *   k_new_host  host fp16 [B][H_kv][d_k]
 *   v_new_host  host fp16 [B][H_kv][d_v]
 *   codebooks   device fp32 [H_kv][m][K][d_sub]
 *   codes       device uint8 [B][H_kv][L_max][m]  (row pos is written)
 *   v           device fp16 [B][H_kv][L_max][d_v] (row pos is written)
 *   out_host    host fp32 [B][H_q][d_v]
 * Requires 0 <= pos < L_max.
 */
lookat_status lookat_decode_step_host(lookat_ctx *ctx, const void *q_host, const void *k_new_host,
                                      const void *v_new_host, int32_t B, const float *codebooks,
                                      uint8_t *codes, void *v, int64_t L_max, int64_t pos,
                                      int32_t n_splits, float *out_host);

/*
 * Which of its two kernels lookat_attend_prefill uses.  Both compute Algorithm
 * 1 for every query; they differ in how the score of Section 3.5 ("Lookup and Sum") is formed:
 *   LOOKAT_PREFILL_TABLES       per-query tables built on chip, then m lookups
 *                               per (query, token) pair (any shape);
 *   LOOKAT_PREFILL_CONTRACTION  the centroids named by a chunk of codes are
 *                               gathered once per 256 queries and the scores
 *                               taken as q . (C_1[c_1], ..., C_m[c_m]) on the
 *                               tensor cores (d_k and d_v in {64, 128}, d_sub 4
 *                               or a multiple of 8, both codebook planes of a head
 *                               in shared memory: K * d_k * 4 bytes; L_max * m a
 *                               multiple of 4); tcgen05.mma with accumulators
 *                               in tensor memory;
 *   LOOKAT_PREFILL_AUTO         (default) contraction where it applies and
 *                               L_q >= 32, tables otherwise.
 * Asking for the contraction form on a shape it does not cover makes
 * lookat_attend_prefill return LOOKAT_ERR_UNSUPPORTED.  Returns
 * LOOKAT_ERR_INVALID_ARG for an unknown value.
 */
enum {
    LOOKAT_PREFILL_AUTO = 0,
    LOOKAT_PREFILL_TABLES = 1,
    LOOKAT_PREFILL_CONTRACTION = 2
};
lookat_status lookat_set_prefill_form(lookat_ctx *ctx, int32_t form);

/*
 * Decode attention with product-quantised VALUES as well.  The paper leaves
 * value compression to future work (Section 5.2); the formulation is this
 * build's own.  The weights alpha are those of Algorithm 1 (scores from the
 * key codes, softmax(s * scale)); the output is o = sum_t alpha_t v^_t with
 * v^_t the value centroids named by the value codes, taken per value subspace
 * as sum_c w[j][c] C^V_j[c], w = the histogram of the weights over the codes.
 * Per token only m + m_v bytes are read.  Value codebooks and codes come from
 * lookat_fit_codebooks / lookat_encode_keys of a context configured with
 * d_k = this context's d_v and m = m_v (values are encoded like keys).
 *
 *   lut          NULL or device fp32 [B][H_q][m][K]; with NULL the tables are
 *                built from q (fp16 [B][H_q][d_k]) and codebooks first
 *   codes        device uint8 [B][H_kv][L_max][m]      (aligned to m bytes)
 *   v_codebooks  device fp32 [H_kv][m_v][K_v][d_v / m_v]
 *   v_codes      device uint8 [B][H_kv][L_max][m_v]    (aligned to m_v bytes)
 *   seq_lens     NULL (all L_max) or device int32 [B], 0..L_max; a row with 0 tokens gives zeros
 *   out          device fp32 [B][H_q][d_v]
 * m and m_v must be 2, 4, 8 or 16 (else LOOKAT_ERR_UNSUPPORTED); K_v <= 256.
 */
lookat_status lookat_attend_pqv(lookat_ctx *ctx, const float *lut, const void *q, const float *codebooks,
                                const uint8_t *codes, const float *v_codebooks, const uint8_t *v_codes, int32_t m_v,
                                int32_t K_v, int32_t B, int64_t L_max, const int32_t *seq_lens, float *out);

/*
 * Measurement aid (the paper has no counterpart): reads `bytes` of the device
 * buffer `buf` (16-byte aligned) `reps` times with a read-only streaming kernel
 * on the context's stream, one untimed pass first, and returns the bandwidth in
 * GB/s (CUDA events around the timed passes; the call synchronises on them).
 * bench.py reports it beside the attend kernel's bandwidth as the read ceiling
 * of the GPU it ran on.
 */
lookat_status lookat_probe_read_bandwidth(lookat_ctx *ctx, const void *buf, uint64_t bytes, int32_t reps,
                                          double *gb_per_s);

/*
 * Self-test of the time-out status: launches a one-warp kernel whose only wait
 * can never be satisfied and gives up after 4096 polls (it ends by itself in
 * microseconds; nothing hangs), raising the context's time-out flag exactly as
 * a prefill kernel would.  After the stream has drained, the next
 * lookat_attend_prefill returns LOOKAT_ERR_TIMEOUT once and clears the flag.
 * The paper has no counterpart.
 */
lookat_status lookat_selftest_timeout(lookat_ctx *ctx);

/* Number of kernels this context has launched since it was created. */
uint64_t lookat_kernel_launches(const lookat_ctx *ctx);

/* Device time of the attend kernel per launch (measurement aid; the paper has
 * no counterpart): CUDA events on the context's stream around every launch
 * made while timing is on, read only afterwards, so the timed run itself is
 * never synchronised.  lookat_set_timing(ctx, n) with n >= 1 resets and starts
 * with room for n launches (at least 64; later launches go untimed), n <= 0
 * stops.  lookat_attend_kernel_stats synchronises on the recorded events and
 * fills stats[0..3] = minimum, median, maximum and mean in milliseconds; it
 * returns the number of launches timed (0: stats untouched).
 * lookat_attend_kernel_ms returns that mean, or -1 when nothing was timed. */
void lookat_set_timing(lookat_ctx *ctx, int32_t launches);
double lookat_attend_kernel_ms(lookat_ctx *ctx);
int32_t lookat_attend_kernel_stats(lookat_ctx *ctx, double *stats);

#ifdef __cplusplus
}
#endif
#endif /* LOOKAT_H */
