// Internal declarations shared by the translation units of liblookat.so.
// Not part of the public interface (that is include/lookat.h).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lookat.h"

namespace lookat {

// Context: configuration, stream, scratch owned by the library.
struct Ctx {
    lookat_config cfg;
    int device;
    cudaStream_t stream;
    int sm_count;
    int max_smem_optin;
    int prefill_form;          // LOOKAT_PREFILL_*
    int *timeout_flag;         // pinned, device-visible: set by a kernel whose bounded barrier wait ran out
    int *status_word;          // pinned, device-visible: LOOKAT_STATUS_* bits set by the debug build's checks
    float scale;           // resolved softmax scale
    char err[512];
    uint64_t launches;

    // attend scratch: chunk partials  o [B][H_q][splits][d_v], (M, l) [B][H_q][splits][2]
    float *part_o;
    float *part_ml;
    size_t part_o_cap, part_ml_cap;       // bytes
    unsigned *tickets;                     // attend: per-unit arrival counters, zero between launches
    size_t tickets_cap;
    // tables built on behalf of the caller (lookat_attend with lut == NULL)
    float *lut_scratch;
    size_t lut_cap;                        // bytes
    // prefill, contraction form: the codebooks as two fp16 planes (rounding, remainder), [2][H_kv][m][K][d_sub]
    __half *split_books;
    size_t split_cap;                      // bytes
    // k-means scratch
    unsigned long long *fit_sums;          // [H_kv][m][K][d_sub] fixed-point sums
    unsigned long long *fit_cnt;           // [H_kv][m][K]
    uint8_t *fit_assign;                   // [B][H_kv][n][m]
    size_t fit_sums_cap, fit_cnt_cap, fit_assign_cap;
    // decode-step staging (device copies of the host rows)
    void *step_q, *step_k;
    float *step_out;
    size_t step_q_cap, step_k_cap, step_out_cap;   // bytes

    // per-launch timing of the attend kernel: an event pair per timed launch, read only after the timed run
    int timing;
    cudaEvent_t *ev0, *ev1;    // [ev_cap]
    int ev_cap, ev_count;      // pairs created / recorded since timing was switched on
    float *times_ms;           // [ev_cap] the launches' durations, filled when the events are drained
    int n_times;
};

lookat_status set_error(Ctx *ctx, lookat_status st, const char *fmt, ...);
lookat_status check_launch(Ctx *ctx, const char *what);
lookat_status ensure(Ctx *ctx, void **ptr, size_t *cap, size_t need_bytes, const char *what);

// ---- launchers (each validates nothing: the API layer has done it) ----
// Shared memory of attend_multi_kernel, byte offsets: tables of `ut` units, the warps' partials of those units, the
// units' queries in fp64, the appended codes, the staged codebooks of one KV head (optional), the copy rings.
struct MultiLayout {
    int tables, partials, q, xk, newc, book, ring, total;
    int set_floats;                 // floats per unit in `tables`
};

struct AttendArgs {
    const float *lut;          // [B][H_q][m][K], or null: built from q and codebooks
    const __half *q;           // [B][H_q][d_k]            (used when lut is null)
    const float *codebooks;    // [H_kv][m][K][d_sub]      (used when lut is null)
    int d_k;
    int fused_lut;             // 1: the streaming kernel builds its tables itself
    unsigned *tickets;         // [n_units] arrival counters (streaming kernel)
    // append fused into the streaming kernel: the key of token new_pos of every (row, KV head) is
    // encoded by the warp that is about to copy the tile holding that token
    const __half *new_keys;    // [B][H_kv][d_k], or null
    uint8_t *codes_w;          // the code cache, writable
    int new_pos;
    const uint8_t *codes;      // [B][H_kv][L_max][m]
    const __half *v;           // [B][H_kv][L_max][d_v]
    const int32_t *seq_lens;   // [B] or null
    int uniform_len;           // tokens per row when seq_lens is null
    float *part_o;             // [B][H_q][n_splits][d_v]
    float *part_ml;            // [B][H_q][n_splits][2]
    float *scores_out;         // [B][H_q][L_max] or null
    float *out;                // [B][H_q][d_v]
    int B, H_q, H_kv, g, d_v, m, K;
    long long L_max;
    // generic kernel: one CTA per (chunk, query head, batch row)
    int chunk;                 // tokens per chunk (multiple of 16)
    int n_splits;              // chunks per row
    // streaming kernel: the (unit, 16-token tile) pairs form one flat sequence, unit =
    // (batch row, KV head, group of <= 4 query heads); CTA c owns a contiguous range of it
    int stream;                // 1: streaming kernel and its partial layout
    int n_units;
    int tiles_per_unit;        // ceil(len / 16), len = L_max with seq_lens, else the uniform length
    long long tiles_per_cta;
    int n_ctas;
    int splits_per_unit;       // > 0: CTA c = chunk c % splits of unit c / splits; 0: flat ranges
    float scale_log2;          // scale * log2(e)
    int *status;               // the context's status word (the debug build's checks; a bulk copy that never completed)
    int bulk;                  // attend_stream_kernel: tiles by cp.async.bulk + mbarrier (else 16-byte cp.async)
    // attend_multi_kernel (rows of up to a few thousand tokens): units ordered KV head first, several per round
    int multi;                 // 1: that kernel
    int ut;                    // units per round (tables resident together)
    int stage_book;            // 1: a KV head's codebooks are staged in shared memory
    int stages;                // depth of the per-warp copy rings
    int ctas_per_head;         // > 0: every KV head's tiles are cut among this many CTAs of its own; 0: one flat cut
    MultiLayout lay;           // its shared-memory layout
};

// Fills the decomposition fields of `a` (kernel choice, chunking) for n_splits as given to the
// API (0 = library's choice) and returns the partial-buffer sizes in floats.
lookat_status plan_attend(Ctx *ctx, AttendArgs &a, int n_splits, size_t *part_o_floats, size_t *part_ml_floats);
lookat_status launch_attend(Ctx *ctx, const AttendArgs &a);
lookat_status launch_combine(Ctx *ctx, const AttendArgs &a);
// attend_multi.cu: shared-memory plan (units per round, staged codebooks, ring depth) and launch
bool multi_fits(const Ctx *ctx, const AttendArgs &a);
lookat_status plan_multi(Ctx *ctx, AttendArgs &a, int ut_wanted);
lookat_status launch_multi(Ctx *ctx, const AttendArgs &a);

struct PrefillArgs {
    const __half *q;           // [B][H_q][L_q][d_k]
    const float *codebooks;    // [H_kv][m][K][d_sub]
    const uint8_t *codes;      // [B][H_kv][L_max][m]
    const __half *v;           // [B][H_kv][L_max][d_v]
    float *out;                // [B][H_q][L_q][d_v]
    float *scores_out;         // [B][H_q][L_q][L_max] or null
    int B, H_q, H_kv, g, d_k, d_v, m, K;
    long long L_q, L_max, q_pos0;
    float scale_log2;
};
lookat_status launch_prefill(Ctx *ctx, const PrefillArgs &a);
// contraction form (prefill_umma.cu): centroids gathered per chunk, scores and value sums on tcgen05 with
// accumulators in tensor memory
bool prefill_umma_covers(const Ctx *ctx, const PrefillArgs &a);
lookat_status launch_prefill_umma(Ctx *ctx, const PrefillArgs &a);
lookat_status launch_timeout_selftest(Ctx *ctx);
// decode attention with product-quantised values as well (attend_pqv.cu)
lookat_status attend_pqv_impl(Ctx *ctx, const float *lut, const uint8_t *codes, const float *v_books, const uint8_t *v_codes,
                              int m_v, int K_v, int B, long long L_max, const int32_t *seq_lens, float *out);
// read-only streaming probe (probe.cu): measurement aid
lookat_status probe_read_bandwidth(Ctx *ctx, const void *buf, size_t bytes, int reps, double *gb_per_s);

lookat_status launch_build_lut(Ctx *ctx, const __half *q, int B, const float *codebooks, float *lut);

struct EncodeArgs {
    const __half *keys;        // [B][H_kv][n][d_k]
    const float *codebooks;    // [H_kv][m][K][d_sub]
    uint8_t *codes;            // [B][H_kv][L_max][m]
    long long n, L_max, pos;
    int B;
    unsigned long long *near_ties;   // or null
    // k-means mode (all null for plain encoding)
    unsigned long long *sums;        // [H_kv][m][K][d_sub]
    unsigned long long *cnt;         // [H_kv][m][K]
    double *distortion;              // &D[0][0][it], stride (iters+1) per problem; or null
    int distortion_stride;
};
lookat_status launch_encode(Ctx *ctx, const EncodeArgs &a);
// bulk encoding with the key-by-centroid products on the tensor cores (d_sub 8, 16, 32)
bool encode_mma_covers(const Ctx *ctx, const EncodeArgs &a);
lookat_status launch_encode_mma(Ctx *ctx, const EncodeArgs &a);

lookat_status launch_fit_init(Ctx *ctx, const __half *keys, int B, long long n, uint64_t seed,
                              const float *init, float *codebooks);
lookat_status launch_fit_update(Ctx *ctx, float *codebooks);

// ---- GPT-2 decoder harness around the attention (linear_umma.cu, gpt2_ops.cu, gpt2.cu) ----
struct LinearArgs {
    const __half *bias;        // [N] or null
    const float *residual;     // fp32 [M][N] or null: added to the result (may be `out`)
    void *out;                 // [M][N] fp16 or fp32 (unused in the q/k/v form)
    int out_fp16, gelu;
    long long M;
    int N, K;
    // q/k/v form: N = 3 * d_model; row = b * T + t; third `sel`, head h, dim d of a row goes to
    // dst[sel][((b * n_head + h) * cap[sel] + off[sel] + t) * 64 + d]
    int qkv, T, n_head;
    __half *dst[3];
    long long cap[3], off[3];
    int *timeout_flag;
};
// out = act(x w_t^T + bias) [+ residual]; x [M][K] fp16 (fp32 accepted for M <= 32), w_t [N][K] fp16
// tensor maps for tiled bulk copies (linear_umma.cu): `map` points at a CUtensorMap; [rows][inner] fp16 row-major, boxes of
// box_rows x box_inner elements, 128-byte swizzle, zeros outside.  False if the driver entry point is missing or refuses.
bool tile_maps_available();
bool make_tile_map_f16(void *map, const void *base, unsigned long long inner, unsigned long long rows, unsigned box_inner,
                       unsigned box_rows);
lookat_status launch_linear(Ctx *ctx, const void *x, int x_fp32, const __half *w_t, LinearArgs p);
lookat_status launch_embed(Ctx *ctx, const int32_t *ids, const __half *wte, const __half *wpe, float *x, long long rows, int T,
                           int pos0, int d, int vocab);
lookat_status launch_layernorm(Ctx *ctx, const float *x, const __half *g, const __half *b, __half *y, long long rows, int d);
lookat_status launch_argmax(Ctx *ctx, const float *logits, int32_t *out, int rows, int n);
lookat_status launch_causal_attention(Ctx *ctx, const __half *q, const __half *k, const __half *v, __half *out, int B, int H, int T,
                                      long long v_cap);

// ---- the debug build's check of cache contents (-DLOOKAT_DEBUG): a code >= K is clamped to K - 1 before it is used as an
//      index, and a bit of the context's status word records it; lookat_last_error reports the word.  In the normal
//      build a code >= K is the caller's error and is used as it is (the streaming kernels' tables hold 256 entries per
//      subspace, so they read garbage but stay in bounds; the generic kernel reads past its table). ----
constexpr int kStatusBadCode = 1;
constexpr int kStatusCopyTimeout = 2;       // a bounded wait for a bulk copy ran out (any build)
#ifdef LOOKAT_DEBUG
__device__ __forceinline__ int checked_code(int code, int K, int *status)
{
    if (code >= K) {
        if (status) atomicOr(status, kStatusBadCode);
        return K - 1;
    }
    return code;
}
#define LOOKAT_CHECKED_CODE(code, K, status) ::lookat::checked_code((code), (K), (status))
#else
#define LOOKAT_CHECKED_CODE(code, K, status) (code)
#endif

// ---- small device helpers ----
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Every finite fp16 is an integer multiple of 2^-24; this returns that integer.
__device__ __forceinline__ long long half_to_fixed24(__half hv)
{
    unsigned short h = __half_as_ushort(hv);
    int e = (h >> 10) & 0x1f;
    long long f = h & 0x3ff;
    long long v = (e == 0) ? f : ((f | 0x400) << (e - 1));
    return (h & 0x8000) ? -v : v;
}

}  // namespace lookat
