// C ABI of liblookat.so: context management, argument validation, dispatch to
// the kernel launchers.  Every entry point is declared in include/lookat.h.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"

namespace lookat {

lookat_status set_error(Ctx *ctx, lookat_status st, const char *fmt, ...)
{
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return st;
}

lookat_status check_launch(Ctx *ctx, const char *what)
{
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess)
        return set_error(ctx, LOOKAT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return LOOKAT_OK;
}

lookat_status ensure(Ctx *ctx, void **ptr, size_t *cap, size_t need_bytes, const char *what)
{
    if (need_bytes <= *cap) return LOOKAT_OK;
    if (*ptr) {
        cudaStreamSynchronize(ctx->stream);       // earlier work may still use the old buffer
        cudaFree(*ptr);
        *ptr = nullptr;
        *cap = 0;
    }
    void *p = nullptr;
    cudaError_t e = cudaMalloc(&p, need_bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return set_error(ctx, LOOKAT_ERR_NOMEM, "%s: cudaMalloc(%zu) failed: %s", what, need_bytes,
                         cudaGetErrorString(e));
    }
    *ptr = p;
    *cap = need_bytes;
    return LOOKAT_OK;
}

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

lookat_status need_ptr(Ctx *ctx, const void *p, const char *name)
{
    if (!p) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "%s is NULL", name);
    if (!aligned16(p)) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
    return LOOKAT_OK;
}

#define LOOKAT_TRY(expr)                         \
    do {                                         \
        lookat_status st__ = (expr);             \
        if (st__ != LOOKAT_OK) return st__;      \
    } while (0)

// the device address of a pinned, mapped host buffer, or NULL if the device cannot address it
static const void *mapped_host_pointer(const void *host)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return attr.type == cudaMemoryTypeHost ? attr.devicePointer : nullptr;
}

lookat_status encode_impl(Ctx *ctx, const void *keys, int32_t B, int64_t n, const float *codebooks,
                          uint8_t *codes, int64_t L_max, int64_t pos, unsigned long long *near_ties);

lookat_status attend_impl(Ctx *ctx, const float *lut, const void *q, const float *codebooks,
                          const uint8_t *codes, const void *v, int32_t B, int64_t L_max,
                          const int32_t *seq_lens, int64_t uniform_len, int32_t n_splits, float *out,
                          float *scores_out, const void *new_keys = nullptr, uint8_t *codes_w = nullptr,
                          int64_t new_pos = 0)
{
    const lookat_config &c = ctx->cfg;
    if (B < 1 || B > 65535) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B=%d out of range 1..65535", B);
    if (L_max < 1 || L_max > (1ll << 30))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "L_max=%lld out of range", (long long)L_max);
    if (n_splits < 0) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "n_splits=%d is negative", n_splits);
    if (lut && (q || codebooks))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "give either lut or (q, codebooks), not both");
    if (!lut && !(q && codebooks))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "lut is NULL and (q, codebooks) is incomplete");
    LOOKAT_TRY(need_ptr(ctx, codes, "codes"));
    LOOKAT_TRY(need_ptr(ctx, v, "v"));
    LOOKAT_TRY(need_ptr(ctx, out, "out"));
    if (lut) LOOKAT_TRY(need_ptr(ctx, lut, "lut"));
    if (q) LOOKAT_TRY(need_ptr(ctx, q, "q"));
    if (codebooks) LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    if (seq_lens && (reinterpret_cast<uintptr_t>(seq_lens) & 3u))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "seq_lens is not 4-byte aligned");
    if (scores_out && (reinterpret_cast<uintptr_t>(scores_out) & 3u))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "scores_out is not 4-byte aligned");

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);

    if ((long long)c.n_q_heads > 65535)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "more than 65535 query heads");
    AttendArgs a;
    memset(&a, 0, sizeof(a));
    a.lut = lut;
    a.q = static_cast<const __half *>(q);
    a.codebooks = codebooks;
    a.d_k = c.d_k;
    a.codes = codes;
    a.v = static_cast<const __half *>(v);
    a.seq_lens = seq_lens;
    a.uniform_len = (int)uniform_len;
    a.scores_out = scores_out;
    a.out = out;
    a.B = B;
    a.H_q = c.n_q_heads;
    a.H_kv = c.n_kv_heads;
    a.g = c.n_q_heads / c.n_kv_heads;
    a.d_v = c.d_v;
    a.m = c.m;
    a.K = c.K;
    a.L_max = L_max;
    a.scale_log2 = ctx->scale * 1.4426950408889634f;
    a.status = ctx->status_word;
    size_t po = 0, pml = 0;
    LOOKAT_TRY(plan_attend(ctx, a, n_splits, &po, &pml));
    if (new_keys) {
        if (a.stream) {
            // the streaming kernel encodes the new key itself, just before it reads the key's tile
            a.new_keys = static_cast<const __half *>(new_keys);
            a.codes_w = codes_w;
            a.new_pos = (int)new_pos;
        } else {
            LOOKAT_TRY(encode_impl(ctx, new_keys, B, 1, codebooks, codes_w, L_max, new_pos, nullptr));
        }
    }
    if (!a.lut && !a.fused_lut) {
        // this shape builds its tables with the stand-alone kernel first
        const size_t need = (size_t)B * c.n_q_heads * c.m * c.K * sizeof(float);
        LOOKAT_TRY(ensure(ctx, (void **)&ctx->lut_scratch, &ctx->lut_cap, need, "table scratch"));
        LOOKAT_TRY(launch_build_lut(ctx, a.q, B, codebooks, ctx->lut_scratch));
        a.lut = ctx->lut_scratch;
    }
    LOOKAT_TRY(ensure(ctx, (void **)&ctx->part_o, &ctx->part_o_cap, po * sizeof(float), "partials"));
    LOOKAT_TRY(ensure(ctx, (void **)&ctx->part_ml, &ctx->part_ml_cap, pml * sizeof(float), "partials"));
    a.part_o = ctx->part_o;
    a.part_ml = ctx->part_ml;
    if (a.stream) {
        // arrival counters of the units, all zero between launches (the kernel resets them)
        const size_t need = (size_t)a.n_units * sizeof(unsigned);
        if (need > ctx->tickets_cap) {
            LOOKAT_TRY(ensure(ctx, (void **)&ctx->tickets, &ctx->tickets_cap, need, "unit counters"));
            if (cudaMemsetAsync(ctx->tickets, 0, ctx->tickets_cap, ctx->stream) != cudaSuccess)
                return set_error(ctx, LOOKAT_ERR_CUDA, "memset failed");
        }
        a.tickets = ctx->tickets;
        return launch_attend(ctx, a);
    }
    LOOKAT_TRY(launch_attend(ctx, a));
    return launch_combine(ctx, a);
}

lookat_status encode_impl(Ctx *ctx, const void *keys, int32_t B, int64_t n, const float *codebooks,
                          uint8_t *codes, int64_t L_max, int64_t pos, unsigned long long *near_ties)
{
    const lookat_config &c = ctx->cfg;
    if (B < 1 || (long long)B * c.n_kv_heads > 65535)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B*n_kv_heads=%lld out of range 1..65535",
                         (long long)B * c.n_kv_heads);
    if (n < 0 || pos < 0 || L_max < 1 || pos + n > L_max)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "need 0 <= pos, 0 <= n, pos+n <= L_max (n=%lld pos=%lld L_max=%lld)",
                         (long long)n, (long long)pos, (long long)L_max);
    if (n > (1ll << 31)) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "n too large");
    LOOKAT_TRY(need_ptr(ctx, keys, "keys"));
    LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    LOOKAT_TRY(need_ptr(ctx, codes, "codes"));
    if (near_ties && (reinterpret_cast<uintptr_t>(near_ties) & 7u))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "near_ties is not 8-byte aligned");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);
    EncodeArgs a;
    memset(&a, 0, sizeof(a));
    a.keys = static_cast<const __half *>(keys);
    a.codebooks = codebooks;
    a.codes = codes;
    a.n = n;
    a.L_max = L_max;
    a.pos = pos;
    a.B = B;
    a.near_ties = near_ties;
    return launch_encode(ctx, a);
}

}  // namespace
}  // namespace lookat

using namespace lookat;

extern "C" {

lookat_status lookat_create(const lookat_config *cfg, int device, void *cuda_stream, lookat_ctx **out)
{
    if (!cfg || !out) return LOOKAT_ERR_INVALID_ARG;
    const lookat_config &c = *cfg;
    if (c.n_q_heads < 1 || c.n_kv_heads < 1 || c.n_q_heads % c.n_kv_heads != 0) return LOOKAT_ERR_INVALID_ARG;
    if (c.d_k < 1 || c.d_k > 1024 || c.d_v < 1 || c.d_v > 1024) return LOOKAT_ERR_INVALID_ARG;
    if (c.m < 1 || c.d_k % c.m != 0) return LOOKAT_ERR_INVALID_ARG;
    if (c.K < 1 || c.K > 256) return LOOKAT_ERR_INVALID_ARG;
    if (c.d_k / c.m > 128) return LOOKAT_ERR_UNSUPPORTED;          // sub-vectors of up to 128 dims
    if (!(c.scale >= 0.f)) return LOOKAT_ERR_INVALID_ARG;          // also rejects NaN

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        cudaGetLastError();
        return LOOKAT_ERR_CUDA;
    }
    Ctx *ctx = new (std::nothrow) Ctx;
    if (!ctx) return LOOKAT_ERR_NOMEM;
    memset(ctx, 0, sizeof(Ctx));
    ctx->cfg = c;
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->scale = c.scale > 0.f ? c.scale : 1.0f / sqrtf((float)c.d_k);
    DeviceGuard guard(device);
    cudaDeviceProp prop;
    if (!guard.ok || cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return LOOKAT_ERR_CUDA;
    }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    ctx->prefill_form = LOOKAT_PREFILL_AUTO;
    if (cudaHostAlloc((void **)&ctx->timeout_flag, sizeof(int), cudaHostAllocMapped) == cudaSuccess) {
        *ctx->timeout_flag = 0;
    } else {
        cudaGetLastError();
        ctx->timeout_flag = nullptr;                       // the tcgen05 prefill kernel is then not used
    }
    if (cudaHostAlloc((void **)&ctx->status_word, sizeof(int), cudaHostAllocMapped) == cudaSuccess) {
        *ctx->status_word = 0;
    } else {
        cudaGetLastError();
        ctx->status_word = nullptr;                        // the debug build's checks then clamp without a record
    }
    *out = reinterpret_cast<lookat_ctx *>(ctx);
    return LOOKAT_OK;
}

void lookat_destroy(lookat_ctx *handle)
{
    if (!handle) return;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    DeviceGuard guard(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    void *bufs[] = {ctx->part_o, ctx->part_ml, ctx->tickets, ctx->lut_scratch, ctx->split_books, ctx->fit_sums, ctx->fit_cnt, ctx->fit_assign,
                    ctx->step_q,  ctx->step_k,  ctx->step_out};
    for (void *p : bufs)
        if (p) cudaFree(p);
    if (ctx->timeout_flag) cudaFreeHost(ctx->timeout_flag);
    if (ctx->status_word) cudaFreeHost(ctx->status_word);
    for (int i = 0; i < ctx->ev_cap; ++i) {
        if (ctx->ev0[i]) cudaEventDestroy(ctx->ev0[i]);
        if (ctx->ev1[i]) cudaEventDestroy(ctx->ev1[i]);
    }
    free(ctx->ev0);
    free(ctx->ev1);
    free(ctx->times_ms);
    cudaGetLastError();
    delete ctx;
}

const char *lookat_last_error(const lookat_ctx *handle)
{
    if (!handle) return "context is NULL";
    Ctx *ctx = const_cast<Ctx *>(reinterpret_cast<const Ctx *>(handle));
    // asynchronous findings of the debug build's device-side checks (meaningful once the caller has synchronised)
    if (ctx->status_word && *(volatile int *)ctx->status_word) {
        const int word = *(volatile int *)ctx->status_word;
        *(volatile int *)ctx->status_word = 0;
        if (word & kStatusCopyTimeout)
            snprintf(ctx->err, sizeof(ctx->err), "attend: a bounded wait for a bulk copy ran out; the output of that call is not valid");
        else
            snprintf(ctx->err, sizeof(ctx->err),
                     "debug check: a code >= K was found in a code cache and clamped to K - 1; results computed from it are not valid");
    }
    return ctx->err;
}

int32_t lookat_is_debug_build(void)
{
#ifdef LOOKAT_DEBUG
    return 1;
#else
    return 0;
#endif
}

uint64_t lookat_kernel_launches(const lookat_ctx *handle)
{
    return handle ? reinterpret_cast<const Ctx *>(handle)->launches : 0;
}

lookat_status lookat_set_prefill_form(lookat_ctx *handle, int32_t form)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (form != LOOKAT_PREFILL_AUTO && form != LOOKAT_PREFILL_TABLES && form != LOOKAT_PREFILL_CONTRACTION)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "set_prefill_form: unknown form %d", (int)form);
    ctx->prefill_form = form;
    return LOOKAT_OK;
}

lookat_status lookat_attend_pqv(lookat_ctx *handle, const float *lut, const void *q, const float *codebooks, const uint8_t *codes,
                                const float *v_codebooks, const uint8_t *v_codes, int32_t m_v, int32_t K_v, int32_t B,
                                int64_t L_max, const int32_t *seq_lens, float *out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    const lookat_config &c = ctx->cfg;
    if (B < 1 || L_max < 1 || L_max > (1ll << 31))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B=%d L_max=%lld out of range", B, (long long)L_max);
    if (!lut && !(q && codebooks))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "lut is NULL and (q, codebooks) is incomplete");
    LOOKAT_TRY(need_ptr(ctx, codes, "codes"));
    LOOKAT_TRY(need_ptr(ctx, v_codebooks, "v_codebooks"));
    LOOKAT_TRY(need_ptr(ctx, v_codes, "v_codes"));
    LOOKAT_TRY(need_ptr(ctx, out, "out"));
    if (seq_lens && (reinterpret_cast<uintptr_t>(seq_lens) & 3u))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "seq_lens is not 4-byte aligned");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);
    if (!lut) {
        LOOKAT_TRY(need_ptr(ctx, q, "q"));
        const size_t need = (size_t)B * c.n_q_heads * c.m * c.K * sizeof(float);
        LOOKAT_TRY(ensure(ctx, (void **)&ctx->lut_scratch, &ctx->lut_cap, need, "table scratch"));
        LOOKAT_TRY(launch_build_lut(ctx, static_cast<const __half *>(q), B, codebooks, ctx->lut_scratch));
        lut = ctx->lut_scratch;
    }
    return attend_pqv_impl(ctx, lut, codes, v_codebooks, v_codes, m_v, K_v, B, L_max, seq_lens, out);
}

lookat_status lookat_probe_read_bandwidth(lookat_ctx *handle, const void *buf, uint64_t bytes, int32_t reps, double *gb_per_s)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!buf || !gb_per_s || bytes < 16 || reps < 1 || ((uintptr_t)buf & 15) != 0)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "probe: need a 16-byte aligned device buffer of at least 16 bytes and reps >= 1");
    DeviceGuard guard(ctx->device);
    return probe_read_bandwidth(ctx, buf, (size_t)bytes, reps, gb_per_s);
}

lookat_status lookat_selftest_timeout(lookat_ctx *handle)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    DeviceGuard guard(ctx->device);
    return launch_timeout_selftest(ctx);
}

// the recorded event pairs into times_ms (synchronises on them)
static void drain_timing(Ctx *ctx)
{
    for (int s = 0; s < ctx->ev_count; ++s) {
        float ms = 0.f;
        cudaEventSynchronize(ctx->ev1[s]);
        if (cudaEventElapsedTime(&ms, ctx->ev0[s], ctx->ev1[s]) == cudaSuccess && ctx->n_times < ctx->ev_cap)
            ctx->times_ms[ctx->n_times++] = ms;
    }
    ctx->ev_count = 0;
}

void lookat_set_timing(lookat_ctx *handle, int32_t launches)
{
    if (!handle) return;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (launches <= 0) {
        ctx->timing = 0;
        return;
    }
    const int want = launches < 64 ? 64 : launches;
    if (want > ctx->ev_cap) {
        DeviceGuard guard(ctx->device);
        cudaEvent_t *e0 = static_cast<cudaEvent_t *>(realloc(ctx->ev0, sizeof(cudaEvent_t) * want));
        if (e0) ctx->ev0 = e0;
        cudaEvent_t *e1 = static_cast<cudaEvent_t *>(realloc(ctx->ev1, sizeof(cudaEvent_t) * want));
        if (e1) ctx->ev1 = e1;
        float *t = static_cast<float *>(realloc(ctx->times_ms, sizeof(float) * want));
        if (t) ctx->times_ms = t;
        if (e0 && e1 && t) {
            while (ctx->ev_cap < want) {
                ctx->ev0[ctx->ev_cap] = ctx->ev1[ctx->ev_cap] = nullptr;
                if (cudaEventCreate(&ctx->ev0[ctx->ev_cap]) != cudaSuccess || cudaEventCreate(&ctx->ev1[ctx->ev_cap]) != cudaSuccess) {
                    cudaGetLastError();
                    if (ctx->ev0[ctx->ev_cap]) cudaEventDestroy(ctx->ev0[ctx->ev_cap]);
                    break;                                 // fewer launches are timed than asked for
                }
                ctx->ev_cap += 1;
            }
        }
    }
    ctx->ev_count = 0;
    ctx->n_times = 0;
    ctx->timing = 1;
}

double lookat_attend_kernel_ms(lookat_ctx *handle)
{
    double st[4];
    return lookat_attend_kernel_stats(handle, st) > 0 ? st[3] : -1.0;
}

int32_t lookat_attend_kernel_stats(lookat_ctx *handle, double *stats)
{
    if (!handle || !stats) return 0;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    DeviceGuard guard(ctx->device);
    drain_timing(ctx);
    const int n = ctx->n_times;
    if (n == 0) return 0;
    // insertion sort of a copy would do; the array is small and owned: sort in place
    float *t = ctx->times_ms;
    for (int i = 1; i < n; ++i) {
        const float v = t[i];
        int k = i - 1;
        while (k >= 0 && t[k] > v) { t[k + 1] = t[k]; --k; }
        t[k + 1] = v;
    }
    double sum = 0.0;
    for (int i = 0; i < n; ++i) sum += t[i];
    stats[0] = t[0];
    stats[1] = (n & 1) ? t[n / 2] : 0.5 * ((double)t[n / 2 - 1] + t[n / 2]);
    stats[2] = t[n - 1];
    stats[3] = sum / n;
    return n;
}

lookat_status lookat_build_lut(lookat_ctx *handle, const void *q, int32_t B, const float *codebooks, float *lut)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (B < 1 || B > 65535) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B=%d out of range 1..65535", B);
    if (ctx->cfg.n_q_heads > 65535) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "more than 65535 query heads");
    LOOKAT_TRY(need_ptr(ctx, q, "q"));
    LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    LOOKAT_TRY(need_ptr(ctx, lut, "lut"));
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);
    return launch_build_lut(ctx, static_cast<const __half *>(q), B, codebooks, lut);
}

lookat_status lookat_attend(lookat_ctx *handle, const float *lut, const void *q, const float *codebooks,
                            const uint8_t *codes, const void *v, int32_t B, int64_t L_max,
                            const int32_t *seq_lens, int32_t n_splits, float *out, float *scores_out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    return attend_impl(reinterpret_cast<Ctx *>(handle), lut, q, codebooks, codes, v, B, L_max, seq_lens, L_max,
                       n_splits, out, scores_out);
}

lookat_status lookat_encode_keys(lookat_ctx *handle, const void *keys, int32_t B, int64_t n,
                                 const float *codebooks, uint8_t *codes, int64_t L_max, int64_t pos,
                                 unsigned long long *near_ties)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    return encode_impl(reinterpret_cast<Ctx *>(handle), keys, B, n, codebooks, codes, L_max, pos, near_ties);
}

lookat_status lookat_fit_codebooks(lookat_ctx *handle, const void *keys, int32_t B, int64_t n, int32_t iters,
                                   uint64_t seed, const float *init, float *codebooks, double *distortion)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    const lookat_config &c = ctx->cfg;
    if (B < 1 || (long long)B * c.n_kv_heads > 65535)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B*n_kv_heads out of range 1..65535");
    if (n < 1 || (long long)B * n > (1ll << 22))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "need 1 <= B*n <= 2^22 keys per head (B*n=%lld)",
                         (long long)B * n);
    if (iters < 0 || iters > 100000) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "iters=%d out of range", iters);
    LOOKAT_TRY(need_ptr(ctx, keys, "keys"));
    LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    if (init) LOOKAT_TRY(need_ptr(ctx, init, "init"));
    if (distortion && (reinterpret_cast<uintptr_t>(distortion) & 7u))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "distortion is not 8-byte aligned");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);

    const int d_sub = c.d_k / c.m;
    const size_t clusters = (size_t)c.n_kv_heads * c.m * c.K;
    const bool fresh_sums = clusters * d_sub * 8 > ctx->fit_sums_cap;
    const bool fresh_cnt = clusters * 8 > ctx->fit_cnt_cap;
    LOOKAT_TRY(ensure(ctx, (void **)&ctx->fit_sums, &ctx->fit_sums_cap, clusters * d_sub * 8, "k-means sums"));
    LOOKAT_TRY(ensure(ctx, (void **)&ctx->fit_cnt, &ctx->fit_cnt_cap, clusters * 8, "k-means counts"));
    LOOKAT_TRY(ensure(ctx, (void **)&ctx->fit_assign, &ctx->fit_assign_cap,
                      (size_t)B * c.n_kv_heads * n * c.m, "k-means assignments"));
    // sums and counts are left at zero by every update; fresh buffers are cleared here
    if (fresh_sums && cudaMemsetAsync(ctx->fit_sums, 0, ctx->fit_sums_cap, ctx->stream) != cudaSuccess)
        return set_error(ctx, LOOKAT_ERR_CUDA, "memset failed");
    if (fresh_cnt && cudaMemsetAsync(ctx->fit_cnt, 0, ctx->fit_cnt_cap, ctx->stream) != cudaSuccess)
        return set_error(ctx, LOOKAT_ERR_CUDA, "memset failed");
    if (distortion &&
        cudaMemsetAsync(distortion, 0, (size_t)c.n_kv_heads * c.m * (iters + 1) * sizeof(double), ctx->stream) !=
            cudaSuccess)
        return set_error(ctx, LOOKAT_ERR_CUDA, "memset failed");

    LOOKAT_TRY(launch_fit_init(ctx, static_cast<const __half *>(keys), B, n, seed, init, codebooks));
    for (int it = 0; it <= iters; ++it) {
        const bool last = it == iters;
        if (last && !distortion) break;                   // the closing pass only measures
        EncodeArgs a;
        memset(&a, 0, sizeof(a));
        a.keys = static_cast<const __half *>(keys);
        a.codebooks = codebooks;
        a.codes = ctx->fit_assign;
        a.n = n;
        a.L_max = n;
        a.pos = 0;
        a.B = B;
        a.sums = ctx->fit_sums;
        a.cnt = ctx->fit_cnt;
        a.distortion = distortion ? distortion + it : nullptr;
        a.distortion_stride = iters + 1;
        LOOKAT_TRY(launch_encode(ctx, a));
        // the closing pass also filled the sums; the update below only clears them then
        LOOKAT_TRY(launch_fit_update(ctx, last ? nullptr : codebooks));
    }
    return LOOKAT_OK;
}

lookat_status lookat_attend_prefill(lookat_ctx *handle, const void *q, const float *codebooks, const uint8_t *codes,
                                    const void *v, int32_t B, int64_t L_q, int64_t L_max, int64_t q_pos0, float *out,
                                    float *scores_out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    const lookat_config &c = ctx->cfg;
    if (ctx->timeout_flag && *(volatile int *)ctx->timeout_flag) {
        *(volatile int *)ctx->timeout_flag = 0;
        return set_error(ctx, LOOKAT_ERR_TIMEOUT,
                         "an earlier attend_prefill kernel gave up a bounded barrier wait; its output is not valid");
    }
    if (B < 1 || B > 65535) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B=%d out of range 1..65535", B);
    if (c.n_q_heads > 65535) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "more than 65535 query heads");
    if (L_q < 1 || L_max < 1 || q_pos0 < 0 || q_pos0 + L_q > L_max || L_max > (1ll << 30))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG,
                         "need 1 <= L_q, 0 <= q_pos0, q_pos0 + L_q <= L_max (L_q=%lld q_pos0=%lld L_max=%lld)",
                         (long long)L_q, (long long)q_pos0, (long long)L_max);
    LOOKAT_TRY(need_ptr(ctx, q, "q"));
    LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    LOOKAT_TRY(need_ptr(ctx, codes, "codes"));
    LOOKAT_TRY(need_ptr(ctx, v, "v"));
    LOOKAT_TRY(need_ptr(ctx, out, "out"));
    if (scores_out && (reinterpret_cast<uintptr_t>(scores_out) & 3u))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "scores_out is not 4-byte aligned");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);
    PrefillArgs a;
    memset(&a, 0, sizeof(a));
    a.q = static_cast<const __half *>(q);
    a.codebooks = codebooks;
    a.codes = codes;
    a.v = static_cast<const __half *>(v);
    a.out = out;
    a.scores_out = scores_out;
    a.B = B;
    a.H_q = c.n_q_heads;
    a.H_kv = c.n_kv_heads;
    a.g = c.n_q_heads / c.n_kv_heads;
    a.d_k = c.d_k;
    a.d_v = c.d_v;
    a.m = c.m;
    a.K = c.K;
    a.L_q = L_q;
    a.L_max = L_max;
    a.q_pos0 = q_pos0;
    a.scale_log2 = ctx->scale * 1.4426950408889634f;
    return launch_prefill(ctx, a);
}

lookat_status lookat_decode_step(lookat_ctx *handle, const void *q, const void *k_new, const float *codebooks,
                                 uint8_t *codes, const void *v, int32_t B, int64_t L_max, int64_t pos,
                                 int32_t n_splits, float *out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (pos < 0 || pos >= L_max)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "need 0 <= pos < L_max (pos=%lld L_max=%lld)", (long long)pos,
                         (long long)L_max);
    LOOKAT_TRY(need_ptr(ctx, k_new, "k_new"));
    LOOKAT_TRY(need_ptr(ctx, q, "q"));
    LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    return attend_impl(ctx, nullptr, q, codebooks, codes, v, B, L_max, nullptr, pos + 1, n_splits, out, nullptr,
                       k_new, codes, pos);
}

lookat_status lookat_decode_step_host(lookat_ctx *handle, const void *q_host, const void *k_new_host,
                                      const void *v_new_host, int32_t B, const float *codebooks, uint8_t *codes,
                                      void *v, int64_t L_max, int64_t pos, int32_t n_splits, float *out_host)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    const lookat_config &c = ctx->cfg;
    if (!q_host || !k_new_host || !v_new_host || !out_host)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "a host buffer is NULL");
    if (B < 1 || B > 65535) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B=%d out of range", B);
    if (pos < 0 || pos >= L_max)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "need 0 <= pos < L_max (pos=%lld L_max=%lld)", (long long)pos,
                         (long long)L_max);
    LOOKAT_TRY(need_ptr(ctx, codebooks, "codebooks"));
    LOOKAT_TRY(need_ptr(ctx, codes, "codes"));
    LOOKAT_TRY(need_ptr(ctx, v, "v"));
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);

    const size_t q_bytes = (size_t)B * c.n_q_heads * c.d_k * 2;
    const size_t k_bytes = (size_t)B * c.n_kv_heads * c.d_k * 2;
    const size_t v_row = (size_t)c.d_v * 2;
    const size_t out_bytes = (size_t)B * c.n_q_heads * c.d_v * 4;
    LOOKAT_TRY(ensure(ctx, &ctx->step_q, &ctx->step_q_cap, q_bytes, "step staging"));
    LOOKAT_TRY(ensure(ctx, &ctx->step_k, &ctx->step_k_cap, k_bytes, "step staging"));
    LOOKAT_TRY(ensure(ctx, (void **)&ctx->step_out, &ctx->step_out_cap, out_bytes, "step staging"));

    cudaStream_t s = ctx->stream;
    // Pinned host buffers that the device can address (any cudaHostAlloc / registered memory under unified
    // addressing) are read and written by the kernel itself: the queries and new keys cross the bus while the first
    // tiles are already streaming, the output rows are posted by the merging CTAs, and three copies leave the stream.
    const void *q_dev = mapped_host_pointer(q_host), *k_dev = mapped_host_pointer(k_new_host);
    float *out_dev = static_cast<float *>(const_cast<void *>(mapped_host_pointer(out_host)));
    const bool direct = q_dev && k_dev && out_dev && ((uintptr_t)q_dev & 15) == 0 && ((uintptr_t)k_dev & 15) == 0 &&
                        ((uintptr_t)out_dev & 15) == 0;
    cudaError_t e = cudaSuccess;
    if (!direct) {
        e = cudaMemcpyAsync(ctx->step_q, q_host, q_bytes, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->step_k, k_new_host, k_bytes, cudaMemcpyHostToDevice, s);
    }
    // value rows go straight into the cache: B*H_kv rows of d_v halves, one per (b, h), at token pos
    if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(static_cast<char *>(v) + (size_t)pos * v_row, (size_t)L_max * v_row, v_new_host, v_row,
                              v_row, (size_t)B * c.n_kv_heads, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return set_error(ctx, LOOKAT_ERR_CUDA, "host-to-device copy: %s", cudaGetErrorString(e));

    // append + attend over tokens 0..pos of every row, one launch where the shape allows
    LOOKAT_TRY(attend_impl(ctx, nullptr, direct ? q_dev : ctx->step_q, codebooks, codes, v, B, L_max, nullptr, pos + 1, n_splits,
                           direct ? out_dev : ctx->step_out, nullptr, direct ? k_dev : ctx->step_k, codes, pos));
    if (!direct) e = cudaMemcpyAsync(out_host, ctx->step_out, out_bytes, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return set_error(ctx, LOOKAT_ERR_CUDA, "device-to-host copy: %s", cudaGetErrorString(e));
    return LOOKAT_OK;
}

}  // extern "C"
