// lookat_attend_static: lookat_attend for callers that must not allocate.
//
// Who needs it: a serving process that has handed the whole device to its own
// memory pool (so a cudaMalloc from a library either fails or steals from the
// pool), and decode loops that cannot take the device-wide synchronisation a
// cudaMalloc / cudaFree implies while other streams are running.  For them the
// partial results and the per-unit arrival counters of the attend kernel live
// in the fixed device array below instead of in scratch the context grows on
// demand.  The price: the array has a fixed size (problems whose partials do
// not fit are rejected), every GPU that loads the library carries it until the
// process exits, and all calls share it.
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace lookat {
namespace {

// Layout of the fixed scratch, in bytes; each part starts on a 256-byte boundary.
constexpr size_t kStaticPartOBytes = 2u << 20;     // weighted-value partials: 524,288 floats
constexpr size_t kStaticPartMlBytes = 64u << 10;   // (max, sum) partials:       16,384 floats
constexpr size_t kStaticTicketBytes = 16u << 10;   // arrival counters:           4,096 units
constexpr size_t kStaticBytes = kStaticPartOBytes + kStaticPartMlBytes + kStaticTicketBytes;

static __device__ __align__(256) unsigned char lookat_static_scratch[kStaticBytes];

// In host code `lookat_static_scratch` is only a handle for the runtime, not a device address:
// the address each device gave the array is looked up once per device and kept here.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char *g_scratch_on_device[kMaxDevices] = {};

lookat_status static_scratch(Ctx *ctx, unsigned char **out)
{
    if (ctx->device < 0 || ctx->device >= kMaxDevices)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "lookat_attend_static: device index %d beyond %d",
                         ctx->device, kMaxDevices - 1);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_on_device[ctx->device]) {
        // the caller has made ctx->device current
        unsigned char *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&ptr, lookat_static_scratch);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            return set_error(ctx, LOOKAT_ERR_CUDA, "lookat_attend_static: cudaGetSymbolAddress failed: %s",
                             cudaGetErrorString(e));
        }
        g_scratch_on_device[ctx->device] = ptr;
    }
    *out = g_scratch_on_device[ctx->device];
    return LOOKAT_OK;
}

struct CurrentDevice {
    int prev;
    bool ok;
    explicit CurrentDevice(int dev) : prev(-1), ok(false)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~CurrentDevice()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

bool misaligned(const void *p, uintptr_t mask) { return (reinterpret_cast<uintptr_t>(p) & mask) != 0; }

}  // namespace
}  // namespace lookat

using namespace lookat;

extern "C" lookat_status lookat_attend_static(lookat_ctx *handle, const float *lut, const void *q,
                                              const float *codebooks, const uint8_t *codes, const void *v,
                                              int32_t B, int64_t L_max, const int32_t *seq_lens,
                                              int32_t n_splits, float *out, float *scores_out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    const lookat_config &c = ctx->cfg;
    if (B < 1 || B > 65535) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "B=%d out of range 1..65535", B);
    if (L_max < 1 || L_max > (1ll << 30))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "L_max=%lld out of range", (long long)L_max);
    if (n_splits < 0) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "n_splits=%d is negative", n_splits);
    if (c.n_q_heads > 65535) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "more than 65535 query heads");
    if (lut && (q || codebooks))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "give either lut or (q, codebooks), not both");
    if (!lut && !(q && codebooks))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "lut is NULL and (q, codebooks) is incomplete");
    if (!codes || !v || !out) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "codes, v or out is NULL");
    if (misaligned(codes, 15) || misaligned(v, 15) || misaligned(out, 15) || misaligned(lut, 15) ||
        misaligned(q, 15) || misaligned(codebooks, 15))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "a data pointer is not 16-byte aligned");
    if (misaligned(seq_lens, 3) || misaligned(scores_out, 3))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "seq_lens or scores_out is not 4-byte aligned");

    CurrentDevice guard(ctx->device);
    if (!guard.ok) return set_error(ctx, LOOKAT_ERR_CUDA, "cannot select device %d", ctx->device);
    unsigned char *scratch = nullptr;
    lookat_status st = static_scratch(ctx, &scratch);
    if (st != LOOKAT_OK) return st;

    AttendArgs a;
    memset(&a, 0, sizeof(a));
    a.lut = lut;
    a.q = static_cast<const __half *>(q);
    a.codebooks = codebooks;
    a.d_k = c.d_k;
    a.codes = codes;
    a.v = static_cast<const __half *>(v);
    a.seq_lens = seq_lens;
    a.uniform_len = (int)L_max;
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
    st = plan_attend(ctx, a, n_splits, &po, &pml);
    if (st != LOOKAT_OK) return st;
    if (!a.lut && !a.fused_lut)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED,
                         "lookat_attend_static: this shape needs ready tables (pass lut); building them here "
                         "would need scratch memory");
    if (po * sizeof(float) > kStaticPartOBytes || pml * sizeof(float) > kStaticPartMlBytes ||
        (a.stream && (size_t)a.n_units * sizeof(unsigned) > kStaticTicketBytes))
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED,
                         "lookat_attend_static: partial results need %zu + %zu bytes and %d counters; the fixed "
                         "scratch holds %zu + %zu bytes and %zu counters (use fewer chunks, or lookat_attend)",
                         po * sizeof(float), pml * sizeof(float), a.stream ? a.n_units : 0, kStaticPartOBytes,
                         kStaticPartMlBytes, kStaticTicketBytes / sizeof(unsigned));
    a.part_o = reinterpret_cast<float *>(scratch);
    a.part_ml = reinterpret_cast<float *>(scratch + kStaticPartOBytes);
    a.tickets = reinterpret_cast<unsigned *>(scratch + kStaticPartOBytes + kStaticPartMlBytes);
    if (a.stream) {
        // the counters must be zero when the kernel starts; an earlier call may have been cut short
        if (cudaMemsetAsync(a.tickets, 0, (size_t)a.n_units * sizeof(unsigned), ctx->stream) != cudaSuccess) {
            cudaGetLastError();
            return set_error(ctx, LOOKAT_ERR_CUDA, "lookat_attend_static: clearing the counters failed");
        }
        return launch_attend(ctx, a);
    }
    st = launch_attend(ctx, a);
    if (st != LOOKAT_OK) return st;
    return launch_combine(ctx, a);
}
