// GPT-2 decoder harness around LOOKAT attention (include/lookat_gpt2.h): the model the paper evaluates on (Section
// 4.1) with exact causal attention over the prompt (Section 3.1) and, for every generated token, the new key encoded
// on append (Section 3.4 "Encoding") and Algorithm 1 in place of q K^T in every layer.  This file is the runtime:
// buffers, the per-layer launch sequences, and the C entry points; the kernels live in linear_umma.cu, gpt2_ops.cu and
// the attention files.  Activations: the residual stream is fp32, everything a product reads is fp16.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "lookat_gpt2.h"

namespace lookat {

struct Gpt2 {
    lookat_gpt2_config cfg;
    int B, capacity, device;
    cudaStream_t stream;
    lookat_ctx *attn;                       // the attention context: H heads of 64 dims, m subspaces, K centroids
    char err[512];
    // weights (caller-owned device memory)
    const __half *wte, *wpe, *lnf_g, *lnf_b;
    std::vector<lookat_gpt2_layer> layers;
    bool have_weights;
    // activations
    float *x;                               // [B * capacity][d]   residual stream
    __half *a16, *att16, *fc16;             // [rows][d], [rows][d], [rows][4 d]
    __half *q16, *k16;                      // [B][H][T][64] of the layer being processed (prompt pass)
    __half *qd, *kd;                        // [B][H][64] of a decode step
    float *attn_out;                        // [B][H * 64] fp32 (what lookat_decode_step writes)
    float *logits;                          // [B][vocab] when the caller passes none
    // per layer state of the compressed cache
    std::vector<float *> books;             // [H][m][K][64 / m]
    std::vector<uint8_t *> codes;           // [B][H][capacity][m]
    std::vector<__half *> values;           // [B][H][capacity][64]
    std::vector<__half *> prompt_keys;      // [B][H][T][64], kept on request (tests)
    int pos;                                // tokens in the cache
    // optional per-category device timing of a decode step (events between the launches of one step)
    bool profile;
    std::vector<cudaEvent_t> prof_ev;       // boundaries, in launch order
    std::vector<int> prof_cat;              // category of the work between boundary i and i + 1
};

namespace {

lookat_status g_fail(Gpt2 *g, lookat_status st, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g->err, sizeof(g->err), fmt, ap);
    va_end(ap);
    return st;
}

Ctx *ctx_of(Gpt2 *g) { return reinterpret_cast<Ctx *>(g->attn); }

template <class T>
bool dev_alloc(T **p, size_t n)
{
    *p = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(p), n * sizeof(T)) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}

#define G_TRY(expr)                                                                              \
    do {                                                                                         \
        lookat_status st__ = (expr);                                                             \
        if (st__ != LOOKAT_OK) {                                                                 \
            if (!g->err[0]) snprintf(g->err, sizeof(g->err), "%s", lookat_last_error(g->attn)); \
            return st__;                                                                         \
        }                                                                                        \
    } while (0)

// when profiling: closes the category of the launches made since the previous mark
void mark(Gpt2 *g, int category)
{
    if (!g->profile) return;
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    cudaEventRecord(e, g->stream);
    g->prof_ev.push_back(e);
    g->prof_cat.push_back(category);
}

LinearArgs plain(const __half *bias, long long M, int N, int K, int gelu, const float *residual, void *out, int out_fp16)
{
    LinearArgs p;
    memset(&p, 0, sizeof(p));
    p.bias = bias;
    p.residual = residual;
    p.out = out;
    p.out_fp16 = out_fp16;
    p.gelu = gelu;
    p.M = M;
    p.N = N;
    p.K = K;
    return p;
}

// the attention-free half of a block: x += W_pr gelu(W_fc LN2(x) + b_fc) + b_pr
lookat_status mlp(Gpt2 *g, const lookat_gpt2_layer &w, long long rows)
{
    Ctx *ctx = ctx_of(g);
    const int d = g->cfg.d_model;
    G_TRY(launch_layernorm(ctx, g->x, (const __half *)w.ln2_g, (const __half *)w.ln2_b, g->a16, rows, d));
    mark(g, LOOKAT_GPT2_CAT_NORM);
    G_TRY(launch_linear(ctx, g->a16, 0, (const __half *)w.w_fc, plain((const __half *)w.b_fc, rows, 4 * d, d, 1, nullptr, g->fc16, 1)));
    G_TRY(launch_linear(ctx, g->fc16, 0, (const __half *)w.w_pr, plain((const __half *)w.b_pr, rows, d, 4 * d, 0, g->x, g->x, 0)));
    mark(g, LOOKAT_GPT2_CAT_MLP);
    return LOOKAT_OK;
}

}  // namespace
}  // namespace lookat

using namespace lookat;

extern "C" {

lookat_status lookat_gpt2_create(const lookat_gpt2_config *cfg, int device, void *cuda_stream, int32_t B, int32_t capacity,
                                 lookat_gpt2 **out)
{
    if (!cfg || !out) return LOOKAT_ERR_INVALID_ARG;
    const lookat_gpt2_config &c = *cfg;
    if (c.n_layer < 1 || c.n_head < 1 || c.d_model != c.n_head * 64 || c.vocab < 1 || c.n_pos < capacity || B < 1 || B > 32 ||
        capacity < 1 || c.m < 1 || 64 % c.m != 0 || c.K < 1 || c.K > 256 || c.fit_iters < 0)
        return LOOKAT_ERR_INVALID_ARG;
    Gpt2 *g = new (std::nothrow) Gpt2();
    if (!g) return LOOKAT_ERR_NOMEM;
    g->cfg = c;
    g->B = B;
    g->capacity = capacity;
    g->device = device;
    g->stream = static_cast<cudaStream_t>(cuda_stream);
    g->err[0] = 0;
    g->have_weights = false;
    g->pos = 0;
    g->profile = false;
    lookat_config ac = {c.n_head, c.n_head, 64, 64, c.m, c.K, 0.f};
    lookat_status st = lookat_create(&ac, device, cuda_stream, &g->attn);
    if (st != LOOKAT_OK) {
        delete g;
        return st;
    }
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(device);
    const size_t rows = (size_t)B * capacity, d = c.d_model, H = c.n_head;
    bool ok = dev_alloc(&g->x, rows * d) && dev_alloc(&g->a16, rows * d) && dev_alloc(&g->att16, rows * d) &&
              dev_alloc(&g->fc16, rows * 4 * d) && dev_alloc(&g->q16, rows * d) && dev_alloc(&g->k16, rows * d) &&
              dev_alloc(&g->qd, (size_t)B * d) && dev_alloc(&g->kd, (size_t)B * d) && dev_alloc(&g->attn_out, (size_t)B * d) &&
              dev_alloc(&g->logits, (size_t)B * c.vocab);
    g->books.assign(c.n_layer, nullptr);
    g->codes.assign(c.n_layer, nullptr);
    g->values.assign(c.n_layer, nullptr);
    g->prompt_keys.assign(c.n_layer, nullptr);
    for (int l = 0; ok && l < c.n_layer; ++l) {
        ok = dev_alloc(&g->books[l], H * c.K * 64) && dev_alloc(&g->codes[l], rows * H * c.m) && dev_alloc(&g->values[l], rows * d);
        if (ok && c.keep_prompt_keys) ok = dev_alloc(&g->prompt_keys[l], rows * d);
        if (ok) ok = cudaMemsetAsync(g->codes[l], 0, rows * H * c.m, g->stream) == cudaSuccess &&
                     cudaMemsetAsync(g->values[l], 0, rows * d * sizeof(__half), g->stream) == cudaSuccess;
    }
    if (prev >= 0) cudaSetDevice(prev);
    if (!ok) {
        lookat_gpt2_destroy(reinterpret_cast<lookat_gpt2 *>(g));
        return LOOKAT_ERR_NOMEM;
    }
    *out = reinterpret_cast<lookat_gpt2 *>(g);
    return LOOKAT_OK;
}

void lookat_gpt2_destroy(lookat_gpt2 *handle)
{
    if (!handle) return;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(g->device);
    cudaStreamSynchronize(g->stream);
    void *bufs[] = {g->x, g->a16, g->att16, g->fc16, g->q16, g->k16, g->qd, g->kd, g->attn_out, g->logits};
    for (void *p : bufs)
        if (p) cudaFree(p);
    for (size_t l = 0; l < g->books.size(); ++l) {
        if (g->books[l]) cudaFree(g->books[l]);
        if (g->codes[l]) cudaFree(g->codes[l]);
        if (g->values[l]) cudaFree(g->values[l]);
        if (g->prompt_keys[l]) cudaFree(g->prompt_keys[l]);
    }
    cudaGetLastError();
    if (prev >= 0) cudaSetDevice(prev);
    for (cudaEvent_t e : g->prof_ev) cudaEventDestroy(e);
    lookat_destroy(g->attn);
    delete g;
}

const char *lookat_gpt2_last_error(const lookat_gpt2 *handle)
{
    return handle ? reinterpret_cast<const Gpt2 *>(handle)->err : "model is NULL";
}

uint64_t lookat_gpt2_kernel_launches(const lookat_gpt2 *handle)
{
    return handle ? lookat_kernel_launches(reinterpret_cast<const Gpt2 *>(handle)->attn) : 0;
}

int32_t lookat_gpt2_position(const lookat_gpt2 *handle) { return handle ? reinterpret_cast<const Gpt2 *>(handle)->pos : -1; }

lookat_status lookat_gpt2_set_weights(lookat_gpt2 *handle, const void *wte, const void *wpe, const void *lnf_g, const void *lnf_b,
                                      const lookat_gpt2_layer *layers)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    g->err[0] = 0;
    if (!wte || !wpe || !lnf_g || !lnf_b || !layers) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "a weight pointer is NULL");
    for (int l = 0; l < g->cfg.n_layer; ++l) {
        const void *ps[] = {layers[l].ln1_g, layers[l].ln1_b, layers[l].w_qkv, layers[l].b_qkv, layers[l].w_o,  layers[l].b_o,
                            layers[l].ln2_g, layers[l].ln2_b, layers[l].w_fc,  layers[l].b_fc,  layers[l].w_pr, layers[l].b_pr};
        for (const void *p : ps)
            if (!p || (reinterpret_cast<uintptr_t>(p) & 15)) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "layer %d: a weight pointer is NULL or not 16-byte aligned", l);
    }
    g->wte = static_cast<const __half *>(wte);
    g->wpe = static_cast<const __half *>(wpe);
    g->lnf_g = static_cast<const __half *>(lnf_g);
    g->lnf_b = static_cast<const __half *>(lnf_b);
    g->layers.assign(layers, layers + g->cfg.n_layer);
    g->have_weights = true;
    return LOOKAT_OK;
}

lookat_status lookat_gpt2_prefill(lookat_gpt2 *handle, const int32_t *ids, int32_t T, uint64_t seed, float *hidden_out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    g->err[0] = 0;
    if (!g->have_weights) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "set the weights first");
    if (!ids || T < 1 || T > g->capacity) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "need ids and 1 <= T <= capacity (T=%d)", T);
    Ctx *ctx = ctx_of(g);
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(g->device);
    struct Restore { int d; ~Restore() { if (d >= 0) cudaSetDevice(d); } } restore{prev};
    const lookat_gpt2_config &c = g->cfg;
    const int d = c.d_model, H = c.n_head, B = g->B;
    const long long rows = (long long)B * T;
    G_TRY(launch_embed(ctx, ids, g->wte, g->wpe, g->x, rows, T, 0, d, c.vocab));
    for (int l = 0; l < c.n_layer; ++l) {
        const lookat_gpt2_layer &w = g->layers[l];
        G_TRY(launch_layernorm(ctx, g->x, (const __half *)w.ln1_g, (const __half *)w.ln1_b, g->a16, rows, d));
        // fused projection, scattered head-major: q and k dense over the prompt, v into the layer's value cache
        LinearArgs p = plain((const __half *)w.b_qkv, rows, 3 * d, d, 0, nullptr, nullptr, 1);
        p.qkv = 1;
        p.T = T;
        p.n_head = H;
        p.dst[0] = g->q16; p.cap[0] = T; p.off[0] = 0;
        p.dst[1] = g->k16; p.cap[1] = T; p.off[1] = 0;
        p.dst[2] = g->values[l]; p.cap[2] = g->capacity; p.off[2] = 0;
        G_TRY(launch_linear(ctx, g->a16, 0, (const __half *)w.w_qkv, p));
        // the prompt attends exactly (Section 3.1): the codebooks do not exist yet
        G_TRY(launch_causal_attention(ctx, g->q16, g->k16, g->values[l], g->att16, B, H, T, g->capacity));
        G_TRY(launch_linear(ctx, g->att16, 0, (const __half *)w.w_o, plain((const __half *)w.b_o, rows, d, d, 0, g->x, g->x, 0)));
        G_TRY(mlp(g, w, rows));
        // Section 3.4: codebooks from the prompt's keys of every head, then the prompt's codes
        G_TRY(lookat_fit_codebooks(g->attn, g->k16, B, T, c.fit_iters, seed + (uint64_t)l, nullptr, g->books[l], nullptr));
        G_TRY(lookat_encode_keys(g->attn, g->k16, B, T, g->books[l], g->codes[l], g->capacity, 0, nullptr));
        if (g->prompt_keys[l] &&
            cudaMemcpyAsync(g->prompt_keys[l], g->k16, (size_t)rows * d * sizeof(__half), cudaMemcpyDeviceToDevice, g->stream) != cudaSuccess)
            return g_fail(g, LOOKAT_ERR_CUDA, "copy of the prompt keys failed");
    }
    if (hidden_out &&
        cudaMemcpyAsync(hidden_out, g->x, (size_t)rows * d * sizeof(float), cudaMemcpyDeviceToDevice, g->stream) != cudaSuccess)
        return g_fail(g, LOOKAT_ERR_CUDA, "copy of the hidden states failed");
    g->pos = T;
    return LOOKAT_OK;
}

lookat_status lookat_gpt2_decode(lookat_gpt2 *handle, const int32_t *ids, float *hidden_out, float *logits, int32_t *next_ids)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    g->err[0] = 0;
    if (!g->have_weights || g->pos < 1) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "run the prompt first");
    if (!ids) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "ids is NULL");
    if (g->pos >= g->capacity) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "the cache is full (%d tokens)", g->capacity);
    Ctx *ctx = ctx_of(g);
    int prev = -1;
    cudaGetDevice(&prev);
    cudaSetDevice(g->device);
    struct Restore { int d; ~Restore() { if (d >= 0) cudaSetDevice(d); } } restore{prev};
    const lookat_gpt2_config &c = g->cfg;
    const int d = c.d_model, H = c.n_head, B = g->B, pos = g->pos;
    mark(g, -1);                                             // opens the step
    G_TRY(launch_embed(ctx, ids, g->wte, g->wpe, g->x, B, 1, pos, d, c.vocab));
    mark(g, LOOKAT_GPT2_CAT_EMBED);
    for (int l = 0; l < c.n_layer; ++l) {
        const lookat_gpt2_layer &w = g->layers[l];
        G_TRY(launch_layernorm(ctx, g->x, (const __half *)w.ln1_g, (const __half *)w.ln1_b, g->a16, B, d));
        mark(g, LOOKAT_GPT2_CAT_NORM);
        LinearArgs p = plain((const __half *)w.b_qkv, B, 3 * d, d, 0, nullptr, nullptr, 1);
        p.qkv = 1;
        p.T = 1;
        p.n_head = H;
        p.dst[0] = g->qd; p.cap[0] = 1; p.off[0] = 0;
        p.dst[1] = g->kd; p.cap[1] = 1; p.off[1] = 0;
        p.dst[2] = g->values[l]; p.cap[2] = g->capacity; p.off[2] = pos;       // the value row goes straight into the cache
        G_TRY(launch_linear(ctx, g->a16, 0, (const __half *)w.w_qkv, p));
        mark(g, LOOKAT_GPT2_CAT_QKV);
        // append (Section 3.4 "Encoding") and Algorithm 1 over tokens 0..pos, one launch
        G_TRY(lookat_decode_step(g->attn, g->qd, g->kd, g->books[l], g->codes[l], g->values[l], B, g->capacity, pos, 0, g->attn_out));
        mark(g, LOOKAT_GPT2_CAT_ATTENTION);
        G_TRY(launch_linear(ctx, g->attn_out, 1, (const __half *)w.w_o, plain((const __half *)w.b_o, B, d, d, 0, g->x, g->x, 0)));
        mark(g, LOOKAT_GPT2_CAT_OUT_PROJ);
        G_TRY(mlp(g, w, B));
    }
    if (hidden_out && cudaMemcpyAsync(hidden_out, g->x, (size_t)B * d * sizeof(float), cudaMemcpyDeviceToDevice, g->stream) != cudaSuccess)
        return g_fail(g, LOOKAT_ERR_CUDA, "copy of the hidden rows failed");
    if (logits || next_ids) {
        float *lg = logits ? logits : g->logits;
        G_TRY(launch_layernorm(ctx, g->x, g->lnf_g, g->lnf_b, g->a16, B, d));
        G_TRY(launch_linear(ctx, g->a16, 0, g->wte, plain(nullptr, B, c.vocab, d, 0, nullptr, lg, 0)));     // tied output projection
        if (next_ids) G_TRY(launch_argmax(ctx, lg, next_ids, B, c.vocab));
        mark(g, LOOKAT_GPT2_CAT_LM_HEAD);
    }
    g->pos = pos + 1;
    return LOOKAT_OK;
}

void lookat_gpt2_set_profile(lookat_gpt2 *handle, int32_t enabled)
{
    if (!handle) return;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    for (cudaEvent_t e : g->prof_ev) cudaEventDestroy(e);
    g->prof_ev.clear();
    g->prof_cat.clear();
    g->profile = enabled != 0;
}

int32_t lookat_gpt2_profile(lookat_gpt2 *handle, double *ms)
{
    if (!handle || !ms) return 0;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    for (int i = 0; i < LOOKAT_GPT2_CATEGORIES; ++i) ms[i] = 0.0;
    int steps = 0;
    for (size_t i = 1; i < g->prof_ev.size(); ++i) {
        if (g->prof_cat[i] < 0) {                           // a step's opening mark: nothing to attribute
            continue;
        }
        float t = 0.f;
        cudaEventSynchronize(g->prof_ev[i]);
        if (cudaEventElapsedTime(&t, g->prof_ev[i - 1], g->prof_ev[i]) == cudaSuccess) ms[g->prof_cat[i]] += t;
    }
    for (int c : g->prof_cat) steps += c < 0 ? 1 : 0;
    return steps;
}

lookat_status lookat_gpt2_layer_state(lookat_gpt2 *handle, int32_t layer, const float **codebooks, const uint8_t **codes,
                                      const void **values, const void **prompt_keys)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Gpt2 *g = reinterpret_cast<Gpt2 *>(handle);
    if (layer < 0 || layer >= g->cfg.n_layer) return g_fail(g, LOOKAT_ERR_INVALID_ARG, "layer %d out of range", layer);
    if (codebooks) *codebooks = g->books[layer];
    if (codes) *codes = g->codes[layer];
    if (values) *values = g->values[layer];
    if (prompt_keys) *prompt_keys = g->prompt_keys[layer];
    return LOOKAT_OK;
}

// ---- the harness's kernels one by one (what the tests compare with the oracle) ----
lookat_status lookat_linear(lookat_ctx *handle, const void *x, int32_t x_fp32, const void *w_t, const void *bias, int64_t M, int32_t N,
                            int32_t K, int32_t gelu, const float *residual, void *out, int32_t out_fp16)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!x || !w_t || !out || ((uintptr_t)x & 15) || ((uintptr_t)w_t & 15) || ((uintptr_t)out & 15) || ((uintptr_t)residual & 15))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "linear: a pointer is NULL or not 16-byte aligned");
    if (M < 1 || N < 1 || K < 8 || K % 8 != 0 || M > (1ll << 22))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "linear: need 1 <= M <= 2^22, N >= 1, K a multiple of 8");
    return launch_linear(ctx, x, x_fp32, static_cast<const __half *>(w_t), plain(static_cast<const __half *>(bias), M, N, K, gelu, residual, out, out_fp16));
}

lookat_status lookat_linear_qkv(lookat_ctx *handle, const void *x, const void *w_t, const void *bias, int32_t B, int32_t T, int32_t n_head,
                                void *q, int64_t q_cap, int64_t q_off, void *k, int64_t k_cap, int64_t k_off, void *v, int64_t v_cap,
                                int64_t v_off)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!x || !w_t || !q || !k || !v || B < 1 || T < 1 || n_head < 1 || q_off + T > q_cap || k_off + T > k_cap || v_off + T > v_cap ||
        q_off < 0 || k_off < 0 || v_off < 0)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "linear_qkv: bad arguments");
    const int d = n_head * 64;
    LinearArgs p = plain(static_cast<const __half *>(bias), (long long)B * T, 3 * d, d, 0, nullptr, nullptr, 1);
    p.qkv = 1;
    p.T = T;
    p.n_head = n_head;
    p.dst[0] = static_cast<__half *>(q); p.cap[0] = q_cap; p.off[0] = q_off;
    p.dst[1] = static_cast<__half *>(k); p.cap[1] = k_cap; p.off[1] = k_off;
    p.dst[2] = static_cast<__half *>(v); p.cap[2] = v_cap; p.off[2] = v_off;
    return launch_linear(ctx, x, 0, static_cast<const __half *>(w_t), p);
}

lookat_status lookat_layernorm(lookat_ctx *handle, const float *x, const void *gain, const void *bias, int64_t rows, int32_t d, void *out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!x || !gain || !bias || !out || rows < 1 || d < 1) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "layernorm: bad arguments");
    return launch_layernorm(ctx, x, static_cast<const __half *>(gain), static_cast<const __half *>(bias), static_cast<__half *>(out), rows, d);
}

lookat_status lookat_embed(lookat_ctx *handle, const int32_t *ids, const void *wte, const void *wpe, int32_t B, int32_t T, int32_t pos0,
                           int32_t d, int32_t vocab, float *out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!ids || !wte || !wpe || !out || B < 1 || T < 1 || pos0 < 0 || d < 2 || d % 2 || vocab < 1)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "embed: bad arguments");
    return launch_embed(ctx, ids, static_cast<const __half *>(wte), static_cast<const __half *>(wpe), out, (long long)B * T, T, pos0, d, vocab);
}

lookat_status lookat_causal_attention(lookat_ctx *handle, const void *q, const void *k, const void *v, int32_t B, int32_t H, int32_t T,
                                      int64_t v_cap, void *out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!q || !k || !v || !out || B < 1 || B > 65535 || H < 1 || H > 65535 || T < 1 || v_cap < T || ((uintptr_t)q & 15) ||
        ((uintptr_t)k & 15) || ((uintptr_t)v & 15) || ((uintptr_t)out & 15))
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "causal_attention: bad arguments");
    return launch_causal_attention(ctx, static_cast<const __half *>(q), static_cast<const __half *>(k), static_cast<const __half *>(v),
                                   static_cast<__half *>(out), B, H, T, v_cap);
}

lookat_status lookat_argmax(lookat_ctx *handle, const float *logits, int32_t rows, int32_t n, int32_t *out)
{
    if (!handle) return LOOKAT_ERR_INVALID_ARG;
    Ctx *ctx = reinterpret_cast<Ctx *>(handle);
    if (!logits || !out || rows < 1 || n < 1) return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "argmax: bad arguments");
    return launch_argmax(ctx, logits, out, rows, n);
}

}  // extern "C"
