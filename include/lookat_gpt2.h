/*
 * lookat_gpt2.h - C ABI of the GPT-2 decoder harness around LOOKAT attention (part of liblookat.so).
 *
 * The paper evaluates its method on GPT-2 (Section 4.1, "Models and Data": 12 layers, 12 heads of 64 dims,
 * d_model 768).  This harness runs that model with random-init weights: the prompt with exact causal attention
 * (Section 3.1), then one token at a time with the keys held only as product-quantisation codes -- codebooks
 * fitted per layer and head on the prompt's keys (Section 3.4 "Prototype Learning"), every new key encoded on
 * append (Section 3.4 "Encoding"), Algorithm 1 in place of q K^T in every layer.  The products, normalisations and
 * activations around the attention are not part of the paper's method; they are hand-written kernels of this library
 * like the rest (tcgen05 for the prompt-sized products, a weight-streaming kernel for the one-token products).
 *
 * Memory: pointers are DEVICE memory owned by the caller unless stated; weights are fp16 and are kept by reference
 * (they must outlive the model).  Linear layers are stored transposed, [out][in].  All work is enqueued on the
 * model's stream; calls do not synchronise.  Errors: lookat_status as in lookat.h; nothing is launched when a call
 * rejects its arguments.
 */
#ifndef LOOKAT_GPT2_H
#define LOOKAT_GPT2_H

#include "lookat.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lookat_gpt2 lookat_gpt2;

typedef struct lookat_gpt2_config {
    int32_t n_layer;
    int32_t n_head;            /* heads of 64 dims */
    int32_t d_model;           /* = 64 * n_head */
    int32_t vocab;
    int32_t n_pos;             /* rows of the position table, >= the cache capacity */
    int32_t m;                 /* key subspaces per head (divides 64) */
    int32_t K;                 /* centroids per subspace, 1..256 */
    int32_t fit_iters;         /* Lloyd iterations on the prompt's keys */
    int32_t keep_prompt_keys;  /* 1: keep every layer's fp16 prompt keys (for checks; costs their memory) */
} lookat_gpt2_config;

/* The weights of one block, all fp16: LayerNorm gains and biases [d], w_qkv [3d][d] (rows: the q, k, v thirds, each
 * head-major), b_qkv [3d], w_o [d][d], b_o [d], w_fc [4d][d], b_fc [4d], w_pr [d][4d], b_pr [d]. */
typedef struct lookat_gpt2_layer {
    const void *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_o, *b_o, *ln2_g, *ln2_b, *w_fc, *b_fc, *w_pr, *b_pr;
} lookat_gpt2_layer;

/* A model for batches of B rows (1..32) and caches of `capacity` tokens per row; allocates its activations and, per
 * layer, codebooks, code cache and fp16 value cache.  *out is set only on success. */
lookat_status lookat_gpt2_create(const lookat_gpt2_config *cfg, int device, void *cuda_stream, int32_t B, int32_t capacity,
                                 lookat_gpt2 **out);
void lookat_gpt2_destroy(lookat_gpt2 *model);
const char *lookat_gpt2_last_error(const lookat_gpt2 *model);

/* wte fp16 [vocab][d] (also the output projection), wpe fp16 [n_pos][d], final LayerNorm gain and bias fp16 [d];
 * layers: HOST array of n_layer structs of device pointers. */
lookat_status lookat_gpt2_set_weights(lookat_gpt2 *model, const void *wte, const void *wpe, const void *lnf_g, const void *lnf_b,
                                      const lookat_gpt2_layer *layers);

/* The prompt: ids int32 [B][T], 1 <= T <= capacity.  Exact causal attention in every layer; afterwards every layer
 * holds codebooks fitted on its prompt keys (seed + layer index seeds the start rule of lookat_fit_codebooks), the
 * prompt's codes and values.  hidden_out: NULL, or fp32 [B][T][d], the residual stream after the last block. */
lookat_status lookat_gpt2_prefill(lookat_gpt2 *model, const int32_t *ids, int32_t T, uint64_t seed, float *hidden_out);

/* One generated token per row: ids int32 [B] is the token at the next position.  In every layer the new key is
 * encoded on append and Algorithm 1 runs over the whole cache (lookat_decode_step).  Outputs, each optional:
 * hidden_out fp32 [B][d] (after the last block), logits fp32 [B][vocab] (final LayerNorm, tied projection),
 * next_ids int32 [B] (first index of the largest logit). */
lookat_status lookat_gpt2_decode(lookat_gpt2 *model, const int32_t *ids, float *hidden_out, float *logits, int32_t *next_ids);

/* Device pointers to a layer's state (for checks): codebooks fp32 [H][m][K][64/m], codes uint8 [B][H][capacity][m],
 * values fp16 [B][H][capacity][64], prompt_keys fp16 [B][H][T][64] (NULL unless kept).  Any out pointer may be NULL. */
lookat_status lookat_gpt2_layer_state(lookat_gpt2 *model, int32_t layer, const float **codebooks, const uint8_t **codes,
                                      const void **values, const void **prompt_keys);

/* Where a decode step's device time goes (measurement aid): with profiling on, lookat_gpt2_decode records a CUDA event
 * after the launches of each category; lookat_gpt2_profile synchronises on them, fills ms[LOOKAT_GPT2_CATEGORIES] with the
 * milliseconds per category summed over the steps decoded since profiling was switched on, and returns that number
 * of steps.  The events add launch gaps: use the shares, time whole steps without profiling. */
enum {
    LOOKAT_GPT2_CAT_EMBED = 0,
    LOOKAT_GPT2_CAT_NORM = 1,       /* both LayerNorms of a block */
    LOOKAT_GPT2_CAT_QKV = 2,        /* fused q/k/v projection */
    LOOKAT_GPT2_CAT_ATTENTION = 3,  /* append-encode + Algorithm 1 (lookat_decode_step) */
    LOOKAT_GPT2_CAT_OUT_PROJ = 4,
    LOOKAT_GPT2_CAT_MLP = 5,        /* both products of the MLP, GELU fused */
    LOOKAT_GPT2_CAT_LM_HEAD = 6,    /* final LayerNorm, tied output projection, argmax */
    LOOKAT_GPT2_CATEGORIES = 7
};
void lookat_gpt2_set_profile(lookat_gpt2 *model, int32_t enabled);
int32_t lookat_gpt2_profile(lookat_gpt2 *model, double *ms);

int32_t lookat_gpt2_position(const lookat_gpt2 *model);          /* tokens in the cache */
uint64_t lookat_gpt2_kernel_launches(const lookat_gpt2 *model);   /* kernels launched since creation */

/*
 * The harness's kernels one by one, on a lookat_ctx (its stream and device; its attention shape plays no part).
 *
 * lookat_linear: out = act(x w_t^T + bias) [+ residual].  x [M][K] fp16 (x_fp32 = 1: fp32, accepted for M <= 32),
 * w_t [N][K] fp16, bias fp16 [N] or NULL, gelu = 1 applies 0.5 x (1 + tanh(sqrt(2/pi)(x + 0.044715 x^3))) after the
 * bias, residual fp32 [M][N] or NULL (may be `out`), out [M][N] fp16 (out_fp16 = 1) or fp32.  K a multiple of 8.
 * M > 32 runs on tcgen05 (TMA operand tiles, accumulator in tensor memory), M <= 32 on the weight-streaming kernel.
 *
 * lookat_linear_qkv: the fused q/k/v projection of a block, N = 3 * 64 * n_head, row = b * T + t, scattered
 * head-major as fp16: third s, head h, dim d goes to dst_s[((b * n_head + h) * cap_s + off_s + t) * 64 + d].
 *
 * lookat_layernorm: per row (x - mean) / sqrt(var + 1e-5) * gain + bias, fp32 in, fp16 out, d <= 1024.
 * lookat_embed: out[b][t] = wte[ids[b][t]] + wpe[pos0 + t], fp32 [B][T][d].
 * lookat_causal_attention: Section 3.1 with a causal mask over a prompt: q, k fp16 [B][H][T][64], v fp16
 * [B][H][v_cap][64] (first T rows used), out fp16 [B][T][H * 64].
 * lookat_argmax: out[r] = first index of the largest of logits[r][0..n).
 */
lookat_status lookat_linear(lookat_ctx *ctx, const void *x, int32_t x_fp32, const void *w_t, const void *bias, int64_t M, int32_t N,
                            int32_t K, int32_t gelu, const float *residual, void *out, int32_t out_fp16);
lookat_status lookat_linear_qkv(lookat_ctx *ctx, const void *x, const void *w_t, const void *bias, int32_t B, int32_t T, int32_t n_head,
                                void *q, int64_t q_cap, int64_t q_off, void *k, int64_t k_cap, int64_t k_off, void *v, int64_t v_cap,
                                int64_t v_off);
lookat_status lookat_layernorm(lookat_ctx *ctx, const float *x, const void *gain, const void *bias, int64_t rows, int32_t d, void *out);
lookat_status lookat_embed(lookat_ctx *ctx, const int32_t *ids, const void *wte, const void *wpe, int32_t B, int32_t T, int32_t pos0,
                           int32_t d, int32_t vocab, float *out);
lookat_status lookat_causal_attention(lookat_ctx *ctx, const void *q, const void *k, const void *v, int32_t B, int32_t H, int32_t T,
                                      int64_t v_cap, void *out);
lookat_status lookat_argmax(lookat_ctx *ctx, const float *logits, int32_t rows, int32_t n, int32_t *out);

#ifdef __cplusplus
}
#endif
#endif /* LOOKAT_GPT2_H */
