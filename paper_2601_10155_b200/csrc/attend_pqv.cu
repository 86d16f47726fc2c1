// Decode attention with product-quantised VALUES as well.  The paper leaves value compression to future work
// (Section 5.2); this formulation is this build's own and has no counterpart there.  The weights are those of
// Algorithm 1 (scores = sums of table entries named by the key codes, stable softmax); the output
//     o = sum_t alpha_t v^_t,   v^_t = (C^V_1[vcode[t][1]], ..., C^V_mv[vcode[t][mv]])
// is taken per value subspace as  o^(j) = sum_c w[j][c] C^V_j[c]  with the weight histogram
// w[j][c] = sum of alpha_t over the tokens whose value code in subspace j is c.  Nothing but codes is read per
// token: m + m_v bytes instead of m + 2 d_v.
//
// One CTA: one unit (batch row, KV head, group of up to 4 query heads) and one chunk of its tokens.  The unit's
// key tables and the histograms sit in shared memory.  Pass 1 finds the chunk's score maxima, pass 2 forms the
// weights against them and adds them to the histograms with shared-memory atomics (no rescaling inside a chunk);
// the histograms are then contracted with the value codebooks into a partial output, and a second kernel merges
// the chunks of a unit.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kPqThreads = 512;
constexpr int kPqStride = 256;       // shared-memory entries per subspace (codes are bytes)
constexpr int kPqHeadPad = 8;        // floats between two heads' tables (bank shift)

struct PqvArgs {
    const float *lut;        // [B][H_q][m][K]
    const uint8_t *codes;    // [B][H_kv][L_max][m]
    const float *v_books;    // [H_kv][m_v][K_v][d_vsub]
    const uint8_t *v_codes;  // [B][H_kv][L_max][m_v]
    const int32_t *seq_lens;
    float *part_o;           // [unit][split][4][d_v]
    float *part_ml;          // [unit][split][4][2]: maximum (base-2 units), sum
    float *out;              // [B][H_q][d_v]
    long long L_max, chunk;
    int B, H_q, H_kv, g, K, K_v, d_vsub, d_v, n_splits;
    float scale_log2;
};

template <int M>
__device__ __forceinline__ void load_codes(const uint8_t *row, uint8_t (&c)[M])
{
    if (M == 16) {
        const uint4 x = *reinterpret_cast<const uint4 *>(row);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 16; ++i) c[i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
    } else if (M == 8) {
        const uint2 x = *reinterpret_cast<const uint2 *>(row);
#pragma unroll
        for (int i = 0; i < 8; ++i) c[i] = (uint8_t)((i < 4 ? x.x : x.y) >> (8 * (i & 3)));
    } else if (M == 4) {
        const uint32_t x = *reinterpret_cast<const uint32_t *>(row);
#pragma unroll
        for (int i = 0; i < 4; ++i) c[i] = (uint8_t)(x >> (8 * i));
    } else {
#pragma unroll
        for (int i = 0; i < M; ++i) c[i] = row[i];
    }
}

template <int M_K, int M_V>
__global__ void __launch_bounds__(kPqThreads) attend_pqv_kernel(PqvArgs a)
{
    extern __shared__ __align__(16) float pq_smem[];
    constexpr int head_stride_k = M_K * kPqStride + kPqHeadPad;
    constexpr int head_stride_v = M_V * kPqStride + kPqHeadPad;
    float *tab = pq_smem;                                  // [4][M_K][256]
    float *hist = pq_smem + 4 * head_stride_k;             // [4][M_V][256]
    __shared__ float s_red[kPqThreads / 32][4];
    __shared__ float s_m[4], s_l[4];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hgroups = (a.g + 3) >> 2;
    const int unit = blockIdx.y, split = blockIdx.x;
    const int hgrp = unit % hgroups, kv_row = unit / hgroups;
    const int b = kv_row / a.H_kv, kvh = kv_row - b * a.H_kv;
    const int heads = min(4, a.g - hgrp * 4);
    const int hq0 = kvh * a.g + hgrp * 4;

    const long long len = a.seq_lens ? a.seq_lens[b] : a.L_max;
    const long long t0 = (long long)split * a.chunk, t1 = min(len, t0 + a.chunk);

    // ---- the unit's key tables into shared memory; histograms cleared ----
    for (int h = 0; h < heads; ++h) {
        const float *src = a.lut + ((size_t)b * a.H_q + hq0 + h) * M_K * a.K;
        for (int i = tid; i < M_K * a.K; i += kPqThreads) {
            const int j = i / a.K;
            tab[h * head_stride_k + j * kPqStride + (i - j * a.K)] = __ldg(src + i);
        }
    }
    for (int i = tid; i < 4 * head_stride_v; i += kPqThreads) hist[i] = 0.f;
    __syncthreads();

    const uint8_t *krow = a.codes + ((size_t)(b * a.H_kv + kvh) * a.L_max) * M_K;
    const uint8_t *vrow = a.v_codes + ((size_t)(b * a.H_kv + kvh) * a.L_max) * M_V;
    auto scores = [&](long long t, float (&x)[4]) {         // x_h = s_h * scale * log2(e)
        uint8_t c[M_K];
        load_codes<M_K>(krow + (size_t)t * M_K, c);
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            float s = 0.f;
            if (h < heads) {
#pragma unroll
                for (int j = 0; j < M_K; ++j) s += tab[h * head_stride_k + j * kPqStride + c[j]];
            }
            x[h] = s * a.scale_log2;
        }
    };

    // ---- pass 1: the chunk's maxima ----
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    for (long long t = t0 + tid; t < t1; t += kPqThreads) {
        float x[4];
        scores(t, x);
#pragma unroll
        for (int h = 0; h < 4; ++h) mx[h] = fmaxf(mx[h], x[h]);
    }
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        for (int s = 16; s; s >>= 1) mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], s));
        if (lane == 0) s_red[warp][h] = mx[h];
    }
    __syncthreads();
    if (tid < 4) {
        float m = -INFINITY;
        for (int w = 0; w < kPqThreads / 32; ++w) m = fmaxf(m, s_red[w][tid]);
        s_m[tid] = m;
    }
    __syncthreads();
    const float m0 = s_m[0], m1 = s_m[1], m2 = s_m[2], m3 = s_m[3];
    __syncthreads();                                       // s_red is reused below

    // ---- pass 2: weights against those maxima, added to the histograms ----
    float l[4] = {0.f, 0.f, 0.f, 0.f};
    for (long long t = t0 + tid; t < t1; t += kPqThreads) {
        float x[4];
        scores(t, x);
        const float p[4] = {ex2_approx(x[0] - m0), ex2_approx(x[1] - m1), ex2_approx(x[2] - m2), ex2_approx(x[3] - m3)};
        uint8_t vc[M_V];
        load_codes<M_V>(vrow + (size_t)t * M_V, vc);
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            if (h < heads) {
                l[h] += p[h];
#pragma unroll
                for (int j = 0; j < M_V; ++j) atomicAdd(hist + h * head_stride_v + j * kPqStride + vc[j], p[h]);
            }
        }
    }
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        for (int s = 16; s; s >>= 1) l[h] += __shfl_xor_sync(0xffffffffu, l[h], s);
        if (lane == 0) s_red[warp][h] = l[h];
    }
    __syncthreads();
    if (tid < 4) {
        float sum = 0.f;
        for (int w = 0; w < kPqThreads / 32; ++w) sum += s_red[w][tid];
        s_l[tid] = sum;
    }
    __syncthreads();

    // ---- partial output of the chunk: o[h][j * d_vsub + i] = sum_c w[h][j][c] * C^V_j[c][i] ----
    const size_t slot = (size_t)unit * a.n_splits + split;
    const float *vb = a.v_books + (size_t)kvh * M_V * a.K_v * a.d_vsub;
    for (int o = tid; o < heads * a.d_v; o += kPqThreads) {
        const int h = o / a.d_v, dim = o - h * a.d_v, j = dim / a.d_vsub, i = dim - j * a.d_vsub;
        const float *w = hist + h * head_stride_v + j * kPqStride;
        const float *cv = vb + (size_t)j * a.K_v * a.d_vsub + i;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};                // independent sums: the loads overlap
        int c = 0;
        for (; c + 4 <= a.K_v; c += 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[u] = fmaf(w[c + u], __ldg(cv + (size_t)(c + u) * a.d_vsub), acc[u]);
        }
        for (; c < a.K_v; ++c) acc[0] = fmaf(w[c], __ldg(cv + (size_t)c * a.d_vsub), acc[0]);
        a.part_o[(slot * 4 + h) * a.d_v + dim] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    }
    if (tid < heads) {
        a.part_ml[(slot * 4 + tid) * 2] = s_m[tid];
        a.part_ml[(slot * 4 + tid) * 2 + 1] = s_l[tid];
    }
}

// one CTA per (batch row, query head): merge the chunks of its unit (empty chunks carry -inf and 0)
__global__ void combine_pqv_kernel(PqvArgs a)
{
    const int hq = blockIdx.x % a.H_q, b = blockIdx.x / a.H_q;
    const int kvh = hq / a.g, hin = hq - kvh * a.g, hgroups = (a.g + 3) >> 2;
    const int unit = (b * a.H_kv + kvh) * hgroups + (hin >> 2), h = hin & 3;
    float M = -INFINITY;
    for (int s = 0; s < a.n_splits; ++s) M = fmaxf(M, a.part_ml[(((size_t)unit * a.n_splits + s) * 4 + h) * 2]);
    float L = 0.f;
    for (int s = 0; s < a.n_splits; ++s) {
        const float *ml = a.part_ml + (((size_t)unit * a.n_splits + s) * 4 + h) * 2;
        if (ml[1] > 0.f) L += ml[1] * ex2_approx(ml[0] - M);
    }
    for (int dim = threadIdx.x; dim < a.d_v; dim += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < a.n_splits; ++s) {
            const size_t slot = (size_t)unit * a.n_splits + s;
            const float *ml = a.part_ml + (slot * 4 + h) * 2;
            if (ml[1] > 0.f) acc += a.part_o[(slot * 4 + h) * a.d_v + dim] * ex2_approx(ml[0] - M);
        }
        a.out[((size_t)b * a.H_q + hq) * a.d_v + dim] = acc / L;
    }
}

template <int M_K, int M_V>
lookat_status launch_pqv(Ctx *ctx, const PqvArgs &a, int n_units)
{
    const size_t smem = (size_t)4 * ((M_K + M_V) * kPqStride + 2 * kPqHeadPad) * sizeof(float);
    auto kern = attend_pqv_kernel<M_K, M_V>;
    if (smem > 48 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "attend_pqv: shared-memory opt-in");
    kern<<<dim3((unsigned)a.n_splits, (unsigned)n_units), kPqThreads, smem, ctx->stream>>>(a);
    lookat_status st = check_launch(ctx, "attend_pqv_kernel");
    if (st != LOOKAT_OK) return st;
    combine_pqv_kernel<<<a.B * a.H_q, 128, 0, ctx->stream>>>(a);
    return check_launch(ctx, "combine_pqv_kernel");
}

template <int M_K>
lookat_status launch_pqv_mv(Ctx *ctx, const PqvArgs &a, int n_units, int m_v)
{
    switch (m_v) {
        case 2: return launch_pqv<M_K, 2>(ctx, a, n_units);
        case 4: return launch_pqv<M_K, 4>(ctx, a, n_units);
        case 8: return launch_pqv<M_K, 8>(ctx, a, n_units);
        case 16: return launch_pqv<M_K, 16>(ctx, a, n_units);
        default: return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: m_v must be 2, 4, 8 or 16");
    }
}

}  // namespace

lookat_status attend_pqv_impl(Ctx *ctx, const float *lut, const uint8_t *codes, const float *v_books, const uint8_t *v_codes,
                              int m_v, int K_v, int B, long long L_max, const int32_t *seq_lens, float *out)
{
    const lookat_config &c = ctx->cfg;
    if (m_v < 1 || c.d_v % m_v != 0 || K_v < 1 || K_v > 256)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "attend_pqv: need m_v | d_v and 1 <= K_v <= 256 (m_v=%d K_v=%d)", m_v, K_v);
    const int g = c.n_q_heads / c.n_kv_heads, hgroups = (g + 3) / 4;
    const long long n_units = (long long)B * c.n_kv_heads * hgroups;
    if (n_units > 65535) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: more than 65535 units");
    // code rows are read with one aligned load of m (m_v) bytes
    if (((uintptr_t)codes % (c.m >= 16 ? 16 : c.m)) != 0 || ((uintptr_t)v_codes % (m_v >= 16 ? 16 : m_v)) != 0)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "attend_pqv: code arrays must be aligned to their row size");
    PqvArgs a;
    memset(&a, 0, sizeof(a));
    a.lut = lut;
    a.codes = codes;
    a.v_books = v_books;
    a.v_codes = v_codes;
    a.seq_lens = seq_lens;
    a.out = out;
    a.L_max = L_max;
    a.chunk = 8192;
    a.n_splits = (int)((L_max + a.chunk - 1) / a.chunk);
    a.B = B;
    a.H_q = c.n_q_heads;
    a.H_kv = c.n_kv_heads;
    a.g = g;
    a.K = c.K;
    a.K_v = K_v;
    a.d_v = c.d_v;
    a.d_vsub = c.d_v / m_v;
    a.scale_log2 = ctx->scale * 1.4426950408889634f;
    const size_t slots = (size_t)n_units * a.n_splits * 4;
    lookat_status st = ensure(ctx, (void **)&ctx->part_o, &ctx->part_o_cap, slots * c.d_v * sizeof(float), "partials");
    if (st == LOOKAT_OK) st = ensure(ctx, (void **)&ctx->part_ml, &ctx->part_ml_cap, slots * 2 * sizeof(float), "partials");
    if (st != LOOKAT_OK) return st;
    a.part_o = ctx->part_o;
    a.part_ml = ctx->part_ml;
    switch (c.m) {
        case 2: return launch_pqv_mv<2>(ctx, a, (int)n_units, m_v);
        case 4: return launch_pqv_mv<4>(ctx, a, (int)n_units, m_v);
        case 8: return launch_pqv_mv<8>(ctx, a, (int)n_units, m_v);
        case 16: return launch_pqv_mv<16>(ctx, a, (int)n_units, m_v);
        default: return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: m must be 2, 4, 8 or 16");
    }
}

}  // namespace lookat
