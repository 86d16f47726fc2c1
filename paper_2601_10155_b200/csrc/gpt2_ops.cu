// The small kernels of the GPT-2 decoder harness around LOOKAT attention (the model of Section 4.1; none of this is
// the paper's method): embeddings, LayerNorm, exact causal attention over the prompt (Section 3.1), argmax.
#include "common.cuh"

namespace lookat {

namespace {

// x[row] = wte[id[row]] + wpe[pos0 + t], row = b * T + t; fp16 tables, fp32 residual stream
__global__ void embed_kernel(const int32_t *__restrict__ ids, const __half *__restrict__ wte, const __half *__restrict__ wpe,
                             float *__restrict__ x, long long rows, int T, int pos0, int d, int vocab)
{
    const long long row = blockIdx.x;
    if (row >= rows) return;
    int id = ids[row];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);        // ids outside the table are clamped, never read past it
    const int t = (int)(row % T);
    const __half2 *e = reinterpret_cast<const __half2 *>(wte + (size_t)id * d);
    const __half2 *p = reinterpret_cast<const __half2 *>(wpe + (size_t)(pos0 + t) * d);
    float2 *o = reinterpret_cast<float2 *>(x + (size_t)row * d);
    for (int i = threadIdx.x; i < d / 2; i += blockDim.x) {
        const float2 a = __half22float2(e[i]), b = __half22float2(p[i]);
        o[i] = make_float2(a.x + b.x, a.y + b.y);
    }
}

// y = (x - mean) / sqrt(var + eps) * g + b per row (biased variance), one warp per row, fp32 in, fp16 out; d <= 1024
constexpr int kLnormPerLane = 32;
__global__ void __launch_bounds__(256) layernorm_kernel(const float *__restrict__ x, const __half *__restrict__ g,
                                                        const __half *__restrict__ b, __half *__restrict__ y, long long rows, int d,
                                                        float eps)
{
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const float *xr = x + (size_t)row * d;
    float v[kLnormPerLane];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kLnormPerLane; ++i) {
        const int c = lane + 32 * i;
        v[i] = c < d ? xr[c] : 0.f;
        s += v[i];
    }
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mean = s / (float)d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < kLnormPerLane; ++i) {
        const int c = lane + 32 * i;
        const float t = c < d ? v[i] - mean : 0.f;
        q += t * t;
    }
    for (int o = 16; o; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    const float rstd = rsqrtf(q / (float)d + eps);
    __half *yr = y + (size_t)row * d;
#pragma unroll
    for (int i = 0; i < kLnormPerLane; ++i) {
        const int c = lane + 32 * i;
        if (c < d) yr[c] = __float2half_rn((v[i] - mean) * rstd * __half2float(g[c]) + __half2float(b[c]));
    }
}

// first index of the largest logit of every row
constexpr int kAmThreads = 1024;
__global__ void __launch_bounds__(kAmThreads) argmax_kernel(const float *__restrict__ logits, int32_t *__restrict__ out, int n)
{
    __shared__ float sv[kAmThreads / 32];
    __shared__ int si[kAmThreads / 32];
    const float *row = logits + (size_t)blockIdx.x * n;
    float best = -INFINITY;
    int idx = 0x7fffffff;
#pragma unroll 4
    for (int i = threadIdx.x; i < n; i += kAmThreads) {
        const float v = row[i];
        if (v > best) { best = v; idx = i; }
    }
    for (int o = 16; o; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (ov > best || (ov == best && oi < idx)) { best = ov; idx = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x < 32) {
        best = sv[threadIdx.x];
        idx = si[threadIdx.x];
        for (int o = 16; o; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (ov > best || (ov == best && oi < idx)) { best = ov; idx = oi; }
        }
        if (threadIdx.x == 0) out[blockIdx.x] = idx == 0x7fffffff ? 0 : idx;
    }
}

// ---- exact causal attention over the prompt: softmax(q k^T / sqrt(64)) v, head dim 64 ----
// One CTA: 64 consecutive queries of one (row, head), 4 warps x 16 query rows; keys and values in blocks of 64 tokens
// through shared memory; scores and the weighted value sum on mma.sync.m16n8k16 (fp16 in, fp32 accumulate), the
// weights rounded to fp16 for the second product, the row sum taken over the rounded weights.
constexpr int kCaThreads = 128, kCaBlock = 64, kCaPitch = 72;     // halfs per staged row (64 + 8: conflict-free fragment reads)

__device__ __forceinline__ void ca_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_half2(float a, float b)
{
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t *>(&h);
}

__global__ void __launch_bounds__(kCaThreads)
causal_attention_kernel(const __half *__restrict__ q, const __half *__restrict__ k, const __half *__restrict__ v,
                        __half *__restrict__ out, int H, int T, long long v_cap, float scale_log2)
{
    __shared__ __align__(16) __half ks[kCaBlock * kCaPitch];
    __shared__ __align__(16) __half vs[kCaBlock * kCaPitch];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int qb = gridDim.x - 1 - blockIdx.x;                  // longest first
    const int h = blockIdx.y, b = blockIdx.z;
    const size_t qk_row0 = ((size_t)b * H + h) * T;
    const __half *vg = v + ((size_t)b * H + h) * v_cap * 64;
    const int q0 = qb * kCaBlock + warp * 16;                    // this warp's first query row

    // the warp's 16 query rows as A fragments of the four 16-dim steps (rows beyond T repeat the last row)
    uint32_t qa[4][4];
    {
        const int r0 = min(q0 + g, T - 1), r1 = min(q0 + g + 8, T - 1);
        const __half *p0 = q + (qk_row0 + r0) * 64, *p1 = q + (qk_row0 + r1) * 64;
#pragma unroll
        for (int ks4 = 0; ks4 < 4; ++ks4) {
            qa[ks4][0] = *reinterpret_cast<const uint32_t *>(p0 + ks4 * 16 + 2 * t);
            qa[ks4][1] = *reinterpret_cast<const uint32_t *>(p1 + ks4 * 16 + 2 * t);
            qa[ks4][2] = *reinterpret_cast<const uint32_t *>(p0 + ks4 * 16 + 2 * t + 8);
            qa[ks4][3] = *reinterpret_cast<const uint32_t *>(p1 + ks4 * 16 + 2 * t + 8);
        }
    }
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m0 = -1e30f, m1 = -1e30f, l0 = 0.f, l1 = 0.f;         // rows g and g + 8

    const int n_blocks = qb + 1;                                 // key blocks up to the diagonal
    for (int kb = 0; kb < n_blocks; ++kb) {
        __syncthreads();
        for (int i = tid; i < kCaBlock * 8; i += kCaThreads) {   // 64 rows x 8 pieces of 16 bytes
            const int r = i >> 3, c = (i & 7) * 8;
            const int tok = kb * kCaBlock + r;
            uint4 kv = make_uint4(0u, 0u, 0u, 0u), vv = kv;
            if (tok < T) {
                kv = *reinterpret_cast<const uint4 *>(k + (qk_row0 + tok) * 64 + c);
                vv = *reinterpret_cast<const uint4 *>(vg + (size_t)tok * 64 + c);
            }
            *reinterpret_cast<uint4 *>(ks + r * kCaPitch + c) = kv;
            *reinterpret_cast<uint4 *>(vs + r * kCaPitch + c) = vv;
        }
        __syncthreads();
        // S = Q K^T: 8 tiles of 8 keys
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int ks4 = 0; ks4 < 4; ++ks4) {
                const __half *kr = ks + (nt * 8 + g) * kCaPitch + ks4 * 16 + 2 * t;
                ca_mma(s[nt], qa[ks4], *reinterpret_cast<const uint32_t *>(kr), *reinterpret_cast<const uint32_t *>(kr + 8));
            }
        }
        // scale, causal mask (key <= query, key < T), row maxima
        float mx0 = -1e30f, mx1 = -1e30f;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int key = kb * kCaBlock + nt * 8 + 2 * t + (i & 1), qr = q0 + g + 8 * (i >> 1);
                const float x = (key <= qr && key < T) ? s[nt][i] * scale_log2 : -INFINITY;
                s[nt][i] = x;
                if (i < 2) mx0 = fmaxf(mx0, x); else mx1 = fmaxf(mx1, x);
            }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
        const float a0 = ex2_approx(m0 - n0), a1 = ex2_approx(m1 - n1);
        m0 = n0; m1 = n1;
        // weights as fp16 A fragments (two key tiles per 16-key step); the row sums are taken over the rounded weights
        uint32_t pa[4][4];
        float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const __half2 w01 = __floats2half2_rn(ex2_approx(s[nt][0] - n0), ex2_approx(s[nt][1] - n0));
            const __half2 w23 = __floats2half2_rn(ex2_approx(s[nt][2] - n1), ex2_approx(s[nt][3] - n1));
            const float2 f01 = __half22float2(w01), f23 = __half22float2(w23);
            sum0 += f01.x + f01.y;
            sum1 += f23.x + f23.y;
            pa[nt >> 1][(nt & 1) * 2] = *reinterpret_cast<const uint32_t *>(&w01);
            pa[nt >> 1][(nt & 1) * 2 + 1] = *reinterpret_cast<const uint32_t *>(&w23);
        }
        sum0 += __shfl_xor_sync(0xffffffffu, sum0, 1); sum0 += __shfl_xor_sync(0xffffffffu, sum0, 2);
        sum1 += __shfl_xor_sync(0xffffffffu, sum1, 1); sum1 += __shfl_xor_sync(0xffffffffu, sum1, 2);
        l0 = l0 * a0 + sum0;
        l1 = l1 * a1 + sum1;
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) { o[dt][0] *= a0; o[dt][1] *= a0; o[dt][2] *= a1; o[dt][3] *= a1; }
        // O += P V: per 16-key step and 8-dim tile, the V fragment comes transposed out of the row-major rows
#pragma unroll
        for (int kt = 0; kt < 4; ++kt)
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
                uint32_t b0, b1;
                const unsigned addr = (unsigned)__cvta_generic_to_shared(vs + (kt * 16 + (lane & 15)) * kCaPitch + dt * 8);
                asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(addr));
                ca_mma(o[dt], pa[kt], b0, b1);
            }
    }
    // out [B][T][H * 64] fp16
    const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
    const int r0 = q0 + g, r1 = q0 + g + 8;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) {
        if (r0 < T)
            *reinterpret_cast<uint32_t *>(out + (((size_t)b * T + r0) * H + h) * 64 + dt * 8 + 2 * t) = pack_half2(o[dt][0] * i0, o[dt][1] * i0);
        if (r1 < T)
            *reinterpret_cast<uint32_t *>(out + (((size_t)b * T + r1) * H + h) * 64 + dt * 8 + 2 * t) = pack_half2(o[dt][2] * i1, o[dt][3] * i1);
    }
}

}  // namespace

lookat_status launch_embed(Ctx *ctx, const int32_t *ids, const __half *wte, const __half *wpe, float *x, long long rows, int T,
                           int pos0, int d, int vocab)
{
    embed_kernel<<<(unsigned)rows, 128, 0, ctx->stream>>>(ids, wte, wpe, x, rows, T, pos0, d, vocab);
    return check_launch(ctx, "embed_kernel");
}

lookat_status launch_layernorm(Ctx *ctx, const float *x, const __half *g, const __half *b, __half *y, long long rows, int d)
{
    if (d > 32 * kLnormPerLane) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "layernorm: rows of more than 1024 elements");
    layernorm_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, ctx->stream>>>(x, g, b, y, rows, d, 1e-5f);
    return check_launch(ctx, "layernorm_kernel");
}

lookat_status launch_argmax(Ctx *ctx, const float *logits, int32_t *out, int rows, int n)
{
    argmax_kernel<<<rows, kAmThreads, 0, ctx->stream>>>(logits, out, n);
    return check_launch(ctx, "argmax_kernel");
}

lookat_status launch_causal_attention(Ctx *ctx, const __half *q, const __half *k, const __half *v, __half *out, int B, int H, int T,
                                      long long v_cap)
{
    dim3 grid((unsigned)((T + kCaBlock - 1) / kCaBlock), (unsigned)H, (unsigned)B);
    causal_attention_kernel<<<grid, kCaThreads, 0, ctx->stream>>>(q, k, v, out, H, T, v_cap, 0.125f * 1.4426950408889634f);
    return check_launch(ctx, "causal_attention_kernel");
}

}  // namespace lookat
