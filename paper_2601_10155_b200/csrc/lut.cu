// Lookup tables (Section 3.5 "Precomputation Lookup Tables"; Algorithm 1, first
// loop):  lut[b][hq][j][c] = q^(j) . C_j[c],  unscaled.
//
// One thread per table entry.  fp16 x fp32 products are exact in fp64, so the
// fp64 accumulation leaves a single rounding (to fp32) in every entry.  The
// work is K*d_k multiply-adds per (query, head) and reads the codebooks once
// per batch row from L2; it is the small step of a decode pass.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kLutThreads = 256;

__global__ void __launch_bounds__(kLutThreads)
build_lut_kernel(const __half *__restrict__ q, const float *__restrict__ codebooks,
                 float *__restrict__ lut, int H_q, int g, int d_k, int m, int K)
{
    extern __shared__ double qs[];                     // the query of this (b, hq), widened
    const int hq = blockIdx.y, b = blockIdx.z;
    const int d_sub = d_k / m;
    const __half *qrow = q + ((size_t)b * H_q + hq) * d_k;
    for (int i = threadIdx.x; i < d_k; i += kLutThreads) qs[i] = (double)__half2float(qrow[i]);
    __syncthreads();

    const int e = blockIdx.x * kLutThreads + threadIdx.x;   // entry j*K + c
    if (e >= m * K) return;
    const int j = e / K;
    const float *cen = codebooks + ((size_t)(hq / g) * m * K + e) * d_sub;
    const double *qj = qs + j * d_sub;
    double acc = 0.0;
    if ((d_sub & 3) == 0) {
        for (int i = 0; i < d_sub; i += 4) {
            const float4 c4 = *reinterpret_cast<const float4 *>(cen + i);
            acc = fma(qj[i], (double)c4.x, acc);
            acc = fma(qj[i + 1], (double)c4.y, acc);
            acc = fma(qj[i + 2], (double)c4.z, acc);
            acc = fma(qj[i + 3], (double)c4.w, acc);
        }
    } else {
        for (int i = 0; i < d_sub; ++i) acc = fma(qj[i], (double)cen[i], acc);
    }
    lut[((size_t)b * H_q + hq) * m * K + e] = (float)acc;
}

}  // namespace

lookat_status launch_build_lut(Ctx *ctx, const __half *q, int B, const float *codebooks, float *lut)
{
    const lookat_config &c = ctx->cfg;
    dim3 grid((c.m * c.K + kLutThreads - 1) / kLutThreads, c.n_q_heads, B);
    build_lut_kernel<<<grid, kLutThreads, c.d_k * sizeof(double), ctx->stream>>>(
        q, codebooks, lut, c.n_q_heads, c.n_q_heads / c.n_kv_heads, c.d_k, c.m, c.K);
    return check_launch(ctx, "build_lut_kernel");
}

}  // namespace lookat
