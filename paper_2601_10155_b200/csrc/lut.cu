// Lookup tables (Section 3.5 "Precomputation Lookup Tables"; Algorithm 1, first
// loop):  lut[b][hq][j][c] = q^(j) . C_j[c],  unscaled.
//
// fp16 x fp32 products are exact in fp64, so the fp64 accumulation (in the order of
// the dims) leaves a single rounding (to fp32) in every entry.  The work is K*d_k
// multiply-adds per (query, head) and reads the codebooks from L2; it is the small
// step of a decode pass.
//
// One thread per (KV head, subspace, centroid) and batch row: it reads the centroid
// once, widens it once and forms the entries of all query heads of the group from
// it (up to four at a time, their query dims side by side in shared memory: one
// 16-byte read serves two heads).  The widening (a conversion per element, on the
// quarter-rate pipe) and the address arithmetic are what a thread per single entry
// spent its time on.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kLutThreads = 256;
constexpr int kLutHeads = 4;           // query heads of a group formed side by side

__global__ void __launch_bounds__(kLutThreads)
build_lut_kernel(const __half *__restrict__ q, const float *__restrict__ codebooks,
                 float *__restrict__ lut, int H_q, int g, int d_k, int m, int K)
{
    extern __shared__ __align__(16) double qs[];       // [ceil(g/4)][d_k][4]: the group's queries, widened, head fastest
    const int kvh = blockIdx.y, b = blockIdx.z;
    const int d_sub = d_k / m;
    const int chunks = (g + kLutHeads - 1) / kLutHeads;
    const int e = blockIdx.x * kLutThreads + threadIdx.x;   // entry j*K + c
    const bool live = e < m * K;
    const float *cen = codebooks + ((size_t)kvh * m * K + (live ? e : 0)) * d_sub;
    const bool vec = (d_sub & 3) == 0;

    // the first 16 dims of the centroid are requested before the queries are staged: one round trip, not two
    float4 pre[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
        pre[u] = (live && vec && 4 * u < d_sub) ? __ldg(reinterpret_cast<const float4 *>(cen) + u) : make_float4(0.f, 0.f, 0.f, 0.f);

    const __half *qrow = q + ((size_t)b * H_q + kvh * g) * d_k;     // the group's g query rows are contiguous
    for (int ch = 0; ch < chunks; ++ch) {
        for (int x = threadIdx.x; x < d_k * kLutHeads; x += kLutThreads) {
            const int hg = ch * kLutHeads + (x & (kLutHeads - 1)), dim = x / kLutHeads;
            qs[ch * d_k * kLutHeads + x] = hg < g ? (double)__half2float(qrow[hg * d_k + dim]) : 0.0;
        }
    }
    __syncthreads();
    if (!live) return;

    const int j = e / K;
    for (int ch = 0; ch < chunks; ++ch) {
        const double *qj = qs + ((size_t)ch * d_k + j * d_sub) * kLutHeads;
        double acc[kLutHeads] = {0.0, 0.0, 0.0, 0.0};
        auto add4 = [&](int i, const float4 &c4) {         // dims i .. i+3, in order
            const double c[4] = {(double)c4.x, (double)c4.y, (double)c4.z, (double)c4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const double2 q01 = *reinterpret_cast<const double2 *>(qj + (i + u) * kLutHeads);
                const double2 q23 = *reinterpret_cast<const double2 *>(qj + (i + u) * kLutHeads + 2);
                acc[0] = fma(q01.x, c[u], acc[0]), acc[1] = fma(q01.y, c[u], acc[1]);
                acc[2] = fma(q23.x, c[u], acc[2]), acc[3] = fma(q23.y, c[u], acc[3]);
            }
        };
        if (vec) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (4 * u < d_sub) add4(4 * u, pre[u]);
            }
            for (int i = 16; i < d_sub; i += 4) add4(i, __ldg(reinterpret_cast<const float4 *>(cen + i)));
        } else {
            for (int i = 0; i < d_sub; ++i) {
                const double c = (double)__ldg(cen + i);
#pragma unroll
                for (int h = 0; h < kLutHeads; ++h) acc[h] = fma(qj[i * kLutHeads + h], c, acc[h]);
            }
        }
#pragma unroll
        for (int h = 0; h < kLutHeads; ++h) {
            const int hg = ch * kLutHeads + h;
            if (hg < g) lut[((size_t)b * H_q + kvh * g + hg) * m * K + e] = (float)acc[h];
        }
    }
}

}  // namespace

lookat_status launch_build_lut(Ctx *ctx, const __half *q, int B, const float *codebooks, float *lut)
{
    const lookat_config &c = ctx->cfg;
    const int g = c.n_q_heads / c.n_kv_heads;
    const size_t smem = (size_t)((g + kLutHeads - 1) / kLutHeads) * kLutHeads * c.d_k * sizeof(double);
    if (smem > (size_t)ctx->max_smem_optin)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "build_lut: %d heads of %d dims per KV head do not fit in shared memory", g, c.d_k);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(build_lut_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "build_lut: shared-memory opt-in");
    dim3 grid((c.m * c.K + kLutThreads - 1) / kLutThreads, c.n_kv_heads, B);
    build_lut_kernel<<<grid, kLutThreads, smem, ctx->stream>>>(q, codebooks, lut, c.n_q_heads, g, c.d_k, c.m, c.K);
    return check_launch(ctx, "build_lut_kernel");
}

}  // namespace lookat
