// Codebook learning (Section 3.4 "Prototype Learning"): Lloyd's algorithm per
// (KV head, subspace).  The assignment step lives in encode.cu (it is the
// encoding search, which also adds each key to its cluster's sums); this file
// holds the start rule and the centroid update.
//
// Sums are exact: every fp16 is an integer multiple of 2^-24, so the members
// of a cluster are added as 64-bit integers (order independent), and the new
// centroid is  float( double(sum) * 2^-24 / double(count) ).
#include "common.cuh"

namespace lookat {

namespace {

// Start: either the caller's centroids, or pooled key rows (off + c*stride) mod N.
__global__ void fit_init_kernel(const __half *__restrict__ keys, int B, long long n, int H_kv, int d_k,
                                int m, int K, unsigned long long seed, const float *__restrict__ init,
                                float *__restrict__ codebooks)
{
    const int d_sub = d_k / m;
    const long long total = (long long)H_kv * m * K * d_sub;
    const unsigned long long N = (unsigned long long)B * (unsigned long long)n;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        if (init) {
            codebooks[e] = init[e];
            continue;
        }
        const int i = (int)(e % d_sub);
        const int c = (int)((e / d_sub) % K);
        const int problem = (int)(e / ((long long)d_sub * K));
        const int h = problem / m, j = problem % m;
        const unsigned long long off = (seed + 0x9E3779B97F4A7C15ull * (unsigned long long)(problem + 1)) % N;
        const unsigned long long stride = (N / (unsigned long long)K) > 0 ? N / (unsigned long long)K : 1;
        const unsigned long long r = (off + (unsigned long long)c * stride) % N;
        const unsigned long long b = r / (unsigned long long)n, t = r % (unsigned long long)n;
        codebooks[e] = __half2float(keys[((b * H_kv + h) * (unsigned long long)n + t) * d_k + j * d_sub + i]);
    }
}

// New centroid = exact mean of its members; a cluster without members keeps its centroid.
// Clears the sums for the next iteration (codebooks == null: only clears).
__global__ void fit_update_kernel(unsigned long long *__restrict__ sums, unsigned long long *__restrict__ cnt,
                                  float *__restrict__ codebooks, long long clusters, int d_sub)
{
    const long long total = clusters * d_sub;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const unsigned long long count = cnt[e / d_sub];
        if (codebooks && count) {
            const double s = (double)(long long)sums[e];
            codebooks[e] = (float)(ldexp(s, -24) / (double)count);
        }
        sums[e] = 0ull;
    }
}

__global__ void fit_clear_counts_kernel(unsigned long long *__restrict__ cnt, long long clusters)
{
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < clusters;
         e += (long long)gridDim.x * blockDim.x)
        cnt[e] = 0ull;
}

}  // namespace

lookat_status launch_fit_init(Ctx *ctx, const __half *keys, int B, long long n, uint64_t seed,
                              const float *init, float *codebooks)
{
    const lookat_config &c = ctx->cfg;
    const long long total = (long long)c.n_kv_heads * c.K * c.d_k;
    const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
    fit_init_kernel<<<blocks, 256, 0, ctx->stream>>>(keys, B, n, c.n_kv_heads, c.d_k, c.m, c.K,
                                                     (unsigned long long)seed, init, codebooks);
    return check_launch(ctx, "fit_init_kernel");
}

lookat_status launch_fit_update(Ctx *ctx, float *codebooks)
{
    const lookat_config &c = ctx->cfg;
    const long long clusters = (long long)c.n_kv_heads * c.m * c.K;
    const long long total = clusters * (c.d_k / c.m);
    const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
    fit_update_kernel<<<blocks, 256, 0, ctx->stream>>>(ctx->fit_sums, ctx->fit_cnt, codebooks, clusters,
                                                       c.d_k / c.m);
    lookat_status st = check_launch(ctx, "fit_update_kernel");
    if (st != LOOKAT_OK) return st;
    const int cblocks = (int)((clusters + 255) / 256 < 1024 ? (clusters + 255) / 256 : 1024);
    fit_clear_counts_kernel<<<cblocks, 256, 0, ctx->stream>>>(ctx->fit_cnt, clusters);
    return check_launch(ctx, "fit_clear_counts_kernel");
}

}  // namespace lookat
