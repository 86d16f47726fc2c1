// Nearest-centroid encoding (Section 3.4 "Encoding"):
//   code[t][j] = argmin_c || k_t^(j) - C_j[c] ||^2,  lowest index on ties,
// and the assignment step of Lloyd's algorithm (Section 3.4 "Prototype
// Learning"), which is the same search plus per-cluster sums.
//
// Distances are evaluated in the difference form in fp32 (a fp16 key widens
// exactly).  Its relative error is below (d_sub+2)*2^-24 < 1e-5 for every
// supported d_sub, so whenever the two smallest fp32 distances differ by more
// than 1e-4 relative the fp32 winner is the true argmin; otherwise the search
// is repeated in fp64 with first-minimum-wins.  The result therefore equals
// the fp64 argmin, including the lowest-index rule for duplicate centroids.
//
// Kernels:
//   encode_tile_kernel<D_SUB,KPT>  bulk: a CTA holds one codebook in shared
//       memory and scores 256*KPT keys of one (batch row, KV head) against it,
//       key sub-vectors in registers, centroid reads are broadcasts.
//   encode_any_kernel              bulk, any d_sub: keys staged in shared memory.
//   encode_warp_kernel             few keys (decode append): one warp per
//       (key, subspace), lanes split the centroids, codebooks read from L2.
#include "common.cuh"
#include "encode_warp.cuh"

namespace lookat {

namespace {

// What follows a decision: store the code, count near ties, and in k-means mode add the key
// to its cluster's exact sums and its fp64 distance to the distortion.
__device__ __forceinline__ double finish_key(const EncodeArgs &a, const __half *x, const float *book,
                                             int problem, int K, int d_sub, size_t code_index,
                                             const Best &r)
{
    int code = r.idx;
    double d64 = -1.0;
    if (needs_fp64(r)) {
        bool tie;
        code = search_fp64(x, book, K, d_sub, &d64, &tie);
        if (tie && a.near_ties) atomicAdd(a.near_ties, 1ull);
    }
    a.codes[code_index] = (uint8_t)code;
    if (a.sums) {
        unsigned long long *s = a.sums + ((size_t)problem * K + code) * d_sub;
        for (int i = 0; i < d_sub; ++i) atomicAdd(s + i, (unsigned long long)half_to_fixed24(x[i]));
        atomicAdd(a.cnt + (size_t)problem * K + code, 1ull);
        if (d64 < 0.0) d64 = dist_fp64(x, book + (size_t)code * d_sub, d_sub);
        return d64;
    }
    return 0.0;
}

__device__ __forceinline__ void add_distortion(const EncodeArgs &a, int problem, double d)
{
    if (!a.distortion) return;                       // uniform over the grid
    __shared__ double red[32];
    for (int s = 16; s; s >>= 1) d += __shfl_xor_sync(0xffffffffu, d, s);
    const int warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    if ((threadIdx.x & 31) == 0) red[warp] = d;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < nwarps; ++w) t += red[w];
        atomicAdd(a.distortion + (size_t)problem * a.distortion_stride, t);
    }
}

constexpr int kEncThreads = 256;

template <int D_SUB, int KPT>
__global__ void __launch_bounds__(kEncThreads)
encode_tile_kernel(EncodeArgs a, int H_kv, int d_k, int m, int K)
{
    extern __shared__ __align__(16) float book_s[];      // [K][D_SUB]
    const int j = blockIdx.y;
    const int bh = blockIdx.z;
    const int h = bh % H_kv;
    const int problem = h * m + j;
    const float *book = a.codebooks + (size_t)problem * K * D_SUB;
    for (int i = threadIdx.x; i < K * D_SUB; i += kEncThreads) book_s[i] = book[i];
    __syncthreads();

    const long long t_first = (long long)blockIdx.x * (kEncThreads * KPT) + threadIdx.x;
    float x[KPT][D_SUB];
    Best r[KPT];
#pragma unroll
    for (int kk = 0; kk < KPT; ++kk) {
        const long long t = t_first + (long long)kk * kEncThreads;
        r[kk].best = INFINITY; r[kk].second = INFINITY; r[kk].idx = 0;
        const __half *row = a.keys + ((size_t)bh * a.n + (t < a.n ? t : 0)) * d_k + j * D_SUB;
#pragma unroll
        for (int i = 0; i < D_SUB; ++i) x[kk][i] = __half2float(row[i]);
    }

    for (int c = 0; c < K; ++c) {
        float d[KPT];
#pragma unroll
        for (int kk = 0; kk < KPT; ++kk) d[kk] = 0.f;
#pragma unroll
        for (int i = 0; i < D_SUB; ++i) {
            const float cv = book_s[c * D_SUB + i];
#pragma unroll
            for (int kk = 0; kk < KPT; ++kk) {
                const float t = x[kk][i] - cv;
                d[kk] = fmaf(t, t, d[kk]);
            }
        }
#pragma unroll
        for (int kk = 0; kk < KPT; ++kk) consider(r[kk], d[kk], c);
    }

    double dsum = 0.0;
#pragma unroll
    for (int kk = 0; kk < KPT; ++kk) {
        const long long t = t_first + (long long)kk * kEncThreads;
        if (t < a.n) {
            const __half *row = a.keys + ((size_t)bh * a.n + t) * d_k + j * D_SUB;
            dsum += finish_key(a, row, book, problem, K, D_SUB,
                               ((size_t)bh * a.L_max + a.pos + t) * m + j, r[kk]);
        }
    }
    add_distortion(a, problem, dsum);
}

// Any d_sub: one thread per key, the key tile and (when it fits) the codebook in shared memory.
constexpr int kAnyThreads = 128;

__global__ void __launch_bounds__(kAnyThreads)
encode_any_kernel(EncodeArgs a, int H_kv, int d_k, int m, int K, int book_in_smem)
{
    extern __shared__ __align__(16) float sm[];
    const int d_sub = d_k / m;
    const int xs_stride = d_sub + 1;
    float *xs = sm;                                       // [kAnyThreads][d_sub+1]
    float *book_s = sm + kAnyThreads * xs_stride;         // [K][d_sub] when book_in_smem
    const int j = blockIdx.y, bh = blockIdx.z, h = bh % H_kv;
    const int problem = h * m + j;
    const float *book = a.codebooks + (size_t)problem * K * d_sub;
    if (book_in_smem)
        for (int i = threadIdx.x; i < K * d_sub; i += kAnyThreads) book_s[i] = book[i];
    const long long t = (long long)blockIdx.x * kAnyThreads + threadIdx.x;
    const __half *row = a.keys + ((size_t)bh * a.n + (t < a.n ? t : 0)) * d_k + j * d_sub;
    for (int i = 0; i < d_sub; ++i) xs[threadIdx.x * xs_stride + i] = __half2float(row[i]);
    __syncthreads();

    const float *cb = book_in_smem ? book_s : book;
    Best r;
    r.best = INFINITY; r.second = INFINITY; r.idx = 0;
    for (int c = 0; c < K; ++c) {
        float d = 0.f;
        for (int i = 0; i < d_sub; ++i) {
            const float tt = xs[threadIdx.x * xs_stride + i] - cb[(size_t)c * d_sub + i];
            d = fmaf(tt, tt, d);
        }
        consider(r, d, c);
    }
    double dsum = 0.0;
    if (t < a.n)
        dsum = finish_key(a, row, book, problem, K, d_sub, ((size_t)bh * a.L_max + a.pos + t) * m + j, r);
    add_distortion(a, problem, dsum);
}

// Few keys: one warp per (key, subspace).
constexpr int kWarpKernelThreads = 128;

__global__ void __launch_bounds__(kWarpKernelThreads)
encode_warp_kernel(EncodeArgs a, int H_kv, int d_k, int m, int K, long long n_tasks)
{
    const long long task = (long long)blockIdx.x * (kWarpKernelThreads / 32) + (threadIdx.x >> 5);
    if (task >= n_tasks) return;                          // whole warp leaves together
    const int lane = threadIdx.x & 31;
    const int d_sub = d_k / m;
    const int j = (int)(task % m);
    const long long key = task / m;                       // bh * n + t
    const long long t = key % a.n;
    const int bh = (int)(key / a.n), h = bh % H_kv;
    const int problem = h * m + j;
    const float *book = a.codebooks + (size_t)problem * K * d_sub;
    const __half *x = a.keys + (size_t)key * d_k + j * d_sub;

    bool tie;
    const int code = nearest_centroid_warp(x, book, K, d_sub, lane, &tie);
    if (lane == 0 && tie && a.near_ties) atomicAdd(a.near_ties, 1ull);
    if (lane == 0) a.codes[((size_t)bh * a.L_max + a.pos + t) * m + j] = (uint8_t)code;
}

template <int D_SUB, int KPT>
lookat_status launch_tile(Ctx *ctx, const EncodeArgs &a)
{
    const lookat_config &c = ctx->cfg;
    const size_t smem = (size_t)c.K * D_SUB * sizeof(float);
    auto kern = encode_tile_kernel<D_SUB, KPT>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "encode: shared-memory opt-in");
    const long long per_cta = (long long)kEncThreads * KPT;
    dim3 grid((unsigned)((a.n + per_cta - 1) / per_cta), c.m, a.B * c.n_kv_heads);
    kern<<<grid, kEncThreads, smem, ctx->stream>>>(a, c.n_kv_heads, c.d_k, c.m, c.K);
    return check_launch(ctx, "encode_tile_kernel");
}

}  // namespace

lookat_status launch_encode(Ctx *ctx, const EncodeArgs &a)
{
    const lookat_config &c = ctx->cfg;
    const int d_sub = c.d_k / c.m;
    const long long n_tasks = (long long)a.B * c.n_kv_heads * a.n * c.m;
    if (n_tasks == 0) return LOOKAT_OK;
    if (!a.sums && n_tasks <= 16384) {
        const int wpb = kWarpKernelThreads / 32;
        encode_warp_kernel<<<(unsigned)((n_tasks + wpb - 1) / wpb), kWarpKernelThreads, 0, ctx->stream>>>(
            a, c.n_kv_heads, c.d_k, c.m, c.K, n_tasks);
        return check_launch(ctx, "encode_warp_kernel");
    }
    if (encode_mma_covers(ctx, a)) return launch_encode_mma(ctx, a);
    switch (d_sub) {
        case 4: return launch_tile<4, 4>(ctx, a);
        case 8: return launch_tile<8, 4>(ctx, a);
        case 16: return launch_tile<16, 2>(ctx, a);
        case 32: return launch_tile<32, 1>(ctx, a);
        default: break;
    }
    size_t smem_x = (size_t)kAnyThreads * (d_sub + 1) * sizeof(float);
    size_t smem_book = (size_t)c.K * d_sub * sizeof(float);
    int book_in_smem = smem_x + smem_book <= (size_t)ctx->max_smem_optin;
    size_t smem = smem_x + (book_in_smem ? smem_book : 0);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(encode_any_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
        return check_launch(ctx, "encode: shared-memory opt-in");
    dim3 grid((unsigned)((a.n + kAnyThreads - 1) / kAnyThreads), c.m, a.B * c.n_kv_heads);
    encode_any_kernel<<<grid, kAnyThreads, smem, ctx->stream>>>(a, c.n_kv_heads, c.d_k, c.m, c.K, book_in_smem);
    return check_launch(ctx, "encode_any_kernel");
}

}  // namespace lookat
