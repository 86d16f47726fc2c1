// Bulk nearest-centroid encoding on the tensor cores (Section 3.4 "Encoding", and the assignment
// step of "Prototype Learning").  The batched key-by-centroid inner products are the dense
// contraction of this step:
//     || x - c ||^2 = ||x||^2 + ( ||c||^2 - 2 x.c ),     argmin_c of the bracket.
// x (fp16) is exact as an MMA operand; every fp32 centroid is split into two fp16 planes (its
// rounding and what the rounding left over), so x.c is carried to ~22 bits with fp32 accumulation:
// two mma.sync.m16n8k16 per 16 keys x 8 centroids.  The winner of this fast search is accepted only
// when its margin over the runner-up exceeds a bound on the search's own error; every other key
// (near ties, duplicate centroids) is decided again by the exact rule of encode_warp.cuh (fp32
// difference form, fp64 inside its band), so the codes equal the fp64 argmin with lowest index on ties.
//
// One CTA: one (batch row, KV head), one subspace, up to 1024 keys; its 8 warps take 32 keys at a time
// (two 16-row operand tiles share each centroid fragment).  The centroid planes sit in shared memory,
// centroid-major with a row pitch chosen so that the fragment reads are bank-conflict free.
#include "common.cuh"
#include "encode_warp.cuh"

namespace lookat {

namespace {

constexpr int kMmaWarps = 8;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kMmaKeysPerWarpStep = 32;
constexpr int kMmaStepsPerCta = 4;
constexpr int kMmaKeysPerCta = kMmaWarps * kMmaKeysPerWarpStep * kMmaStepsPerCta;   // 1024
// Margin below which the fast winner is not trusted: kMmaBand * ||x|| * (||x|| + ||c_best||).
// A fast score errs by at most e(c) = 2 * 64 * 2^-23 * ||x|| ||c|| < 1.6e-5 ||x|| ||c|| (up to 64 exact
// products accumulated in fp32, plus the 2^-22 split error).  A centroid with ||c|| > 2||x|| + ||c_best||
// is farther than the winner whatever its error; for all others e(c) + e(c_best) stays below
// 1.6e-5 * ||x|| * (2||x|| + 2||c_best||) < the margin required here.
constexpr float kMmaBand = 6.0e-5f;

template <int D_SUB>
struct MmaShape {
    static constexpr int kSteps = D_SUB >= 16 ? D_SUB / 16 : 1;            // k-steps of 16 dims
    static constexpr int kWords = D_SUB / 2;                               // 32-bit words per centroid row
    // row pitch in words: 8 rows x 4 lanes must land in 32 different banks
    static constexpr int kPitch = D_SUB == 8 ? 4 : (D_SUB == 16 ? 12 : 20);
};

__device__ __forceinline__ void enc_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The exact rule for one (key, subspace), by the whole warp; out of line (it is the rare path).
__device__ __noinline__ int exact_code_warp(const __half *x, const float *book, int K, int d_sub, int lane,
                                            int *tie_out)
{
    bool tie;
    const int code = nearest_centroid_warp(x, book, K, d_sub, lane, &tie);
    *tie_out = tie ? 1 : 0;
    return code;
}

// smaller distance wins, then smaller index; the loser's best is a runner-up
__device__ __forceinline__ void merge_best(Best &r, float ob, float os, int oi)
{
    const bool other_wins = ob < r.best || (ob == r.best && oi < r.idx);
    const float loser = other_wins ? r.best : ob;
    r.second = fminf(fminf(r.second, os), loser);
    if (other_wins) {
        r.best = ob;
        r.idx = oi;
    }
}

template <int D_SUB>
__global__ void __launch_bounds__(kMmaThreads)
encode_mma_kernel(EncodeArgs a, int H_kv, int d_k, int m, int K)
{
    using S = MmaShape<D_SUB>;
    extern __shared__ __align__(16) uint32_t sm_words[];
    const int n_cols = (K + 7) & ~7;                                   // centroid columns, whole n-tiles
    uint32_t *c_hi = sm_words;                                         // [n_cols][kPitch]
    uint32_t *c_lo = c_hi + n_cols * S::kPitch;
    float *c_norm = reinterpret_cast<float *>(c_lo + n_cols * S::kPitch);   // [n_cols], +inf beyond K
    __shared__ int s_force_exact;
    __shared__ double s_red[kMmaWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int j = blockIdx.y, bh = blockIdx.z, h = bh % H_kv;
    const int problem = h * m + j;
    const float *book = a.codebooks + (size_t)problem * K * D_SUB;

    // ---- centroid planes and norms ----
    if (tid == 0) s_force_exact = 0;
    __syncthreads();
    for (int c = tid; c < n_cols; c += kMmaThreads) {
        float norm = 0.f;
        bool bad = false;
        for (int w = 0; w < S::kWords; ++w) {
            float v0 = 0.f, v1 = 0.f;
            if (c < K) {
                v0 = book[(size_t)c * D_SUB + 2 * w];
                v1 = book[(size_t)c * D_SUB + 2 * w + 1];
            }
            norm = fmaf(v0, v0, fmaf(v1, v1, norm));
            const __half h0 = __float2half_rn(v0), h1 = __float2half_rn(v1);
            const __half l0 = __float2half_rn(v0 - __half2float(h0)), l1 = __float2half_rn(v1 - __half2float(h1));
            bad = bad || !(fabsf(v0) < 60000.f) || !(fabsf(v1) < 60000.f);
            c_hi[c * S::kPitch + w] = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
            c_lo[c * S::kPitch + w] = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
        }
        c_norm[c] = c < K ? norm : INFINITY;
        if (bad) s_force_exact = 1;                       // outside fp16 range: every key takes the exact path
    }
    __syncthreads();
    const bool force_exact = s_force_exact != 0;

    double dsum = 0.0;
    const long long cta_key0 = (long long)blockIdx.x * kMmaKeysPerCta;
    for (int step = 0; step < kMmaStepsPerCta; ++step) {
        const long long key0 = cta_key0 + ((long long)step * kMmaWarps + warp) * kMmaKeysPerWarpStep;
        if (key0 >= a.n) break;                            // warp-uniform
        // ---- operand tiles of 2 x 16 keys: rows g and g+8 of each, dims 2t,2t+1 (+8) per k-step ----
        uint32_t xa[2][S::kSteps][4];
        float xnorm[2][2];
        const __half *rowp[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                long long key = key0 + u * 16 + g + rr * 8;
                if (key >= a.n) key = a.n - 1;              // clamped rows are computed and dropped
                rowp[u][rr] = a.keys + ((size_t)bh * a.n + key) * d_k + j * D_SUB;
                float nn = 0.f;
#pragma unroll
                for (int ks = 0; ks < S::kSteps; ++ks) {
                    const uint32_t w0 = *reinterpret_cast<const uint32_t *>(rowp[u][rr] + ks * 16 + 2 * t);
                    uint32_t w1 = 0u;
                    if (D_SUB >= 16) w1 = *reinterpret_cast<const uint32_t *>(rowp[u][rr] + ks * 16 + 2 * t + 8);
                    xa[u][ks][rr] = w0;                     // a0 (row g) / a1 (row g+8)
                    xa[u][ks][2 + rr] = w1;                 // a2 / a3: dims +8
                    const float2 f0 = __half22float2(*reinterpret_cast<const __half2 *>(&w0));
                    const float2 f1 = __half22float2(*reinterpret_cast<const __half2 *>(&w1));
                    nn += f0.x * f0.x + f0.y * f0.y + f1.x * f1.x + f1.y * f1.y;
                }
                nn += __shfl_xor_sync(0xffffffffu, nn, 1);
                nn += __shfl_xor_sync(0xffffffffu, nn, 2);
                xnorm[u][rr] = nn;
            }

        Best best[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                best[u][rr].best = INFINITY;
                best[u][rr].second = INFINITY;
                best[u][rr].idx = 0x7fffffff;
            }

        // ---- all centroids, 8 at a time ----
        for (int nt = 0; nt < n_cols / 8; ++nt) {
            float acc[2][4];
#pragma unroll
            for (int u = 0; u < 2; ++u) acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0.f;
            const uint32_t *bh_row = c_hi + (nt * 8 + g) * S::kPitch + t;
            const uint32_t *bl_row = c_lo + (nt * 8 + g) * S::kPitch + t;
#pragma unroll
            for (int ks = 0; ks < S::kSteps; ++ks) {
                const uint32_t h0 = bh_row[ks * 8], l0 = bl_row[ks * 8];
                const uint32_t h1 = D_SUB >= 16 ? bh_row[ks * 8 + 4] : 0u, l1 = D_SUB >= 16 ? bl_row[ks * 8 + 4] : 0u;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    enc_mma(acc[u], xa[u][ks], h0, h1);
                    enc_mma(acc[u], xa[u][ks], l0, l1);
                }
            }
            const float2 cn = *reinterpret_cast<const float2 *>(c_norm + nt * 8 + 2 * t);
            const int c0 = nt * 8 + 2 * t;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                consider(best[u][0], fmaf(-2.f, acc[u][0], cn.x), c0);
                consider(best[u][0], fmaf(-2.f, acc[u][1], cn.y), c0 + 1);
                consider(best[u][1], fmaf(-2.f, acc[u][2], cn.x), c0);
                consider(best[u][1], fmaf(-2.f, acc[u][3], cn.y), c0 + 1);
            }
        }

        // ---- the 4 lanes of a row merge; rows whose margin is inside the error bound are redone exactly ----
        unsigned redo[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                Best &r = best[u][rr];
#pragma unroll
                for (int s = 1; s <= 2; s <<= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, r.best, s);
                    const float os = __shfl_xor_sync(0xffffffffu, r.second, s);
                    const int oi = __shfl_xor_sync(0xffffffffu, r.idx, s);
                    merge_best(r, ob, os, oi);
                }
                const float xn = sqrtf(xnorm[u][rr]);
                const float cb = sqrtf(c_norm[r.idx < n_cols ? r.idx : 0]);
                const bool unsure = force_exact || !(r.second - r.best > kMmaBand * xn * (xn + cb));
                redo[u][rr] = __ballot_sync(0xffffffffu, unsure && t == 0);
            }
        int tie_count = 0;
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                unsigned todo = redo[u][rr];
                while (todo) {                              // warp-uniform loop over the flagged rows
                    const int src = __ffs(todo) - 1;        // lane (g', t = 0) that owns the row
                    todo &= todo - 1;
                    const unsigned long long p =
                        __shfl_sync(0xffffffffu, (unsigned long long)(uintptr_t)rowp[u][rr], src);
                    int tie;
                    const int code = exact_code_warp(reinterpret_cast<const __half *>((uintptr_t)p), book, K, D_SUB,
                                                     lane, &tie);
                    if (lane == src) {
                        best[u][rr].idx = code;
                        tie_count += tie;
                    }
                }
            }

        // ---- store: lane t = 0 of a row writes its code (and, for k-means, adds the key to its cluster) ----
        if (t == 0) {
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const long long key = key0 + u * 16 + g + rr * 8;
                    if (key >= a.n) continue;
                    const int code = best[u][rr].idx;
                    a.codes[((size_t)bh * a.L_max + a.pos + key) * m + j] = (uint8_t)code;
                    if (a.sums) {
                        const __half *x = rowp[u][rr];
                        unsigned long long *s = a.sums + ((size_t)problem * K + code) * D_SUB;
#pragma unroll
                        for (int i = 0; i < D_SUB; ++i)
                            atomicAdd(s + i, (unsigned long long)half_to_fixed24(x[i]));
                        atomicAdd(a.cnt + (size_t)problem * K + code, 1ull);
                        if (a.distortion) dsum += dist_fp64(x, book + (size_t)code * D_SUB, D_SUB);
                    }
                }
            if (tie_count && a.near_ties) atomicAdd(a.near_ties, (unsigned long long)tie_count);
        }
    }

    if (a.distortion) {                                     // uniform over the grid
        for (int s = 16; s; s >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, s);
        if (lane == 0) s_red[warp] = dsum;
        __syncthreads();
        if (tid == 0) {
            double tot = 0.0;
            for (int w = 0; w < kMmaWarps; ++w) tot += s_red[w];
            atomicAdd(a.distortion + (size_t)problem * a.distortion_stride, tot);
        }
    }
}

template <int D_SUB>
lookat_status launch_mma(Ctx *ctx, const EncodeArgs &a)
{
    const lookat_config &c = ctx->cfg;
    const int n_cols = (c.K + 7) & ~7;
    const size_t smem = (size_t)n_cols * (2 * MmaShape<D_SUB>::kPitch + 1) * 4;
    auto kern = encode_mma_kernel<D_SUB>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "encode: shared-memory opt-in");
    dim3 grid((unsigned)((a.n + kMmaKeysPerCta - 1) / kMmaKeysPerCta), c.m, a.B * c.n_kv_heads);
    kern<<<grid, kMmaThreads, smem, ctx->stream>>>(a, c.n_kv_heads, c.d_k, c.m, c.K);
    return check_launch(ctx, "encode_mma_kernel");
}

}  // namespace

bool encode_mma_covers(const Ctx *ctx, const EncodeArgs &a)
{
    const lookat_config &c = ctx->cfg;
    const int d_sub = c.d_k / c.m;
    // 4-byte operand loads: key rows and sub-vectors must start on even half indices
    return (d_sub == 8 || d_sub == 16 || d_sub == 32) && (c.d_k & 1) == 0 && ((uintptr_t)a.keys & 3) == 0;
}

lookat_status launch_encode_mma(Ctx *ctx, const EncodeArgs &a)
{
    switch (ctx->cfg.d_k / ctx->cfg.m) {
        case 8: return launch_mma<8>(ctx, a);
        case 16: return launch_mma<16>(ctx, a);
        default: return launch_mma<32>(ctx, a);
    }
}

}  // namespace lookat
