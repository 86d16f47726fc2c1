// Bulk nearest-centroid encoding on the tensor cores (Section 3.4 "Encoding", and the assignment
// step of "Prototype Learning").  The batched key-by-centroid inner products are the dense
// contraction of this step:
//     || x - c ||^2 = ||x||^2 + s(c),     s(c) = ||c||^2 - 2 x.c,     argmin_c s(c).
// x (fp16) is exact as an MMA operand; -2c (fp32) is split into two fp16 planes (its rounding and
// what the rounding left over), and ||c||^2 enters as the accumulator's initial value, so one chain
// of mma.sync.m16n8k16 per 16 keys x 8 centroids leaves s(c) itself in the accumulators.  The low 8
// bits of every score are then replaced by the centroid's index, which turns the search for the two
// smallest scores into plain float min/max.  The winner of this fast search is accepted only when
// its margin over the runner-up exceeds a bound on the search's own error; every other key (near
// ties, duplicate centroids, non-finite input) is decided again by the exact rule of encode_warp.cuh
// (fp32 difference form, fp64 inside its band), so the codes equal the fp64 argmin with lowest index
// on ties.
//
// One CTA: one (batch row, KV head), one subspace, up to 1024 keys; its 8 warps take 32 keys at a time
// (two 16-row operand tiles share each centroid fragment).  Shared memory holds, per centroid and
// lane-in-group t, the words that lane needs as one 16-byte (d_sub 8: 8-byte) fragment, and per
// 8-centroid tile the four initial accumulator values of each t.
#include "common.cuh"
#include "encode_warp.cuh"

namespace lookat {

namespace {

constexpr int kMmaWarps = 8;
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kMmaKeysPerWarpStep = 32;
constexpr int kMmaStepsPerCta = 4;

// Error of a fast score, for the winner w and for the true nearest centroid c* (both have
// ||c|| <= R = ||x|| + dist(x, w), and |s| <= Q = max(||x||^2, dist(x, w)^2)):
//   ||c||^2 summed in fp32                      <= 32 * 2^-24 ||c||^2          <= 2^-19 R^2
//   what the two fp16 planes of -2c leave out   <= 2^-22 ||x|| ||c||           <= 2^-22 R^2
//                                                  + 2^-25 per term (fp16 subnormal floor)
//   up to 4 chained MMAs, each taken to err by 8 units in the last place of the largest partial sum
//                                               <= 2^-18 (||c||^2 + 2 ||x|| ||c||) <= 3 * 2^-18 R^2
//   the 8 bits given to the index               <= 2^-15 |s|                   <= 2^-15 Q
// in total < 1.4e-5 R^2 + 3.1e-5 Q + 1e-6 ||x||.  The winner is accepted when its margin exceeds twice
// that, with a tenth added because R and Q are themselves computed from the fast score.
constexpr float kMmaErrR2 = 3.1e-5f;
constexpr float kMmaErrQ = 6.9e-5f;
constexpr float kMmaErrX = 2.2e-6f;
constexpr float kMmaMaxCentroid = 30000.f;   // |-2c| must stay inside fp16 range

template <int D_SUB>
struct MmaShape {
    static constexpr int kSteps = D_SUB >= 16 ? D_SUB / 16 : 1;            // k-steps of 16 dims
    static constexpr int kFragWords = D_SUB >= 16 ? 4 : 2;                 // words per (centroid, t) fragment
};

// D = A.B + C, C given as its own four registers
__device__ __forceinline__ void enc_mma_init(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1,
                                             const float4 &c)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c.x), "f"(c.y), "f"(c.z), "f"(c.w));
}

__device__ __forceinline__ void enc_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float min3(float a, float b, float c)
{
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// score with its low 8 mantissa bits replaced by the centroid index
__device__ __forceinline__ float tag(float s, int c)
{
    return __uint_as_float((__float_as_uint(s) & 0xffffff00u) | (uint32_t)c);
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

// KMEANS: the assignment step of Lloyd's iteration (cluster sums, counts, distortion) on top of the codes
template <int D_SUB, bool KMEANS>
__global__ void __launch_bounds__(kMmaThreads, 2)
encode_mma_kernel(EncodeArgs a, int H_kv, int d_k, int m, int K, int steps_per_cta)
{
    using S = MmaShape<D_SUB>;
    extern __shared__ __align__(16) uint32_t sm_words[];
    const int n_cols = (K + 7) & ~7;                                   // centroid columns, whole n-tiles
    uint32_t *frag = sm_words;                                         // [kSteps][n_cols][4 t][kFragWords]
    float *cn4 = reinterpret_cast<float *>(frag + S::kSteps * n_cols * 4 * S::kFragWords);   // [n_cols/8][4 t][4]
    // k-means mode: this CTA's share of the per-cluster sums and counts, flushed to global memory once at the end
    unsigned long long *sums_s = reinterpret_cast<unsigned long long *>(cn4 + 2 * n_cols);   // [K][D_SUB]
    unsigned *cnt_s = reinterpret_cast<unsigned *>(sums_s + (size_t)K * D_SUB);               // [K]
    __shared__ int s_force_exact;
    __shared__ double s_red[kMmaWarps];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int j = blockIdx.y, bh = blockIdx.z, h = bh % H_kv;
    const int problem = h * m + j;
    const float *book = a.codebooks + (size_t)problem * K * D_SUB;

    // ---- planes of -2c in fragment order, and ||c||^2 as initial accumulators ----
    if (tid == 0) s_force_exact = 0;
    if (KMEANS) {
        for (int e = tid; e < K * D_SUB; e += kMmaThreads) sums_s[e] = 0ull;
        for (int e = tid; e < K; e += kMmaThreads) cnt_s[e] = 0u;
    }
    __syncthreads();
    for (int c = tid; c < n_cols; c += kMmaThreads) {
        float norm = 0.f;
        bool bad = false;
        for (int w = 0; w < D_SUB / 2; ++w) {
            float v0 = 0.f, v1 = 0.f;
            if (c < K) {
                v0 = book[(size_t)c * D_SUB + 2 * w];
                v1 = book[(size_t)c * D_SUB + 2 * w + 1];
            }
            norm = fmaf(v0, v0, fmaf(v1, v1, norm));
            bad = bad || !(fabsf(v0) < kMmaMaxCentroid) || !(fabsf(v1) < kMmaMaxCentroid);
            v0 *= -2.f;
            v1 *= -2.f;
            const __half h0 = __float2half_rn(v0), h1 = __float2half_rn(v1);
            const __half l0 = __float2half_rn(v0 - __half2float(h0)), l1 = __float2half_rn(v1 - __half2float(h1));
            const uint32_t hi = (uint32_t)__half_as_ushort(h0) | ((uint32_t)__half_as_ushort(h1) << 16);
            const uint32_t lo = (uint32_t)__half_as_ushort(l0) | ((uint32_t)__half_as_ushort(l1) << 16);
            if (D_SUB >= 16) {
                // lane t of a group takes words t and t+4 of each k-step: {hi, hi+4, lo, lo+4}
                const int ks = w >> 3, r = w & 7;
                uint32_t *f = frag + ((size_t)(ks * n_cols + c) * 4 + (r & 3)) * 4 + (r >> 2);
                f[0] = hi;
                f[2] = lo;
            } else {
                // d_sub 8: one k-step holds both planes, {hi, lo} of word t
                uint32_t *f = frag + ((size_t)c * 4 + w) * 2;
                f[0] = hi;
                f[1] = lo;
            }
        }
        // columns beyond K keep a large finite score (an infinity would turn into a NaN when tagged)
        const float cn = c < K ? norm : 3.0e38f;
        float *q = cn4 + ((c >> 3) * 4 + ((c & 7) >> 1)) * 4 + (c & 1);
        q[0] = cn;
        q[2] = cn;
        if (bad) s_force_exact = 1;                       // outside fp16 range: every key takes the exact path
    }
    __syncthreads();
    const bool force_exact = s_force_exact != 0;

    double dsum = 0.0;
    const long long cta_key0 = (long long)blockIdx.x * steps_per_cta * (kMmaWarps * kMmaKeysPerWarpStep);
    // operand words of the 2 x 16 keys of a step: rows g and g+8 of each tile, dims 2t,2t+1 (+8) per k-step
    auto fetch_keys = [&](long long key0, uint32_t (&dst)[2][S::kSteps][4]) {
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                long long key = key0 + u * 16 + g + rr * 8;
                if (key >= a.n) key = a.n - 1;              // clamped rows are computed and dropped
                const __half *row = a.keys + ((size_t)bh * a.n + key) * d_k + j * D_SUB;
#pragma unroll
                for (int ks = 0; ks < S::kSteps; ++ks) {
                    const uint32_t w0 = *reinterpret_cast<const uint32_t *>(row + ks * 16 + 2 * t);
                    // d_sub 8: the second half of the k-step meets the remainder plane, so it repeats x
                    uint32_t w1 = w0;
                    if (D_SUB >= 16) w1 = *reinterpret_cast<const uint32_t *>(row + ks * 16 + 2 * t + 8);
                    dst[u][ks][rr] = w0;                    // a0 (row g) / a1 (row g+8)
                    dst[u][ks][2 + rr] = w1;                // a2 / a3
                }
            }
    };
    uint32_t xa_next[2][S::kSteps][4];
    {
        const long long first = cta_key0 + (long long)warp * kMmaKeysPerWarpStep;
        if (first < a.n) fetch_keys(first, xa_next);
    }
    for (int step = 0; step < steps_per_cta; ++step) {
        const long long key0 = cta_key0 + ((long long)step * kMmaWarps + warp) * kMmaKeysPerWarpStep;
        if (key0 >= a.n) break;                            // warp-uniform
        // ---- this step's keys arrived while the previous step searched; the next step's are requested now ----
        uint32_t xa[2][S::kSteps][4];
        float xnorm[2][2];
        const __half *rowp[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int ks = 0; ks < S::kSteps; ++ks)
#pragma unroll
                for (int i = 0; i < 4; ++i) xa[u][ks][i] = xa_next[u][ks][i];
        {
            const long long next0 = key0 + (long long)kMmaWarps * kMmaKeysPerWarpStep;
            if (step + 1 < steps_per_cta && next0 < a.n) fetch_keys(next0, xa_next);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                long long key = key0 + u * 16 + g + rr * 8;
                if (key >= a.n) key = a.n - 1;
                rowp[u][rr] = a.keys + ((size_t)bh * a.n + key) * d_k + j * D_SUB;
                float nn = 0.f;
#pragma unroll
                for (int ks = 0; ks < S::kSteps; ++ks) {
                    const float2 f0 = __half22float2(*reinterpret_cast<const __half2 *>(&xa[u][ks][rr]));
                    nn += f0.x * f0.x + f0.y * f0.y;
                    if (D_SUB >= 16) {
                        const float2 f1 = __half22float2(*reinterpret_cast<const __half2 *>(&xa[u][ks][2 + rr]));
                        nn += f1.x * f1.x + f1.y * f1.y;
                    }
                }
                nn += __shfl_xor_sync(0xffffffffu, nn, 1);
                nn += __shfl_xor_sync(0xffffffffu, nn, 2);
                xnorm[u][rr] = nn;
            }

        float best[2][2], second[2][2];                     // tagged scores
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) best[u][rr] = second[u][rr] = INFINITY;

        // ---- all centroids, 8 at a time ----
        for (int nt = 0; nt < n_cols / 8; ++nt) {
            float acc[2][4];
            const float4 cq = *reinterpret_cast<const float4 *>(cn4 + (nt * 4 + t) * 4);
            if (D_SUB >= 16) {
#pragma unroll
                for (int ks = 0; ks < S::kSteps; ++ks) {
                    const uint4 f = *reinterpret_cast<const uint4 *>(frag + ((size_t)(ks * n_cols + nt * 8 + g) * 4 + t) * 4);
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        if (ks == 0) enc_mma_init(acc[u], xa[u][0], f.x, f.y, cq);
                        else enc_mma(acc[u], xa[u][ks], f.x, f.y);
                        enc_mma(acc[u], xa[u][ks], f.z, f.w);
                    }
                }
            } else {
                const uint2 f = *reinterpret_cast<const uint2 *>(frag + ((size_t)(nt * 8 + g) * 4 + t) * 2);
#pragma unroll
                for (int u = 0; u < 2; ++u) enc_mma_init(acc[u], xa[u][0], f.x, f.y, cq);
            }
            const int c0 = nt * 8 + 2 * t;
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const float d0 = tag(acc[u][2 * rr], c0), d1 = tag(acc[u][2 * rr + 1], c0 + 1);
                    const float lo = fminf(d0, d1), hi = fmaxf(d0, d1);
                    second[u][rr] = min3(second[u][rr], hi, fmaxf(best[u][rr], lo));
                    best[u][rr] = fminf(best[u][rr], lo);
                }
        }

        // ---- the 4 lanes of a row merge; rows whose margin is inside the error bound are redone exactly ----
        int code[2][2];
        unsigned redo[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                float b = best[u][rr], s = second[u][rr];
#pragma unroll
                for (int sh = 1; sh <= 2; sh <<= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, b, sh);
                    const float os = __shfl_xor_sync(0xffffffffu, s, sh);
                    s = min3(s, os, fmaxf(b, ob));
                    b = fminf(b, ob);
                }
                code[u][rr] = (int)(__float_as_uint(b) & 0xffu);
                const float x2 = xnorm[u][rr];
                const float dw2 = fmaxf(b + x2, 0.f);       // squared distance to the winner
                const float r = sqrtf(x2) + sqrtf(dw2);
                const float err = kMmaErrR2 * r * r + kMmaErrQ * fmaxf(x2, dw2) + kMmaErrX * sqrtf(x2);
                const bool unsure = force_exact || !(s - b > err);      // also true when anything is not a number
                // rows past the end were clamped to the last key: they are dropped, so they are not redone (nor counted)
                const bool exists = key0 + u * 16 + g + rr * 8 < a.n;
                redo[u][rr] = __ballot_sync(0xffffffffu, unsure && t == 0 && exists);
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
                    const int exact = exact_code_warp(reinterpret_cast<const __half *>((uintptr_t)p), book, K, D_SUB,
                                                      lane, &tie);
                    if (lane == src) {
                        code[u][rr] = exact;
                        tie_count += tie;
                    }
                }
            }

        // ---- store: lane t = 0 of a row writes its code; for k-means the four lanes of a row add the dims they hold ----
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const long long key = key0 + u * 16 + g + rr * 8;
                const int cd = __shfl_sync(0xffffffffu, code[u][rr], lane & ~3);     // the exact path told lane t = 0 only
                if (key >= a.n) continue;
                if (t == 0) a.codes[((size_t)bh * a.L_max + a.pos + key) * m + j] = (uint8_t)cd;
                if (KMEANS) {
                    unsigned long long *srow = sums_s + (size_t)cd * D_SUB;
#pragma unroll
                    for (int ks = 0; ks < S::kSteps; ++ks) {
                        const __half2 w0 = *reinterpret_cast<const __half2 *>(&xa[u][ks][rr]);
                        atomicAdd(srow + ks * 16 + 2 * t, (unsigned long long)half_to_fixed24(__low2half(w0)));
                        atomicAdd(srow + ks * 16 + 2 * t + 1, (unsigned long long)half_to_fixed24(__high2half(w0)));
                        if (D_SUB >= 16) {
                            const __half2 w1 = *reinterpret_cast<const __half2 *>(&xa[u][ks][2 + rr]);
                            atomicAdd(srow + ks * 16 + 2 * t + 8, (unsigned long long)half_to_fixed24(__low2half(w1)));
                            atomicAdd(srow + ks * 16 + 2 * t + 9, (unsigned long long)half_to_fixed24(__high2half(w1)));
                        }
                    }
                    if (t == 0) {
                        atomicAdd(cnt_s + cd, 1u);
                        if (a.distortion) dsum += dist_fp64(rowp[u][rr], book + (size_t)cd * D_SUB, D_SUB);
                    }
                }
            }
        if (t == 0 && tie_count && a.near_ties) atomicAdd(a.near_ties, (unsigned long long)tie_count);
    }

    if (KMEANS) {                                           // flush this CTA's share
        __syncthreads();
        unsigned long long *gs = a.sums + (size_t)problem * K * D_SUB;
        for (int e = tid; e < K * D_SUB; e += kMmaThreads) {
            const unsigned long long v = sums_s[e];
            if (v) atomicAdd(gs + e, v);
        }
        for (int e = tid; e < K; e += kMmaThreads) {
            const unsigned c = cnt_s[e];
            if (c) atomicAdd(a.cnt + (size_t)problem * K + e, (unsigned long long)c);
        }
    }

    if (KMEANS && a.distortion) {                           // uniform over the grid
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
    // k-means mode keeps a CTA's share of the cluster sums in shared memory and gives it more keys to amortise the flush
    const int steps = a.sums ? 4 * kMmaStepsPerCta : kMmaStepsPerCta;
    const size_t smem = (size_t)n_cols * (MmaShape<D_SUB>::kSteps * 4 * MmaShape<D_SUB>::kFragWords + 2) * 4 +
                        (a.sums ? (size_t)c.K * D_SUB * 8 + (size_t)c.K * 4 : 0);
    auto kern = a.sums ? encode_mma_kernel<D_SUB, true> : encode_mma_kernel<D_SUB, false>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "encode: shared-memory opt-in");
    const long long per_cta = (long long)steps * kMmaWarps * kMmaKeysPerWarpStep;
    dim3 grid((unsigned)((a.n + per_cta - 1) / per_cta), c.m, a.B * c.n_kv_heads);
    kern<<<grid, kMmaThreads, smem, ctx->stream>>>(a, c.n_kv_heads, c.d_k, c.m, c.K, steps);
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
