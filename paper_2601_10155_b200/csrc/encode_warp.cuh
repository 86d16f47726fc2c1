// Nearest-centroid search shared by the encoding kernels (Section 3.4 "Encoding"): the decision
// rule (fp32 difference-form distances, re-taken in fp64 when the two best are within kBand) and
// the warp-cooperative search used where few keys are encoded at a time.
#pragma once

#include "common.cuh"

namespace lookat {

constexpr float kBand = 1.0e-4f;     // fp32 decisions closer than this are re-taken in fp64
constexpr double kNearTie = 1.0e-6;  // reporting threshold for near ties (relative gap)

struct Best {
    float best, second;
    int idx;
};

__device__ __forceinline__ void consider(Best &r, float d, int c)
{
    if (d < r.best) {
        r.second = r.best;
        r.best = d;
        r.idx = c;
    } else if (d < r.second) {
        r.second = d;
    }
}

__device__ __forceinline__ bool needs_fp64(const Best &r)
{
    return !(r.second - r.best > kBand * r.second);
}

// Full search in fp64 by one thread; first minimum wins.  Returns the code, the
// winning distance, and whether the two best distances form a near tie.
static __device__ int search_fp64(const __half *x, const float *book, int K, int d_sub, double *best_out,
                           bool *near_tie)
{
    double best = INFINITY, second = INFINITY;
    int idx = 0;
    for (int c = 0; c < K; ++c) {
        double acc = 0.0;
        for (int i = 0; i < d_sub; ++i) {
            const double t = (double)__half2float(x[i]) - (double)book[(size_t)c * d_sub + i];
            acc = __dadd_rn(acc, __dmul_rn(t, t));      // product and sum rounded separately
        }
        if (acc < best) {
            second = best;
            best = acc;
            idx = c;
        } else if (acc < second) {
            second = acc;
        }
    }
    *best_out = best;
    const double gap = (K < 2) ? INFINITY : (second == 0.0 ? 0.0 : (second - best) / second);
    *near_tie = gap > 0.0 && gap < kNearTie;
    return idx;
}

static __device__ double dist_fp64(const __half *x, const float *cen, int d_sub)
{
    double acc = 0.0;
    for (int i = 0; i < d_sub; ++i) {
        const double t = (double)__half2float(x[i]) - (double)cen[i];
        acc = __dadd_rn(acc, __dmul_rn(t, t));
    }
    return acc;
}

// One (key sub-vector, codebook) search by a whole warp: lane l owns centroids l, l+32, ...
// Every lane returns the code; *near_tie (if given) tells whether the fp64 gap of the two best
// distances lies in (0, kNearTie).
__device__ __forceinline__ int nearest_centroid_warp(const __half *x, const float *book, int K, int d_sub,
                                                     int lane, bool *near_tie)
{
    // lane l owns centroids l, l+32, ... (at most 8, K <= 256); dimensions in the outer loop so
    // that the lane's centroid loads of one step are independent of each other
    float d[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) d[k] = 0.f;
    if ((d_sub & 3) == 0) {
#pragma unroll 2
        for (int i = 0; i < d_sub; i += 4) {
            const float x0 = __half2float(x[i]), x1 = __half2float(x[i + 1]);
            const float x2 = __half2float(x[i + 2]), x3 = __half2float(x[i + 3]);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int c = lane + 32 * k;
                if (c < K) {
                    const float4 cv = __ldg(reinterpret_cast<const float4 *>(book + (size_t)c * d_sub + i));
                    float t = x0 - cv.x; d[k] = fmaf(t, t, d[k]);
                    t = x1 - cv.y; d[k] = fmaf(t, t, d[k]);
                    t = x2 - cv.z; d[k] = fmaf(t, t, d[k]);
                    t = x3 - cv.w; d[k] = fmaf(t, t, d[k]);
                }
            }
        }
    } else {
        for (int i = 0; i < d_sub; ++i) {
            const float xi = __half2float(x[i]);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int c = lane + 32 * k;
                if (c < K) {
                    const float t = xi - __ldg(book + (size_t)c * d_sub + i);
                    d[k] = fmaf(t, t, d[k]);
                }
            }
        }
    }
    Best r;
    r.best = INFINITY; r.second = INFINITY; r.idx = 0x7fffffff;
#pragma unroll
    for (int k = 0; k < 8; ++k)
        if (lane + 32 * k < K) consider(r, d[k], lane + 32 * k);
    // merge lanes: smaller distance wins, then smaller index; the loser's best is a runner-up
    for (int s = 16; s; s >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, r.best, s);
        const float os = __shfl_xor_sync(0xffffffffu, r.second, s);
        const int oi = __shfl_xor_sync(0xffffffffu, r.idx, s);
        const bool other_wins = ob < r.best || (ob == r.best && oi < r.idx);
        const float loser = other_wins ? r.best : ob;
        r.second = fminf(fminf(r.second, os), loser);
        if (other_wins) { r.best = ob; r.idx = oi; }
    }
    int code = r.idx;
    bool tie = false;
    if (needs_fp64(r)) {
        double best = INFINITY, second = INFINITY;
        int idx = 0x7fffffff;
        for (int c = lane; c < K; c += 32) {
            const double d = dist_fp64(x, book + (size_t)c * d_sub, d_sub);
            if (d < best) { second = best; best = d; idx = c; }
            else if (d < second) second = d;
        }
        for (int s = 16; s; s >>= 1) {
            const double ob = __shfl_xor_sync(0xffffffffu, best, s);
            const double os = __shfl_xor_sync(0xffffffffu, second, s);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, s);
            const bool other_wins = ob < best || (ob == best && oi < idx);
            const double loser = other_wins ? best : ob;
            second = fmin(fmin(second, os), loser);
            if (other_wins) { best = ob; idx = oi; }
        }
        code = idx;
        const double gap = (K < 2) ? INFINITY : (second == 0.0 ? 0.0 : (second - best) / second);
        tie = gap > 0.0 && gap < kNearTie;
    }
    if (near_tie) *near_tie = tie;
    return code;
}

}  // namespace lookat
