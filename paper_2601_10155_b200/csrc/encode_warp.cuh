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

// Where the centroids of one codebook (K rows of d_sub floats) are read from.
struct GlobalBook {                    // row-major in global memory
    const float *p;
    int d_sub;
    __device__ __forceinline__ float4 load4(int c, int i) const
    {
        return __ldg(reinterpret_cast<const float4 *>(p + (size_t)c * d_sub + i));
    }
    __device__ __forceinline__ float load1(int c, int i) const { return __ldg(p + (size_t)c * d_sub + i); }
};

// Position (in 16-byte pieces) of piece `c4` of row `e` in a codebook staged in shared memory: rows stay where they
// are, the n_c = d_sub / 4 pieces of a row are permuted so that eight consecutive rows read the same piece from
// eight different 16-byte bank groups.  n_c must be 1, 2, 4, 8 or 16.
__device__ __forceinline__ int staged_shift(int n_c) { return n_c >= 8 ? 0 : (n_c == 4 ? 1 : (n_c == 2 ? 2 : 3)); }
__device__ __forceinline__ int staged_piece(int e, int c4, int n_c, int shift)
{
    return c4 ^ ((e >> shift) & (n_c - 1));
}

struct StagedBook {                    // a head's codebooks staged in shared memory; this codebook starts at row row0
    const float *p;
    int row0, d_sub, n_c, shift;
    __device__ __forceinline__ float4 load4(int c, int i) const
    {
        const int e = row0 + c;
        return *reinterpret_cast<const float4 *>(p + e * d_sub + staged_piece(e, i >> 2, n_c, shift) * 4);
    }
    __device__ __forceinline__ float load1(int c, int i) const
    {
        const int e = row0 + c;
        return p[e * d_sub + staged_piece(e, i >> 2, n_c, shift) * 4 + (i & 3)];
    }
};

// The code of one key sub-vector from the fp32 squared distances dj[0..K) of all centroids, formed as in the warp search
// below (difference form, fmaf in dimension order), by one warp: the two smallest decide; where they are within kBand the
// centroids within twice the band of the smallest are decided again in fp64 -- no other centroid can be the fp64 minimum,
// the fp32 error being below (d_sub + 2) 2^-24 relative -- lowest index first.  Every lane returns the code.
template <class Book>
__device__ __forceinline__ int code_from_distances(const float *dj, const float *x, const Book &book, int K, int d_sub, int lane)
{
    float d[8];
    Best r;
    r.best = INFINITY; r.second = INFINITY; r.idx = 0x7fffffff;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int c = lane + 32 * k;
        d[k] = c < K ? dj[c] : INFINITY;
        if (c < K) consider(r, d[k], c);
    }
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
    if (needs_fp64(r)) {                               // warp-uniform
        const float limit = r.best * (1.f + 2.f * kBand);
        double best = INFINITY;
        int idx = 0x7fffffff;
#pragma unroll 1
        for (int k = 0; k < 8; ++k) {
            const int c = lane + 32 * k;
            if (c < K && d[k] <= limit) {
                double dd = 0.0;
                for (int i = 0; i < d_sub; ++i) {
                    const double t = (double)x[i] - (double)book.load1(c, i);
                    dd = __dadd_rn(dd, __dmul_rn(t, t));      // product and sum rounded separately
                }
                if (dd < best) { best = dd; idx = c; }
            }
        }
        for (int s = 16; s; s >>= 1) {
            const double ob = __shfl_xor_sync(0xffffffffu, best, s);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, s);
            if (ob < best || (ob == best && oi < idx)) { best = ob; idx = oi; }
        }
        code = idx;
    }
    return code;
}

// the key sub-vector as fp16 (global memory) or already widened to fp32 (shared memory): both exact
__device__ __forceinline__ float key_dim(const __half *x, int i) { return __half2float(x[i]); }
__device__ __forceinline__ float key_dim(const float *x, int i) { return x[i]; }

// One (key sub-vector, codebook) search by a whole warp: lane l owns centroids l, l+32, ...
// Every lane returns the code; *near_tie (if given) tells whether the fp64 gap of the two best
// distances lies in (0, kNearTie).
template <class Book, class KeyT>
__device__ __forceinline__ int nearest_centroid_warp_in(const KeyT *x, const Book &book, int K, int d_sub,
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
            const float x0 = key_dim(x, i), x1 = key_dim(x, i + 1);
            const float x2 = key_dim(x, i + 2), x3 = key_dim(x, i + 3);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int c = lane + 32 * k;
                if (c < K) {
                    const float4 cv = book.load4(c, i);
                    float t = x0 - cv.x; d[k] = fmaf(t, t, d[k]);
                    t = x1 - cv.y; d[k] = fmaf(t, t, d[k]);
                    t = x2 - cv.z; d[k] = fmaf(t, t, d[k]);
                    t = x3 - cv.w; d[k] = fmaf(t, t, d[k]);
                }
            }
        }
    } else {
        for (int i = 0; i < d_sub; ++i) {
            const float xi = key_dim(x, i);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int c = lane + 32 * k;
                if (c < K) {
                    const float t = xi - book.load1(c, i);
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
        // the lane's (up to 8) centroids side by side: eight independent sums, each taken in dimension order
        double dd[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) dd[k] = 0.0;
        for (int i = 0; i < d_sub; ++i) {
            const double xd = (double)key_dim(x, i);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int c = lane + 32 * k;
                if (c < K) {
                    const double t = xd - (double)book.load1(c, i);
                    dd[k] = __dadd_rn(dd[k], __dmul_rn(t, t));      // product and sum rounded separately
                }
            }
        }
        double best = INFINITY, second = INFINITY;
        int idx = 0x7fffffff;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int c = lane + 32 * k;
            if (c < K) {
                if (dd[k] < best) { second = best; best = dd[k]; idx = c; }
                else if (dd[k] < second) second = dd[k];
            }
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

__device__ __forceinline__ int nearest_centroid_warp(const __half *x, const float *book, int K, int d_sub,
                                                     int lane, bool *near_tie)
{
    return nearest_centroid_warp_in(x, GlobalBook{book, d_sub}, K, d_sub, lane, near_tie);
}

}  // namespace lookat
