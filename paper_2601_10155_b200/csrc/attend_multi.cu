// Streaming attend kernel for rows of up to a few thousand tokens (Section 3.5 "Lookup and Sum"; Algorithm 1,
// second loop and continuation; Section 3.4 "Encoding" for the appended key).
//
// Same work decomposition as attend_stream_kernel (attend.cu) -- the flat sequence of (unit, 16-token tile) pairs
// cut into one contiguous range per persistent CTA, 16 warps taking tiles round-robin through private cp.async
// rings, scores from tables in shared memory, P.V on mma.sync -- but organised so that what a unit costs besides
// its bytes is paid once per CTA, not once per unit.  With short rows a CTA's range crosses several units, and a
// table build, two block-wide merges and a counter round trip per unit are then most of the time.  Here:
//   * units are ordered KV head first, so the units of a range share their codebooks; the head's codebooks are
//     staged in shared memory once (when they fit), pieces of a row permuted so that reads are conflict free;
//   * a ROUND covers up to `ut` consecutive units of one KV head: their tables are built together at the start of
//     the round (each centroid is widened once and meets the queries of every unit of the round), the warps then
//     stream the round's tiles without any block-wide barrier -- a warp that crosses into the next unit writes its
//     partial (max, sum, weighted values) of the unit it leaves to shared memory and switches tables -- and the
//     units' partials are merged together at the end of the round;
//   * a unit that lies wholly inside the CTA's range is written to the output directly; only a unit shared with a
//     neighbouring CTA (the first or last of a range) goes through global partials and its arrival counter;
//   * the key appended by a decode step is encoded at the start of the round that holds its tile, by the whole CTA
//     (distances to all centroids from the staged codebooks, then one warp per (unit, subspace) takes the decision),
//     stored to the cache, and handed to the warp that scores that tile through shared memory, so no copy has to
//     wait for the store.
// The phases outside the token loop are out of line (their registers are their own) and written for few
// instructions: with 16 warps per CTA every instruction of such a phase is issued 16 times.
#include <type_traits>

#include "common.cuh"
#include "attend_tile.cuh"
#include "encode_warp.cuh"

namespace lookat {

namespace {

// position in the CTA's range of the flat tile sequence (t counts from the range's first tile) with the unit's row
// facts; units are ordered (KV head, head group, batch row)
struct MCursor {
    int t;
    int unit, lt;
    int len;
    size_t row0;         // first token of the tile, as a row index into the code and value caches
};

struct UnitId {
    int b, kvh, hgrp;
};

__device__ __forceinline__ UnitId unit_id(const AttendArgs &a, int unit, int hgroups)
{
    UnitId u;
    const int per_head = hgroups * a.B;
    u.kvh = unit / per_head;
    const int r = unit - u.kvh * per_head;
    u.hgrp = r / a.B;
    u.b = r - u.hgrp * a.B;
    return u;
}

template <int M_SUB, int DV>
__device__ __forceinline__ void mc_enter_unit(const AttendArgs &a, MCursor &c, int hgroups)
{
    if (c.unit < a.n_units) {
        const UnitId u = unit_id(a, c.unit, hgroups);
        c.len = (int)min((long long)(a.seq_lens ? a.seq_lens[u.b] : a.uniform_len), a.L_max);
        c.row0 = ((size_t)u.b * a.H_kv + u.kvh) * a.L_max + (size_t)c.lt * kTile;
    } else {
        c.len = 0;
    }
}

template <int M_SUB, int DV>
__device__ __forceinline__ void mc_advance(const AttendArgs &a, MCursor &c, int hgroups)
{
    c.t += kWarps;
    c.lt += kWarps;
    c.row0 += kWarps * kTile;
    if (c.lt >= a.tiles_per_unit) {
        do {
            c.lt -= a.tiles_per_unit;
            c.unit += 1;
        } while (c.lt >= a.tiles_per_unit);
        mc_enter_unit<M_SUB, DV>(a, c, hgroups);
    }
}

__device__ __forceinline__ int mc_valid(const MCursor &c)
{
    const int left = c.len - c.lt * kTile;
    return left >= kTile ? kTile : (left > 0 ? left : 0);
}

// shared-memory areas (offsets come with the kernel's arguments)
#define MS_TABLES(a, sm) (reinterpret_cast<float *>((sm) + (a).lay.tables))        /* [ut][heads_max][head_stride] */
#define MS_PARTIALS(a, sm) (reinterpret_cast<float *>((sm) + (a).lay.partials))    /* [ut][kWarps][heads_max][d_v + 2] */
#define MS_Q(a, sm) (reinterpret_cast<double *>((sm) + (a).lay.q))                 /* [ut][d_k][QH] */
#define MS_XK(a, sm) (reinterpret_cast<float *>((sm) + (a).lay.xk))                /* [ut][d_k] appended keys, widened */
#define MS_NEWC(a, sm) ((sm) + (a).lay.newc)                                        /* [ut][16] appended codes */
#define MS_BOOK(a, sm) (reinterpret_cast<float *>((sm) + (a).lay.book))

// The units of a round, decoded once (by the first threads) for everyone: batch row and head group; the KV head is
// the round's.
struct RoundUnits {
    int b[kMaxRoundUnits], hgrp[kMaxRoundUnits];
};

// What the out-of-line phases need of the kernel's arguments, read once into registers: the arguments sit in
// constant memory behind a reference there, and a field read through it is re-read after every store.
struct RoundFacts {
    int H_q, H_kv, g, heads_max, d_k, d_v, m, K, d_sub, table, head_stride, QH, set_floats, tiles_per_unit;
    __device__ __forceinline__ explicit RoundFacts(const AttendArgs &a)
    {
        H_q = a.H_q; H_kv = a.H_kv; g = a.g;
        heads_max = g < 4 ? g : 4;
        d_k = a.d_k; d_v = a.d_v; m = a.m; K = a.K;
        d_sub = d_k / m;
        table = m * K;
        head_stride = m * kTableStride + kHeadPad;
        QH = a.stage_book ? (g == 1 ? 1 : (g == 2 ? 2 : 4)) : 4;
        set_floats = a.lay.set_floats;
        tiles_per_unit = a.tiles_per_unit;
    }
};

// The round's queries widened to fp64, its appended keys widened to fp32, and every (unit, warp) partial marked
// "nothing seen".
__device__ __noinline__ void round_fill(const AttendArgs &a, unsigned char *sm, const RoundUnits *ru, int kvh, int nr)
{
    const int tid = threadIdx.x;
    const RoundFacts f(a);
    const __half *qg = a.lut ? nullptr : a.q;              // (ready tables need no queries)
    const __half *kg = a.new_keys;
    double *q_s = MS_Q(a, sm);
    float *xk = MS_XK(a, sm);
    float *pa = MS_PARTIALS(a, sm);
    for (int ul = 0; ul < nr; ++ul) {
        const int b = ru->b[ul], hq0 = kvh * f.g + ru->hgrp[ul] * 4;
        const int heads_here = min(4, f.g - ru->hgrp[ul] * 4);
        if (qg) {
            const __half *qrow = qg + ((size_t)b * f.H_q + hq0) * f.d_k;
            for (int dim = tid; dim < f.d_k; dim += kThreads)
                for (int h = 0; h < f.QH; ++h)
                    q_s[((size_t)ul * f.d_k + dim) * f.QH + h] =
                        h < heads_here ? (double)__half2float(qrow[(size_t)h * f.d_k + dim]) : 0.0;
        }
        if (kg) {
            const __half *krow = kg + ((size_t)b * f.H_kv + kvh) * f.d_k;
            for (int dim = tid; dim < f.d_k; dim += kThreads) xk[ul * f.d_k + dim] = __half2float(krow[dim]);
        }
    }
    const int MG = f.d_v + 2;
    for (int i = tid; i < nr * kWarps * f.heads_max; i += kThreads) {
        pa[(size_t)i * MG + f.d_v] = kNegBig;
        pa[(size_t)i * MG + f.d_v + 1] = 0.f;
    }
}

// Section 3.5 "Precomputation Lookup Tables" for the `nr` units of a round from the staged codebooks of their KV
// head: lut[ul][h][j][c] = q_{ul,h}^(j) . C_j[c], fp64 accumulation, one rounding.  A thread owns table entries; each
// centroid is read and widened once per group of four units.  q_s is [unit][dim][QH] with QH = HEADS.
// With DIST the fp32 squared distance of every centroid to the matching sub-vector of each unit's appended key (xk,
// [unit][d_k]) goes to dist[unit][table] on the way -- formed as the warp search of encode_warp.cuh forms it (difference,
// fmaf, dimensions in order) -- so that the append needs no pass of its own over the codebooks.
template <int HEADS, bool DIST>
__device__ __forceinline__ void build_round_tables(const float *book_s, const double *q_s, float *lut_s, int nr, int table,
                                                   int K, int d_k, int d_sub, int heads_max, int set_floats, int head_stride,
                                                   int tid, const float *xk, float *dist)
{
    const int n_c = d_sub >> 2, sh = staged_shift(n_c);
    for (int e = tid; e < table; e += kThreads) {
        const int j = e / K;
        const int es = j * kTableStride + (e - j * K);
        const float *row = book_s + (size_t)e * d_sub;
        for (int ul0 = 0; ul0 < nr; ul0 += 4) {
            double t[4][HEADS];
            float dacc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int h = 0; h < HEADS; ++h) t[k][h] = 0.0;
            for (int c0 = 0; c0 < n_c; c0 += 4) {              // 16 dims at a time
                double cv[16];
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (c0 + c4 < n_c) f = *reinterpret_cast<const float4 *>(row + staged_piece(e, c0 + c4, n_c, sh) * 4);
                    cv[4 * c4] = (double)f.x; cv[4 * c4 + 1] = (double)f.y; cv[4 * c4 + 2] = (double)f.z; cv[4 * c4 + 3] = (double)f.w;
                    if constexpr (DIST) {
                        if (c0 + c4 < n_c) {
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                if (ul0 + k < nr) {
                                    const float4 xv = *reinterpret_cast<const float4 *>(xk + (ul0 + k) * d_k + j * d_sub + 4 * (c0 + c4));
                                    float d = xv.x - f.x; dacc[k] = fmaf(d, d, dacc[k]);
                                    d = xv.y - f.y; dacc[k] = fmaf(d, d, dacc[k]);
                                    d = xv.z - f.z; dacc[k] = fmaf(d, d, dacc[k]);
                                    d = xv.w - f.w; dacc[k] = fmaf(d, d, dacc[k]);
                                }
                            }
                        }
                    }
                }
                const int dims = min(16, d_sub - 4 * c0);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (ul0 + k < nr) {
                        const double *qj = q_s + ((size_t)(ul0 + k) * d_k + j * d_sub + 4 * c0) * HEADS;
                        if constexpr (HEADS == 1) {
#pragma unroll
                            for (int i = 0; i < 16; i += 2) {
                                if (i < dims) {
                                    const double2 q2 = *reinterpret_cast<const double2 *>(qj + i);
                                    t[k][0] = fma(q2.x, cv[i], t[k][0]);
                                    t[k][0] = fma(q2.y, cv[i + 1], t[k][0]);
                                }
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                if (i < dims) {
#pragma unroll
                                    for (int h = 0; h < HEADS; h += 2) {
                                        const double2 q2 = *reinterpret_cast<const double2 *>(qj + i * HEADS + h);
                                        t[k][h] = fma(q2.x, cv[i], t[k][h]);
                                        t[k][h + 1] = fma(q2.y, cv[i], t[k][h + 1]);
                                    }
                                }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (ul0 + k < nr) {
                    float *dst = lut_s + (size_t)(ul0 + k) * set_floats + es;
#pragma unroll
                    for (int h = 0; h < HEADS; ++h)
                        if (h < heads_max) dst[h * head_stride] = (float)t[k][h];
                    if constexpr (DIST) dist[(size_t)(ul0 + k) * table + e] = dacc[k];
                }
            }
        }
    }
}

// Section 3.4 "Encoding" for the appended keys of a round from the staged codebooks, by the whole CTA.  Pass 1: every
// thread takes table entries (subspace j, centroid c) and forms the fp32 squared distance of each unit's key to that
// centroid (difference form, dimensions in order: the arithmetic of nearest_centroid_warp_in) into `dist`
// [unit][set_floats].  Pass 2: one warp per (unit, subspace) finds the two smallest; where they are within kBand, the
// centroids within kBand of the smallest are decided again in fp64 (no other centroid can be the fp64 minimum: the
// fp32 error is below (d_sub + 2) 2^-24 relative), lowest index first.  `mine[ul]` tells whether this CTA's range
// holds the unit's newest token.
__device__ __forceinline__ void append_round_staged(const RoundFacts &f, const float *book_s, const float *xk, float *dist,
                                                    unsigned char *newc, uint8_t *cache, const RoundUnits *ru, int kvh,
                                                    long long L_max, int new_pos, int nr, unsigned mine)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_c = f.d_sub >> 2, sh = staged_shift(n_c);
    for (int e = tid; e < f.table; e += kThreads) {
        const int j = e / f.K;
        const float *row = book_s + (size_t)e * f.d_sub;
        float acc[kMaxRoundUnits];
#pragma unroll
        for (int ul = 0; ul < kMaxRoundUnits; ++ul) acc[ul] = 0.f;
        for (int c4 = 0; c4 < n_c; ++c4) {
            const float4 cv = *reinterpret_cast<const float4 *>(row + staged_piece(e, c4, n_c, sh) * 4);
#pragma unroll
            for (int ul = 0; ul < kMaxRoundUnits; ++ul) {
                if (ul < nr) {
                    const float4 xv = *reinterpret_cast<const float4 *>(xk + ul * f.d_k + j * f.d_sub + 4 * c4);
                    float t = xv.x - cv.x; acc[ul] = fmaf(t, t, acc[ul]);
                    t = xv.y - cv.y; acc[ul] = fmaf(t, t, acc[ul]);
                    t = xv.z - cv.z; acc[ul] = fmaf(t, t, acc[ul]);
                    t = xv.w - cv.w; acc[ul] = fmaf(t, t, acc[ul]);
                }
            }
        }
#pragma unroll
        for (int ul = 0; ul < kMaxRoundUnits; ++ul)
            if (ul < nr) dist[(size_t)ul * f.set_floats + e] = acc[ul];
    }
    __syncthreads();
    for (int task = warp; task < nr * f.m; task += kWarps) {
        const int ul = task / f.m, j = task - ul * f.m;
        if (!((mine >> ul) & 1u)) continue;
        const float *dj = dist + (size_t)ul * f.set_floats + j * f.K;
        const int code = code_from_distances(dj, xk + ul * f.d_k + j * f.d_sub, StagedBook{book_s, j * f.K, f.d_sub, n_c, sh}, f.K,
                                             f.d_sub, lane);
        if (lane == 0) {
            cache[(((size_t)ru->b[ul] * f.H_kv + kvh) * L_max + new_pos) * f.m + j] = (uint8_t)code;
            newc[ul * 16 + j] = (unsigned char)code;
        }
    }
    __syncthreads();                                       // `dist` is the table area: the tables come next
}

// Section 3.4 "Encoding" for the appended key of every unit of the round whose newest token lies in this CTA's range
// (the code goes to the cache and to the hand-over bytes in shared memory), then Section 3.5 "Precomputation Lookup
// Tables" for the round's units.
__device__ __noinline__ void round_tables(const AttendArgs &a, unsigned char *sm, const RoundUnits *ru, int kvh, int u0,
                                          int nr, int t_lo, int t_hi)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const RoundFacts f(a);
    float *lut_s = MS_TABLES(a, sm);
    const float *book_s = MS_BOOK(a, sm);
    const double *q_s = MS_Q(a, sm);
    const bool staged = a.stage_book != 0;
    const float *books_g = a.codebooks;
    const float *lut_g = a.lut;
    bool fused = false;
    unsigned mine_units = 0;
    if (a.new_keys) {
        const int new_pos = a.new_pos;
        unsigned mine = 0;                                 // units whose newest token's tile lies in this CTA's range
        for (int ul = 0; ul < nr; ++ul) {
            const int t_new = (u0 + ul) * f.tiles_per_unit + (new_pos >> 4);
            if (t_new >= t_lo && t_new < t_hi) mine |= 1u << ul;
        }
        mine_units = mine;
        // (every head group of a KV row encodes the key for itself: same code, and no unit depends on another's store)
        // A round of one unit whose partial-result area can hold the distances for the moment: the table build below forms
        // them on its way through the codebooks, and only the pick of the codes remains (with more units in the round
        // the separate pass measured faster: 30.1 against 30.8 us on the GPT-2 layer step at batch 32).
        fused = mine && staged && nr == 1 && f.table <= kWarps * f.heads_max * (f.d_v + 2);
        if (fused) {
            // nothing here: see below
        } else if (mine && staged) {
            append_round_staged(f, book_s, MS_XK(a, sm), lut_s, MS_NEWC(a, sm), a.codes_w, ru, kvh, a.L_max, new_pos, nr, mine);
        } else if (mine) {
            const float *xk = MS_XK(a, sm);
            unsigned char *newc = MS_NEWC(a, sm);
            uint8_t *cache = a.codes_w;
            const long long L_max = a.L_max;
            for (int task = warp; task < nr * f.m; task += kWarps) {
                const int ul = task / f.m, j = task - ul * f.m;
                if (!((mine >> ul) & 1u)) continue;
                const int code = nearest_centroid_warp_in(xk + ul * f.d_k + j * f.d_sub,
                                                          GlobalBook{books_g + ((size_t)kvh * f.m + j) * f.K * f.d_sub, f.d_sub},
                                                          f.K, f.d_sub, lane, nullptr);
                if (lane == 0) {
                    cache[(((size_t)ru->b[ul] * f.H_kv + kvh) * L_max + new_pos) * f.m + j] = (uint8_t)code;
                    newc[ul * 16 + j] = (unsigned char)code;
                }
            }
        }
    }
    if (staged && fused) {
        float *dist = MS_PARTIALS(a, sm);                  // [unit][table], in place of the partial results for the moment
        const float *xk = MS_XK(a, sm);
        if (f.QH == 1)
            build_round_tables<1, true>(book_s, q_s, lut_s, nr, f.table, f.K, f.d_k, f.d_sub, f.heads_max, f.set_floats, f.head_stride, tid, xk, dist);
        else if (f.QH == 2)
            build_round_tables<2, true>(book_s, q_s, lut_s, nr, f.table, f.K, f.d_k, f.d_sub, f.heads_max, f.set_floats, f.head_stride, tid, xk, dist);
        else
            build_round_tables<4, true>(book_s, q_s, lut_s, nr, f.table, f.K, f.d_k, f.d_sub, f.heads_max, f.set_floats, f.head_stride, tid, xk, dist);
        __syncthreads();
        const int n_c = f.d_sub >> 2, sh = staged_shift(n_c);
        unsigned char *newc = MS_NEWC(a, sm);
        for (int task = warp; task < nr * f.m; task += kWarps) {
            const int ul = task / f.m, j = task - ul * f.m;
            if (!((mine_units >> ul) & 1u)) continue;
            const int code = code_from_distances(dist + (size_t)ul * f.table + j * f.K, xk + ul * f.d_k + j * f.d_sub,
                                                 StagedBook{book_s, j * f.K, f.d_sub, n_c, sh}, f.K, f.d_sub, lane);
            if (lane == 0) {
                a.codes_w[(((size_t)ru->b[ul] * f.H_kv + kvh) * a.L_max + a.new_pos) * f.m + j] = (uint8_t)code;
                newc[ul * 16 + j] = (unsigned char)code;
            }
        }
        __syncthreads();
        // the area goes back to the partial results: every (unit, warp) marked "nothing seen" again
        float *pa = MS_PARTIALS(a, sm);
        const int MG = f.d_v + 2;
        for (int i = tid; i < nr * kWarps * f.heads_max; i += kThreads) {
            pa[(size_t)i * MG + f.d_v] = kNegBig;
            pa[(size_t)i * MG + f.d_v + 1] = 0.f;
        }
    } else if (staged) {
        if (f.QH == 1)
            build_round_tables<1, false>(book_s, q_s, lut_s, nr, f.table, f.K, f.d_k, f.d_sub, f.heads_max, f.set_floats, f.head_stride, tid, nullptr, nullptr);
        else if (f.QH == 2)
            build_round_tables<2, false>(book_s, q_s, lut_s, nr, f.table, f.K, f.d_k, f.d_sub, f.heads_max, f.set_floats, f.head_stride, tid, nullptr, nullptr);
        else
            build_round_tables<4, false>(book_s, q_s, lut_s, nr, f.table, f.K, f.d_k, f.d_sub, f.heads_max, f.set_floats, f.head_stride, tid, nullptr, nullptr);
    } else if (lut_g) {
        for (int ul = 0; ul < nr; ++ul) {
            const int heads_here = min(4, f.g - ru->hgrp[ul] * 4);
            for (int h = 0; h < heads_here; ++h) {
                const float *src = lut_g + ((size_t)ru->b[ul] * f.H_q + kvh * f.g + ru->hgrp[ul] * 4 + h) * f.table;
                float *dst = lut_s + (size_t)ul * f.set_floats + h * f.head_stride;
                if (f.K == kTableStride) {
                    for (int i = tid; i < (f.table >> 2); i += kThreads)
                        reinterpret_cast<float4 *>(dst)[i] = __ldg(reinterpret_cast<const float4 *>(src) + i);
                } else {
                    for (int i = tid; i < f.table; i += kThreads) {
                        const int j = i / f.K;
                        dst[j * kTableStride + (i - j * f.K)] = __ldg(src + i);
                    }
                }
            }
        }
    } else {
        for (int ul = 0; ul < nr; ++ul) {
            const int heads_here = min(4, f.g - ru->hgrp[ul] * 4);
            build_unit_tables<false>(books_g + (size_t)kvh * f.table * f.d_sub, q_s + (size_t)ul * f.d_k * 4,
                              lut_s + (size_t)ul * f.set_floats, f.table, f.K, f.d_sub, heads_here, f.head_stride, tid, nullptr, nullptr);
        }
    }
}

// End of a round: the 16 warps' partials of every unit are merged.  A unit that lies wholly inside this CTA's range goes
// to the output at once; a unit shared with a neighbouring CTA (only the first and the last of a range can be) goes to
// global partials, and the CTA that arrives last at it (a counter per unit, no waiting) merges those into the output.
__device__ __noinline__ void round_merge(const AttendArgs &a, unsigned char *sm, const RoundUnits *ru, int kvh, int u0, int nr,
                                         int t_lo, int t_hi, int *s_last)
{
    const int tid = threadIdx.x;
    const RoundFacts f(a);
    const int DV = f.d_v, MG = f.d_v + 2, heads_max = f.heads_max;
    const float *pa = MS_PARTIALS(a, sm);
    float *out = a.out, *part_o = a.part_o, *part_ml = a.part_ml;
    unsigned *tickets = a.tickets;
    const int tiles_per_cta = (int)a.tiles_per_cta;
    const int splits_per_unit = a.splits_per_unit, ctas_per_head = a.ctas_per_head;
    const int head_lo = ctas_per_head > 0 ? kvh * (((f.g + 3) >> 2) * a.B) * f.tiles_per_unit : 0;   // first tile of the KV head
    const int c = blockIdx.x;
    auto is_whole = [&](int unit) {
        const int t0 = unit * f.tiles_per_unit;
        return t0 >= t_lo && t0 + f.tiles_per_unit <= t_hi;
    };
    auto unit_ctas = [&](int unit, int *c_lo, int *c_hi) {
        if (splits_per_unit > 0) {
            *c_lo = unit * splits_per_unit;
            *c_hi = *c_lo + splits_per_unit - 1;
        } else {
            // (with per-head ranges: the CTAs of this KV head, counted from the head's first tile)
            *c_lo = kvh * ctas_per_head + (unit * f.tiles_per_unit - head_lo) / tiles_per_cta;
            *c_hi = kvh * ctas_per_head + ((unit + 1) * f.tiles_per_unit - 1 - head_lo) / tiles_per_cta;
        }
    };
    // only the first and the last unit of a range can be shared with another CTA
    const bool any_split = !is_whole(u0) || !is_whole(u0 + nr - 1);
    // thread -> (value column dv, then head, then unit): DV is a power of two times 64, so no division by it
    for (int idx = tid; idx < nr * heads_max * DV; idx += kThreads) {
        const int dv = idx & (DV - 1), uh = idx / DV;
        const int ul = uh / heads_max, h = uh - ul * heads_max;
        const int unit = u0 + ul;
        if (h >= min(4, f.g - ru->hgrp[ul] * 4)) continue;
        const float *mgu = pa + (size_t)ul * kWarps * heads_max * MG + h * MG;
        float M = kNegBig;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, mgu[w * heads_max * MG + DV]);
        float o = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float mw = mgu[w * heads_max * MG + DV];
            if (mw > kNegBig) {                            // a warp that saw no token of the unit left no values
                const float fw = ex2_approx(mw - M);
                o += fw * mgu[w * heads_max * MG + dv];
                l += fw * mgu[w * heads_max * MG + DV + 1];
            }
        }
        if (is_whole(unit)) {
            out[((size_t)ru->b[ul] * f.H_q + kvh * f.g + ru->hgrp[ul] * 4 + h) * DV + dv] = l > 0.f ? o / l : 0.f;
        } else {
            const size_t pslot = (size_t)(c + unit) * 4 + h;
            part_o[pslot * DV + dv] = o;
            if (dv == 0) {
                part_ml[pslot * 2] = M;
                part_ml[pslot * 2 + 1] = l;
            }
        }
    }
    if (!any_split) return;                                // block-uniform
    __threadfence();                                       // this thread's partial writes are visible
    __syncthreads();
    if (tid < nr) {
        const int unit = u0 + tid;
        int last = 0;
        if (!is_whole(unit)) {
            int c_lo, c_hi;
            unit_ctas(unit, &c_lo, &c_hi);
            const unsigned arrived = atomicAdd(tickets + unit, 1u);
            last = arrived == (unsigned)(c_hi - c_lo);
            if (last) tickets[unit] = 0u;                  // ready for the next launch
        }
        s_last[tid] = last;
    }
    __syncthreads();
    for (int ul = 0; ul < nr; ++ul) {
        if (!s_last[ul]) continue;
        __threadfence();
        const int unit = u0 + ul;
        const int heads_here = min(4, f.g - ru->hgrp[ul] * 4);
        int c_lo, c_hi;
        unit_ctas(unit, &c_lo, &c_hi);
        for (int idx = tid; idx < heads_here * DV; idx += kThreads) {
            const int h = idx / DV, dv = idx - h * DV;
            float M = kNegBig;
            for (int cp2 = c_lo; cp2 <= c_hi; ++cp2)
                M = fmaxf(M, __ldcg(part_ml + ((size_t)(cp2 + unit) * 4 + h) * 2));
            float o = 0.f, l = 0.f;
            for (int cp2 = c_lo; cp2 <= c_hi; ++cp2) {
                const size_t pp = (size_t)(cp2 + unit) * 4 + h;
                const float fw = ex2_approx(__ldcg(part_ml + pp * 2) - M);
                l += fw * __ldcg(part_ml + pp * 2 + 1);
                o += fw * __ldcg(part_o + pp * DV + dv);
            }
            out[((size_t)ru->b[ul] * f.H_q + kvh * f.g + ru->hgrp[ul] * 4 + h) * DV + dv] = l > 0.f ? o / l : 0.f;
        }
    }
}

template <int M_SUB, int DV, int STAGES>
__global__ void __launch_bounds__(kThreads, 1) attend_multi_kernel(const __grid_constant__ AttendArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int ROW = DV * 2 + 16;                      // a V row plus 16 bytes of padding
    constexpr int SLOT = kTile * ROW + kTile * M_SUB;     // V rows, then the tile's codes
    constexpr int V_CHUNKS = kTile * DV * 2 / 512;        // 16-byte pieces per lane and tile
    constexpr int MG = DV + 2;
    constexpr int head_stride = M_SUB * kTableStride + kHeadPad;
    __shared__ int s_last[kMaxRoundUnits];

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int n = lane >> 2, q = lane & 3;
    const int hl = n & 3;                                 // head (within the group) this lane scores
    const int part = n >> 2;                              // 0: weight, 1: its fp16 remainder
    const int hgroups = (a.g + 3) >> 2;
    const int heads_max = a.g < 4 ? a.g : 4;
    const int units_per_head = hgroups * a.B;

    unsigned char *ring = smem_raw + a.lay.ring + (size_t)warp * STAGES * SLOT;
    const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ring);

    constexpr int ROWS_PER_IT = 512 / (DV * 2);
    const int copy_row = (lane * 16) / (DV * 2);
    const unsigned copy_dst = (unsigned)(copy_row * ROW + (lane * 16) % (DV * 2));
    const unsigned frag_src = (unsigned)(((lane & 7) + ((lane >> 4) & 1) * 8) * ROW + ((lane >> 3) & 1) * 16);

    // ---- this CTA's range of the flat tile sequence (the host keeps the tile count below 2^31 for this kernel) ----
    int T_lo, T_hi;
    {
        const int c = blockIdx.x, per_cta = (int)a.tiles_per_cta;
        if (a.splits_per_unit > 0) {
            const int u = c / a.splits_per_unit, s = c - u * a.splits_per_unit;
            T_lo = u * a.tiles_per_unit + s * per_cta;
            T_hi = min((u + 1) * a.tiles_per_unit, T_lo + per_cta);
        } else if (a.ctas_per_head > 0) {                  // a KV head's tiles are cut among its own CTAs
            const int kvh = c / a.ctas_per_head, s = c - kvh * a.ctas_per_head;
            const int head_lo = kvh * units_per_head * a.tiles_per_unit;
            T_lo = head_lo + s * per_cta;
            T_hi = min(head_lo + units_per_head * a.tiles_per_unit, T_lo + per_cta);
        } else {
            T_lo = c * per_cta;
            T_hi = min(a.n_units * a.tiles_per_unit, T_lo + per_cta);
        }
    }
    if (T_hi <= T_lo) return;
    const int t_end = T_hi - T_lo;                        // tiles in this CTA's range
    const int unit_first = T_lo / a.tiles_per_unit;
    const int unit_last = (T_hi - 1) / a.tiles_per_unit;

    // ---- the codebooks of a KV head into shared memory (one copy group; rows keep their place, pieces permuted) ----
    auto stage_book = [&](int kvh) {
        // n_c (1, 2, 4, 8 or 16) divides the thread count: a thread keeps its piece index, its rows step by 512 / n_c
        const int d_sub = a.d_k / M_SUB, n_c = d_sub >> 2, sh = staged_shift(n_c), lg = 31 - __clz(n_c);
        const unsigned char *src = reinterpret_cast<const unsigned char *>(a.codebooks + (size_t)kvh * M_SUB * a.K * d_sub) + tid * 16;
        const unsigned dst0 = (unsigned)__cvta_generic_to_shared(smem_raw + a.lay.book);
        const int c4 = tid & (n_c - 1), rows = M_SUB * a.K;
        for (int e = tid >> lg; e < rows; e += kThreads >> lg) {
            cp_async16(dst0 + (unsigned)(e * d_sub + staged_piece(e, c4, n_c, sh) * 4) * 4u, src);
            src += kThreads * 16;
        }
        cp_async_commit();
    };
    int staged_head = -1;
    int book_pending = 0;                                 // 1: copied before the ring's first tiles, 2: after ring copies
    if (a.stage_book) {
        staged_head = unit_first / units_per_head;
        stage_book(staged_head);
        book_pending = 1;
    }

    // ---- producer: the cursor's tile into ring slot `slot` (always closes one copy group) ----
    auto issue = [&](const MCursor &pc, int slot) {
        const int nv = pc.t < t_end ? mc_valid(pc) : 0;
        if (nv > 0) {
            const unsigned char *vsrc = reinterpret_cast<const unsigned char *>(a.v) + pc.row0 * (DV * 2);
            const unsigned char *csrc = a.codes + pc.row0 * M_SUB;
            unsigned char *dst = ring + slot * SLOT;
            const unsigned dst_s = ring_s + slot * SLOT;
            if (nv == kTile) {
#pragma unroll
                for (int it = 0; it < V_CHUNKS; ++it)
                    cp_async16(dst_s + copy_dst + it * (ROWS_PER_IT * ROW), vsrc + lane * 16 + it * 512);
                if (lane < M_SUB) cp_async16(dst_s + kTile * ROW + lane * 16, csrc + lane * 16);
            } else {
                // ragged end of a row: rows at or beyond seq_len are never read, zeros stand in
#pragma unroll
                for (int it = 0; it < V_CHUNKS; ++it) {
                    const unsigned d = copy_dst + it * (ROWS_PER_IT * ROW);
                    if (copy_row + it * ROWS_PER_IT < nv) cp_async16(dst_s + d, vsrc + lane * 16 + it * 512);
                    else *reinterpret_cast<uint4 *>(dst + d) = make_uint4(0, 0, 0, 0);
                }
                if (lane < kTile) {
#pragma unroll
                    for (int j = 0; j < M_SUB; ++j)
                        dst[kTile * ROW + lane * M_SUB + j] = lane < nv ? csrc[lane * M_SUB + j] : 0;
                }
            }
        }
        cp_async_commit();
    };

    // ---- prologue: fill the ring with this warp's first STAGES tiles ----
    MCursor cc;
    cc.t = warp;
    cc.unit = (T_lo + warp) / a.tiles_per_unit;
    cc.lt = T_lo + warp - cc.unit * a.tiles_per_unit;
    cc.row0 = 0;
    mc_enter_unit<M_SUB, DV>(a, cc, hgroups);
    MCursor pc = cc;
#pragma unroll
    for (int s = 0; s < STAGES; ++s) {
        issue(pc, s);
        mc_advance<M_SUB, DV>(a, pc, hgroups);
    }
    int slot = 0;
    const int ts_off = 2 * q + 8 * part;                  // the two tokens of a tile this lane scores

    // ---- rounds: up to a.ut consecutive units of one KV head ----
    __shared__ RoundUnits s_units[2];                      // by round parity: written before the barrier that opens a round
    int u0 = unit_first, par = 0;
    while (u0 <= unit_last) {
        const int kvh = u0 / units_per_head;
        int u1 = min(unit_last, u0 + a.ut - 1);
        u1 = min(u1, (kvh + 1) * units_per_head - 1);
        const int nr = u1 - u0 + 1;
        par ^= 1;
        const RoundUnits *ru = &s_units[par];
        if (tid < nr) {
            const UnitId id = unit_id(a, u0 + tid, hgroups);
            s_units[par].b[tid] = id.b;
            s_units[par].hgrp[tid] = id.hgrp;
        }
        __syncthreads();                                   // the previous round's merge is over
        if (a.stage_book && staged_head != kvh) {          // the range crossed into the next head (block-uniform)
            staged_head = kvh;
            stage_book(kvh);
            book_pending = 2;
        }
        round_fill(a, smem_raw, ru, kvh, nr);
        // the codebook copies are older than the STAGES ring copies in flight, unless they were issued just above
        if (book_pending == 1) cp_async_wait<STAGES>();
        else if (book_pending == 2) cp_async_wait<0>();
        book_pending = 0;
        __syncthreads();
        round_tables(a, smem_raw, ru, kvh, u0, nr, T_lo, T_hi);
        __syncthreads();

        // ---- the round's tiles, unit by unit for this warp; no block-wide barrier in here ----
        const int round_end = min(T_hi, (u1 + 1) * a.tiles_per_unit) - T_lo;
        while (cc.t < round_end) {
            // this warp's tiles of unit cc.unit (it may have none in a unit shorter than 16 tiles)
            const int ul = cc.unit - u0;
            const int seg_end = min(round_end, (cc.unit + 1) * a.tiles_per_unit - T_lo);
            const int hgrp = ru->hgrp[ul];
            const int heads_here = min(4, a.g - hgrp * 4);
            const bool head_ok = hl < heads_here;
            const bool full_unit = heads_here == 4 && !a.scores_out;
            const float *my_table = MS_TABLES(a, smem_raw) + (size_t)ul * a.lay.set_floats + (hl < heads_max ? hl : 0) * head_stride;
            float *scores_row = (a.scores_out && head_ok)
                                    ? a.scores_out + ((size_t)ru->b[ul] * a.H_q + kvh * a.g + hgrp * 4 + hl) * a.L_max
                                    : nullptr;
            const int new_lt = a.new_keys ? (a.new_pos >> 4) : -1;     // tile whose newest token's codes come from shared memory

            float acc[DV / 16][4];
#pragma unroll
            for (int i = 0; i < DV / 16; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
            float m_run = kNegBig, l_run = 0.f;
            bool any = false;

            while (cc.t < seg_end) {
                cp_async_wait<STAGES - 1>();               // this lane's copies of the tile have landed
                __syncwarp();                              // ... and every other lane's
                const int nv = mc_valid(cc);
                const unsigned char *sl = ring + slot * SLOT;
                uint32_t vf[DV / 16][4];
                CodePair<M_SUB> cp;
                if (nv > 0) {                              // tile -> registers, so the slot can be refilled
                    cp = read_code_pair<M_SUB>(sl + kTile * ROW + ts_off * M_SUB);
#pragma unroll
                    for (int i = 0; i < DV / 16; ++i)
                        ldmatrix_x4_trans(vf[i], ring_s + slot * SLOT + frag_src + i * 32);
                }
                __syncwarp();                              // all lanes have read the slot
                issue(pc, slot);
                mc_advance<M_SUB, DV>(a, pc, hgroups);
                if (nv > 0) {
                    any = true;
                    const bool fast = full_unit && nv == kTile && cc.lt != new_lt;
                    if (!fast && cc.lt == new_lt && ((a.new_pos & 15) >> 1) == (ts_off >> 1)) {
                        // the appended key's codes come from shared memory: the copy of the tile may predate the store
                        const unsigned char *nc = MS_NEWC(a, smem_raw) + ul * 16;
                        const int odd = a.new_pos & 1;             // which of the lane's two tokens
#pragma unroll
                        for (int byte = 0; byte < 2 * M_SUB; ++byte) {   // (static word indices: the pair stays in registers)
                            const unsigned sh = (unsigned)(byte & 3) * 8u;
                            if (byte / M_SUB == odd)
                                cp.w[byte >> 2] = (cp.w[byte >> 2] & ~(0xffu << sh)) | ((uint32_t)nc[byte % M_SUB] << sh);
                        }
                    }
                    // ---- lookup-and-sum for this lane's two (token, head) pairs ----
                    float s0 = 0.f, s1 = 0.f;
                    if (fast || head_ok) {
#pragma unroll
                        for (int j = 0; j < M_SUB; ++j) {
                            s0 += my_table[j * kTableStride + LOOKAT_CHECKED_CODE(code_at<M_SUB>(cp, 0, j), a.K, a.status)];
                            s1 += my_table[j * kTableStride + LOOKAT_CHECKED_CODE(code_at<M_SUB>(cp, 1, j), a.K, a.status)];
                        }
                    }
                    float x0 = s0 * a.scale_log2, x1 = s1 * a.scale_log2;
                    if (!fast) {
                        const bool ok0 = head_ok && ts_off < nv, ok1 = head_ok && ts_off + 1 < nv;
                        if (scores_row) {
                            const int t0 = cc.lt * kTile;
                            if (ok0) scores_row[t0 + ts_off] = s0;
                            if (ok1) scores_row[t0 + ts_off + 1] = s1;
                        }
                        x0 = ok0 ? x0 : -INFINITY;
                        x1 = ok1 ? x1 : -INFINITY;
                    }
                    // ---- running maximum per head (8 lanes share a head) ----
                    float mt = fmaxf(x0, x1);
                    mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 1));
                    mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 2));
                    mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 16));
                    const float m_new = fmaxf(m_run, mt);
                    const float alpha = ex2_approx(m_run - m_new);
                    const float p0 = ex2_approx(x0 - m_new);
                    const float p1 = ex2_approx(x1 - m_new);
                    l_run = l_run * alpha + (p0 + p1);
                    m_run = m_new;
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
                        // accumulator columns 2q, 2q+1 belong to heads 2(q&1), 2(q&1)+1
                        const float al0 = __shfl_sync(0xffffffffu, alpha, (2 * (q & 1)) << 2);
                        const float al1 = __shfl_sync(0xffffffffu, alpha, (2 * (q & 1) + 1) << 2);
#pragma unroll
                        for (int i = 0; i < DV / 16; ++i) {
                            acc[i][0] *= al0; acc[i][1] *= al1; acc[i][2] *= al0; acc[i][3] *= al1;
                        }
                    }
                    // ---- weights into the MMA's B layout: rows 2q,2q+1 and 2q+8,2q+9 of column n ----
                    const float o0 = __shfl_xor_sync(0xffffffffu, p0, 16);
                    const float o1 = __shfl_xor_sync(0xffffffffu, p1, 16);
                    const float w0 = part ? o0 : p0, w1 = part ? o1 : p1;   // tokens 2q, 2q+1
                    const float w2 = part ? p0 : o0, w3 = part ? p1 : o1;   // tokens 2q+8, 2q+9
                    const uint32_t b0 = weight_pair(w0, w1, part);
                    const uint32_t b1 = weight_pair(w2, w3, part);
                    // ---- O^T += V^T P on the tensor cores ----
#pragma unroll
                    for (int i = 0; i < DV / 16; ++i) mma_16816(acc[i], vf[i][0], vf[i][1], vf[i][2], vf[i][3], b0, b1);
                }
                slot = slot + 1 == STAGES ? 0 : slot + 1;
                mc_advance<M_SUB, DV>(a, cc, hgroups);
            }

            // ---- this warp's partial of the unit to shared memory (weight and remainder columns folded) ----
            if (any) {
#pragma unroll
                for (int i = 0; i < DV / 16; ++i)
#pragma unroll
                    for (int k = 0; k < 4; ++k) acc[i][k] += __shfl_xor_sync(0xffffffffu, acc[i][k], 2);
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
                l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);
                float *mgw = MS_PARTIALS(a, smem_raw) + (size_t)(ul * kWarps + warp) * heads_max * MG;
                if (q < 2) {
                    const bool h0 = 2 * q < heads_max, h1 = 2 * q + 1 < heads_max;
#pragma unroll
                    for (int i = 0; i < DV / 16; ++i) {
                        float *o = mgw + (2 * q) * MG + 16 * i + n;
                        if (h0) { o[0] = acc[i][0]; o[8] = acc[i][2]; }            // (dv, head 2q), (dv + 8, head 2q)
                        if (h1) { o[MG] = acc[i][1]; o[MG + 8] = acc[i][3]; }      // head 2q + 1
                    }
                }
                if (q == 0 && part == 0 && hl < heads_max) {
                    mgw[hl * MG + DV] = m_run;
                    mgw[hl * MG + DV + 1] = l_run;
                }
            }
        }
        __syncthreads();
        round_merge(a, smem_raw, ru, kvh, u0, nr, T_lo, T_hi, s_last);
        u0 = u1 + 1;
    }
    cp_async_wait<0>();
}

template <int M_SUB, int DV, int STAGES>
lookat_status multi_kernel_ready(Ctx *ctx, const AttendArgs &a, size_t smem)
{
    auto kern = attend_multi_kernel<M_SUB, DV, STAGES>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "attend: shared-memory opt-in");
    return LOOKAT_OK;
}

template <int M_SUB, int DV, int STAGES>
lookat_status multi_launch(Ctx *ctx, const AttendArgs &a, size_t smem)
{
    attend_multi_kernel<M_SUB, DV, STAGES><<<a.n_ctas, kThreads, smem, ctx->stream>>>(a);
    return check_launch(ctx, "attend_multi_kernel");
}

template <typename F>
lookat_status dispatch_multi(int m, int d_v, int stages, F &&f)
{
#define LOOKAT_CASE(M, D, S) \
    if (m == M && d_v == D && stages == S) return f.template operator()<M, D, S>();
#define LOOKAT_CASES(M) \
    LOOKAT_CASE(M, 64, 4) LOOKAT_CASE(M, 64, 3) LOOKAT_CASE(M, 64, 2) LOOKAT_CASE(M, 128, 3) LOOKAT_CASE(M, 128, 2)
    LOOKAT_CASES(1) LOOKAT_CASES(2) LOOKAT_CASES(4) LOOKAT_CASES(8) LOOKAT_CASES(16)
#undef LOOKAT_CASES
#undef LOOKAT_CASE
    return LOOKAT_ERR_UNSUPPORTED;
}

}  // namespace

// Whether the kernel's smallest configuration (one unit per round, nothing staged, two ring slots) fits.
bool multi_fits(const Ctx *ctx, const AttendArgs &a)
{
    return (size_t)multi_layout(a.m, a.d_v, a.d_k, a.K, a.g, 1, 0, 2).total <= (size_t)ctx->max_smem_optin;
}

// Chooses the units per round, whether the codebooks are staged, and the ring depth so that the kernel's shared
// memory fits; fills a.ut, a.stage_book, a.stages.  `ut_wanted` = the most units a CTA's range can touch.
lookat_status plan_multi(Ctx *ctx, AttendArgs &a, int ut_wanted)
{
    const int d_sub = a.d_k / a.m;
    const int n_c = d_sub / 4;
    const size_t book_bytes = (size_t)a.K * a.d_k * 4;
    const bool can_stage = !a.lut && a.codebooks && d_sub % 4 == 0 && (n_c & (n_c - 1)) == 0 && n_c <= 16 &&
                           book_bytes <= 64 * 1024;
    if (ut_wanted > kMaxRoundUnits) ut_wanted = kMaxRoundUnits;
    if (ut_wanted < 1) ut_wanted = 1;
    const int stage_opts[2] = {can_stage ? 1 : 0, 0};
    for (int so = 0; so < (can_stage ? 2 : 1); ++so) {
        for (int ut = ut_wanted; ut >= 1; ut = ut > 2 ? (ut + 1) / 2 : ut - 1) {
            for (int stages = (a.d_v == 64 ? 4 : 3); stages >= 2; --stages) {
                if (stage_opts[so] && stages == 4) continue;
                const MultiLayout lay = multi_layout(a.m, a.d_v, a.d_k, a.K, a.g, ut, stage_opts[so], stages);
                if ((size_t)lay.total > (size_t)ctx->max_smem_optin) continue;
                a.ut = ut;
                a.stage_book = stage_opts[so];
                a.stages = stages;
                a.lay = lay;
                return dispatch_multi(a.m, a.d_v, stages, [&]<int M, int D, int S>() {
                    return multi_kernel_ready<M, D, S>(ctx, a, (size_t)lay.total);
                });
            }
        }
    }
    return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend: the streaming kernel's tables do not fit in shared memory");
}

lookat_status launch_multi(Ctx *ctx, const AttendArgs &a)
{
    return dispatch_multi(a.m, a.d_v, a.stages, [&]<int M, int D, int S>() {
        return multi_launch<M, D, S>(ctx, a, (size_t)a.lay.total);
    });
}

}  // namespace lookat
