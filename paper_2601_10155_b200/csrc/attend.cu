// Fused ADC scoring + online softmax + value accumulation (Section 3.5 "Lookup
// and Sum"; Algorithm 1, second loop and continuation), split over the
// sequence, plus the merge of the partial results.
//
// Streaming kernel (attend_stream_kernel).  Work is the flat sequence of
// (unit, 16-token tile) pairs, unit = (batch row, KV head, group of <= 4 query
// heads sharing that KV head); each persistent CTA owns one contiguous range of
// it, so all CTAs stream the same number of bytes and the tables are reloaded
// only where a range crosses into the next unit.  Inside a CTA the 16 warps take
// tiles round-robin and never wait for each other in the token loop:
//   * V rows and codes travel global -> shared memory into a private ring of
//     STAGES tiles per warp: by the bulk-copy engine -- one lane issues, per
//     tile, a tiled copy (cp.async.bulk.tensor.2d, boxes of 16 rows x 128 bytes
//     with the 128-byte swizzle, which the fragment reads undo with one XOR) per
//     64 value columns and a plain bulk copy of the codes, completion counted
//     in bytes on an mbarrier per slot with a bounded wait -- or, where the
//     driver offers no tensor maps, as 16-byte cp.async pieces into rows padded
//     by 16 bytes; a warp moves a landed tile into registers and refills its
//     slot at once, so close to STAGES tiles of about 4 KB stay in flight per
//     warp (the bulk form: 371 -> about 330 warp instructions per tile, 11 %
//     less time under the power cap),
//   * the unit's tables sit in shared memory, one set per head, sets shifted by
//     8 banks; a lane scores two (token, head) pairs per tile, m gathers each,
//   * the weighted value sum  O^T[d_v x heads] += V^T[d_v x 16 tokens] . P[16 x heads]
//     runs on the tensor cores (mma.sync m16n8k16, fp16 in, fp32 accumulate).
//     The 8 columns hold the <= 4 heads twice: the fp16 rounding of each weight
//     and the fp16 rounding of its remainder, so weights carry ~22 bits.  The
//     V^T operand comes from the row-major V rows by ldmatrix with transpose.
// With q and codebooks instead of ready tables, a CTA builds the tables of a
// unit itself when it enters the unit (fp64 accumulation as in lut.cu).
// At the end of a unit the warps of a CTA merge through shared memory into one
// partial (max, sum, weighted values) per (CTA, unit); the CTA that arrives last
// at a unit (a counter per unit, no waiting) merges the unit's partials and
// writes the output rows.
//
// Generic kernel (attend_generic_kernel): any shape, plain loads, tables read
// from global memory; used where the streaming kernel's layout assumptions
// (d_v in {64,128}, m in {1,2,4,8,16}, 16-byte aligned rows) do not hold.
#include <cuda.h>           // CUtensorMap only

#include <cstdlib>
#include <cstring>
#include <type_traits>

#include "common.cuh"
#include "attend_tile.cuh"
#include "encode_warp.cuh"

namespace lookat {

namespace {

// Position in the flat tile sequence: tile `lt` of unit `unit`, with that unit's row facts and the tile's first row of
// the caches.  Kept small (the streaming loop holds two of them in registers): the position is counted from the start of
// the CTA's range, addresses are formed from the row where a copy is issued.
template <class Row>     // int where the caches have fewer than 2^31 rows (the plan sends only those to the bulk copies)
struct TileCursor {
    int t;               // flat index minus the first tile of the CTA's range
    int unit, lt;
    int len;             // tokens in the unit's batch row (0 beyond the last unit)
    Row row0;            // (batch row * H_kv + KV head) * L_max + 16 lt
};

template <class Row>
__device__ __forceinline__ void cursor_enter_unit(const AttendArgs &a, TileCursor<Row> &c, int hgroups)
{
    if (c.unit < a.n_units) {
        const int kv_row = c.unit / hgroups;             // (batch row, KV head) of the unit
        const int b = kv_row / a.H_kv;
        c.len = (int)min((long long)(a.seq_lens ? a.seq_lens[b] : a.uniform_len), a.L_max);
        c.row0 = (Row)((long long)kv_row * a.L_max + (long long)c.lt * kTile);
    } else {
        c.len = 0;
    }
}

template <class Row>
__device__ __forceinline__ TileCursor<Row> cursor_at(const AttendArgs &a, long long T_lo, int t, int hgroups)
{
    TileCursor<Row> c;
    const long long T = T_lo + t;
    c.t = t;
    c.unit = (int)(T / a.tiles_per_unit);
    c.lt = (int)(T - (long long)c.unit * a.tiles_per_unit);
    c.row0 = 0;
    cursor_enter_unit(a, c, hgroups);
    return c;
}

template <class Row>
__device__ __forceinline__ void cursor_advance(const AttendArgs &a, TileCursor<Row> &c, int hgroups)
{
    c.t += kWarps;
    c.lt += kWarps;
    c.row0 += kWarps * kTile;
    if (c.lt >= a.tiles_per_unit) {
        do {
            c.lt -= a.tiles_per_unit;
            c.unit += 1;
        } while (c.lt >= a.tiles_per_unit);
        cursor_enter_unit(a, c, hgroups);
    }
}

// The cursor `ahead` tiles further on.  The copies run a fixed distance ahead of the tile a warp works on, so their
// position is derived from that tile's instead of being carried along; only next to a unit's end is it looked up anew.
template <class Row>
__device__ __forceinline__ TileCursor<Row> cursor_ahead(const AttendArgs &a, const TileCursor<Row> &c, long long T_lo, int ahead,
                                                        int hgroups)
{
    if (c.lt + ahead < a.tiles_per_unit && c.unit < a.n_units) {
        TileCursor<Row> p = c;
        p.t += ahead;
        p.lt += ahead;
        p.row0 += (Row)(ahead * kTile);
        return p;
    }
    return cursor_at<Row>(a, T_lo, c.t + ahead, hgroups);
}

// Tokens of the cursor's tile that exist (0..16).
template <class Row>
__device__ __forceinline__ int cursor_valid(const TileCursor<Row> &c)
{
    const int left = c.len - c.lt * kTile;
    return left >= kTile ? kTile : (left > 0 ? left : 0);
}

// Append fused into attention (Section 3.4 "Encoding" for one new key): the warp encodes the key of
// one (batch row, KV head), stores its m codes at token new_pos and fences the stores; the caller
// synchronises the CTA before any warp copies that tile.  Kept out of line: it runs once per unit.
__device__ __noinline__ void append_encode_warp(const __half *x_sub, const float *book, uint8_t *code_out, int K,
                                                int d_sub, int lane)
{
    const int code = nearest_centroid_warp(x_sub, book, K, d_sub, lane, nullptr);
    if (lane == 0) *code_out = (uint8_t)code;
    __threadfence();
    asm volatile("fence.proxy.async;" ::: "memory");       // the tile may be fetched by the bulk-copy engine
    __syncwarp();
}


template <int M_SUB, int DV, int STAGES, bool BULK>
__global__ void __launch_bounds__(kThreads, 1) attend_stream_kernel(AttendArgs a, const __grid_constant__ CUtensorMap v_map)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int ROW = DV * 2 + 16;                      // a V row plus 16 bytes of padding
    constexpr int SLOT = kTile * ROW + kTile * M_SUB;     // V rows, then the tile's codes
    constexpr int V_CHUNKS = kTile * DV * 2 / 512;        // 16-byte pieces per lane and tile

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int n = lane >> 2, q = lane & 3;
    const int hl = n & 3;                                 // head (within the group) this lane scores
    const int part = n >> 2;                              // 0: weight, 1: its fp16 remainder
    const int hgroups = (a.g + 3) >> 2;
    const int heads_max = a.g < 4 ? a.g : 4;
    const int table = M_SUB * a.K;                        // floats per head in global memory
    // in shared memory every subspace gets kTableStride entries whatever K is: offsets are constants
    constexpr int head_stride = M_SUB * kTableStride + kHeadPad;
    const int lut_bytes = (heads_max * head_stride * 4 + 15) & ~15;

    // shared memory: [tables | merge buffer (same bytes, used in turn)] [queries, fp64] [rings]
    const int merge_bytes = kWarps * 4 * (DV + 2) * 4;
    const int region0 = lut_bytes > merge_bytes ? lut_bytes : merge_bytes;
    const int q_bytes = a.fused_lut ? 4 * a.d_k * 8 : 0;             // four heads' dims, widened (unused heads zero)
    float *lut_s = reinterpret_cast<float *>(smem_raw);
    double *q_s = reinterpret_cast<double *>(smem_raw + region0);
    unsigned char *ring = smem_raw + region0 + q_bytes + (size_t)warp * STAGES * SLOT;
    const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ring);
    // BULK: the V rows of a tile arrive as DV/64 tiled bulk copies (TMA boxes of 16 rows x 128 bytes, 128-byte swizzle instead
    // of row padding: the fragment reads below XOR the 16-byte piece index with the row) and the codes as one bulk copy,
    // completion counted in bytes on an mbarrier per (warp, ring slot); else 16-byte cp.async pieces counted in copy groups.
    // BULK layout after the queries: [V ring, 1024-byte aligned: warp x slot x DV/64 boxes of 2 KB][codes ring][barriers]
    constexpr int VT = (DV / 64) * 2048;                   // V bytes of a tile
    const unsigned ring0_s = (unsigned)__cvta_generic_to_shared(smem_raw + region0 + q_bytes);
    const unsigned vring_s = ((ring0_s + 1023u) & ~1023u) + (unsigned)(warp * STAGES * VT);
    const unsigned cring_off = (unsigned)(kWarps * STAGES * VT + warp * STAGES * kTile * M_SUB) - (unsigned)(warp * STAGES * VT);
    const unsigned bar_s = ((ring0_s + 1023u) & ~1023u) + (unsigned)(kWarps * STAGES * (VT + kTile * M_SUB) + warp * STAGES * 8);
    if (BULK) {
        if (lane == 0) {
#pragma unroll
            for (int st = 0; st < STAGES; ++st) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_s + 8 * st));
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
    }

    // the streamed bytes are used once: marked to leave L2 first, so that what the CTAs read again and again (codebooks,
    // queries, partials) stays
    // (the value createpolicy.fractional.L2::evict_first yields for the whole line, as CUTLASS's cache-hint constants
    // have it; as a constant it occupies no registers between copies)
    constexpr unsigned long long stream_policy = 0x12F0000000000000ull;

    const float *my_table = lut_s + hl * head_stride;

    // a lane copies the 16-byte piece (lane*16 + it*512) of a tile's V bytes, it = 0..V_CHUNKS-1
    constexpr int ROWS_PER_IT = 512 / (DV * 2);
    const int copy_row = (lane * 16) / (DV * 2);
    const unsigned copy_dst = (unsigned)(copy_row * ROW + (lane * 16) % (DV * 2));
    // ... and reads, per MMA, one row of four 8x8 blocks: tokens (lane&7) + 8*bit4, dv 8*bit3
    const unsigned frag_src = (unsigned)(((lane & 7) + ((lane >> 4) & 1) * 8) * ROW + ((lane >> 3) & 1) * 16);
    // the same row of the swizzled layout: r * 128 + ((2 k + hi) ^ (r & 7)) * 16 = (r * 128 + ((hi ^ r & 1) * 16 + (r >> 1 & 3) * 32)) ^ (k * 32)
    const unsigned swz_base = (unsigned)(((lane & 7) + ((lane >> 4) & 1) * 8) * 128 + ((((lane >> 3) & 1) ^ (lane & 1)) << 4) +
                                         (((lane >> 1) & 3) << 5));

    // ---- this CTA's range of the flat tile sequence ----
    long long T_lo, T_hi;
    const long long c = blockIdx.x;
    if (a.splits_per_unit > 0) {
        const long long u = c / a.splits_per_unit, s = c - u * a.splits_per_unit;
        T_lo = u * a.tiles_per_unit + s * a.tiles_per_cta;
        T_hi = min((u + 1) * a.tiles_per_unit, T_lo + a.tiles_per_cta);
    } else {
        T_lo = c * a.tiles_per_cta;
        T_hi = min((long long)a.n_units * a.tiles_per_unit, T_lo + a.tiles_per_cta);
    }

    const int t_hi = (int)(T_hi - T_lo);                  // a CTA's range is far below 2^31 tiles

    // ---- producer: the cursor's tile into ring slot `slot` (always closes one copy group) ----
    using Cursor = TileCursor<std::conditional_t<BULK, int, long long>>;
    auto issue = [&](const Cursor &pc, int slot) {
        const int nv = pc.t < t_hi ? cursor_valid(pc) : 0;
        const unsigned char *const pc_vptr = reinterpret_cast<const unsigned char *>(a.v) + (size_t)pc.row0 * (DV * 2);
        const unsigned char *const pc_cptr = a.codes + (size_t)pc.row0 * M_SUB;
        if (BULK) {
            const unsigned bar = bar_s + 8 * slot;
            const unsigned vdst_s = vring_s + slot * VT;
            if (nv == kTile) {
                if (lane == 0) {
                    // one arrival that also announces the tile's bytes, then the copies
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "n"(VT + kTile * M_SUB) : "memory");
                    const int row0 = (int)pc.row0;
#pragma unroll
                    for (int nb = 0; nb < DV / 64; ++nb)
                        asm volatile(
                            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(
                                vdst_s + nb * 2048),
                            "l"(reinterpret_cast<uint64_t>(&v_map)), "r"(nb * 64), "r"(row0), "r"(bar), "l"(stream_policy)
                            : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                                     vring_s + cring_off + slot * (kTile * M_SUB)),
                                 "l"(pc_cptr), "n"(kTile * M_SUB), "r"(bar), "l"(stream_policy)
                                 : "memory");
                }
            } else {
                if (nv > 0) {
                    // ragged end of a row: plain copies into the same layout; rows at or beyond seq_len are never read from
                    // memory, zeros stand in
                    unsigned char *const vring = smem_raw + region0 + q_bytes + (vring_s - ring0_s);
                    unsigned char *vdst = vring + slot * VT, *cdst = vring + cring_off + slot * (kTile * M_SUB);
#pragma unroll
                    for (int it = 0; it < V_CHUNKS; ++it) {
                        const int o = lane * 16 + it * 512, r = o / (DV * 2), ci = (o % (DV * 2)) >> 4;
                        uint4 val = make_uint4(0, 0, 0, 0);
                        if (r < nv) val = *reinterpret_cast<const uint4 *>(pc_vptr + o);
                        *reinterpret_cast<uint4 *>(vdst + (ci >> 3) * 2048 + r * 128 + (((ci & 7) ^ (r & 7)) << 4)) = val;
                    }
                    if (lane < kTile) {
#pragma unroll
                        for (int j = 0; j < M_SUB; ++j) cdst[lane * M_SUB + j] = lane < nv ? pc_cptr[lane * M_SUB + j] : 0;
                    }
                    __syncwarp();
                }
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");   // the phase completes at once
            }
            return;
        }
        if (nv > 0) {
            const unsigned char *vsrc = pc_vptr;
            const unsigned char *csrc = pc_cptr;
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

    // ---- running state of the unit being accumulated ----
    float acc[DV / 16][4];
    float m_run = kNegBig, l_run = 0.f;

    // token offset inside a tile of the two tokens this lane scores
    const int ts_off = 2 * q + 8 * part;

    // one tile, already in registers: vf = V^T operand fragments (MMA i covers dv 16i..16i+15),
    // cp = the codes of this lane's two tokens
    // `full` (a compile-time flag): all 16 tokens exist, all 4 heads of the group are in use and no
    // raw scores are wanted, so none of the per-lane conditions below is needed.
    auto process_tile = [&](auto full, int t0, int nv, const uint32_t (&vf)[DV / 16][4],
                            const CodePair<M_SUB> &cp, bool head_ok, float *scores_row) {
        constexpr bool FULL = decltype(full)::value;
        // ---- lookup-and-sum for this lane's two (token, head) pairs ----
        float s0 = 0.f, s1 = 0.f;
        if (FULL || head_ok) {
#pragma unroll
            for (int j = 0; j < M_SUB; ++j) {
                s0 += my_table[j * kTableStride + LOOKAT_CHECKED_CODE(code_at<M_SUB>(cp, 0, j), a.K, a.status)];
                s1 += my_table[j * kTableStride + LOOKAT_CHECKED_CODE(code_at<M_SUB>(cp, 1, j), a.K, a.status)];
            }
        }
        float x0 = s0 * a.scale_log2, x1 = s1 * a.scale_log2;
        if constexpr (!FULL) {
            const bool ok0 = head_ok && ts_off < nv, ok1 = head_ok && ts_off + 1 < nv;
            if (scores_row) {
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
    };

    // ---- append: the new key of every unit whose token new_pos lies in this CTA's range is encoded
    //      before any copy of that token's tile is issued, one warp per (unit, subspace).  Normally
    //      that tile is far down the range and the encoding runs while the first tiles are in flight
    //      (the barriers at the start of the first unit order it before every later copy); if the
    //      tile is among the first STAGES tiles of a warp, the encoding comes first. ----
    auto append_new_keys = [&]() {
        const int u_first = (int)(T_lo / a.tiles_per_unit);
        const int u_last = T_hi > T_lo ? (int)((T_hi - 1) / a.tiles_per_unit) : u_first - 1;
        for (int task = warp; task < (u_last - u_first + 1) * M_SUB; task += kWarps) {
            const int u = u_first + task / M_SUB, j = task % M_SUB;
            const long long T_new = (long long)u * a.tiles_per_unit + (a.new_pos >> 4);
            if (T_new >= T_lo && T_new < T_hi) {
                const int kv_row = u / hgroups, d_sub = a.d_k / M_SUB;
                append_encode_warp(a.new_keys + (size_t)kv_row * a.d_k + j * d_sub,
                                   a.codebooks + ((size_t)(kv_row % a.H_kv) * M_SUB + j) * a.K * d_sub,
                                   a.codes_w + ((size_t)kv_row * a.L_max + a.new_pos) * M_SUB + j, a.K, d_sub, lane);
            }
        }
    };
    bool append_first = false;
    if (a.new_keys) {
        // does a new token's tile fall into the part of the range the ring prologue covers?
        const long long head_hi = min(T_hi, T_lo + (long long)kWarps * STAGES);
        const long long lt_new = a.new_pos >> 4;
        const long long u0 = T_lo / a.tiles_per_unit;
        for (long long u = u0; u * a.tiles_per_unit < head_hi; ++u) {
            const long long T_new = u * a.tiles_per_unit + lt_new;
            append_first = append_first || (T_new >= T_lo && T_new < head_hi);
        }
        if (append_first) {
            append_new_keys();
            __syncthreads();
        }
    }

    // ---- prologue: fill the ring with this warp's first STAGES tiles ----
    Cursor cc = cursor_at<decltype(Cursor::row0)>(a, T_lo, warp, hgroups);   // tile this warp consumes next
#pragma unroll
    for (int s = 0; s < STAGES; ++s) issue(cursor_ahead(a, cc, T_lo, s * kWarps, hgroups), s);
    if (a.new_keys && !append_first) append_new_keys();
    int slot = 0;                                          // ring slot of the consumer's tile
    unsigned ring_parity = 0;                              // BULK: phase of the slots' barriers the consumer waits for

    // ---- one pass per unit this CTA's range touches ----
    __shared__ int s_last;
    float *mg = reinterpret_cast<float *>(smem_raw);      // merge buffer [kWarps][4][DV+2], aliases the tables
    constexpr int MG = DV + 2;
    const int unit_first = (int)(T_lo / a.tiles_per_unit);
    const int unit_last = T_hi > T_lo ? (int)((T_hi - 1) / a.tiles_per_unit) : unit_first - 1;
    for (int unit = unit_first; unit <= unit_last; ++unit) {
        const int hgrp = unit % hgroups;
        const int kv_row = unit / hgroups;
        const int b = kv_row / a.H_kv, kvh = kv_row - b * a.H_kv;
        const int heads_here = min(4, a.g - hgrp * 4);
        const int hq0 = kvh * a.g + hgrp * 4;
        const bool head_ok = hl < heads_here;

        __syncthreads();                                   // the previous unit's merge is over
        if (a.lut) {
            for (int h = 0; h < heads_here; ++h) {
                const float *src = a.lut + ((size_t)b * a.H_q + hq0 + h) * table;
                float *dst = lut_s + h * head_stride;
                if (a.K == kTableStride) {
                    for (int i = tid; i < (table >> 2); i += kThreads)
                        reinterpret_cast<float4 *>(dst)[i] = __ldg(reinterpret_cast<const float4 *>(src) + i);
                } else {
                    for (int i = tid; i < table; i += kThreads) {
                        const int j = i / a.K;
                        dst[j * kTableStride + (i - j * a.K)] = __ldg(src + i);
                    }
                }
            }
        } else {
            // Section 3.5 "Precomputation Lookup Tables" for the heads of this unit:
            // lut[h][j][c] = q_h^(j) . C_j[c], fp64 accumulation, one rounding.
            // the unit's queries, widened, head fastest: one 16-byte read serves two heads
            for (int i = tid; i < 4 * a.d_k; i += kThreads) {
                const int h = i & 3, dim = i >> 2;
                q_s[i] = h < heads_here ? (double)__half2float(a.q[((size_t)b * a.H_q + hq0 + h) * a.d_k + dim]) : 0.0;
            }
            __syncthreads();

            const int d_sub = a.d_k / M_SUB;
            const float *book = a.codebooks + (size_t)kvh * table * d_sub;
            build_unit_tables<false>(book, q_s, lut_s, table, a.K, d_sub, heads_here, head_stride, tid, nullptr, nullptr);
        }
        __syncthreads();

#pragma unroll
        for (int i = 0; i < DV / 16; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
        m_run = kNegBig;
        l_run = 0.f;

        const int seg_hi = (int)(min(T_hi, (long long)(unit + 1) * a.tiles_per_unit) - T_lo);
        const bool full_unit = heads_here == 4 && !a.scores_out;
        while (cc.t < seg_hi) {
            if (BULK) {
                // the tile's bytes have landed when the slot's barrier completes the phase (bounded: a copy that never
                // completes is reported through the status word and the tile is taken as it is)
                unsigned ok = 0;                           // each try may park the warp for up to ~2 us instead of spinning
                for (int it = 0; it < (1 << 17) && !ok; ++it)
                    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}"
                                 : "=r"(ok)
                                 : "r"(bar_s + 8 * slot), "r"(ring_parity), "r"(2000u)
                                 : "memory");
                if (!ok && a.status) atomicOr(a.status, kStatusCopyTimeout);
            } else {
                cp_async_wait<STAGES - 1>();               // this lane's copies of the tile have landed
            }
            __syncwarp();                                  // ... and every other lane's
            const int nv = cursor_valid(cc);
            const unsigned char *sl = ring + slot * SLOT;
            uint32_t vf[DV / 16][4];
            CodePair<M_SUB> cp;
            if (nv > 0) {                                  // tile -> registers, so the slot can be refilled
                if (BULK) {
                    cp = read_code_pair_s<M_SUB>(vring_s + cring_off + slot * (kTile * M_SUB) + ts_off * M_SUB);
                    // row r of box nb at nb * 2048 + r * 128, its 16-byte piece c at (c ^ (r & 7)) * 16; MMA i wants pieces
                    // 2 i and 2 i + 1 of the 256-byte row: box i / 4, piece 2 (i % 4) + hi
#pragma unroll
                    for (int i = 0; i < DV / 16; ++i)
                        ldmatrix_x4_trans(vf[i], vring_s + slot * VT + (i >> 2) * 2048 + (swz_base ^ (unsigned)((i & 3) << 5)));
                } else {
                    cp = read_code_pair<M_SUB>(sl + kTile * ROW + ts_off * M_SUB);
#pragma unroll
                    for (int i = 0; i < DV / 16; ++i)
                        ldmatrix_x4_trans(vf[i], ring_s + slot * SLOT + frag_src + i * 32);
                }
            }
            __syncwarp();                                  // all lanes have read the slot
            issue(cursor_ahead(a, cc, T_lo, STAGES * kWarps, hgroups), slot);   // the tile STAGES of this warp's tiles ahead
            if (nv == kTile && full_unit)
                process_tile(std::true_type{}, 0, kTile, vf, cp, true, nullptr);
            else if (nv > 0)
                process_tile(std::false_type{}, cc.lt * kTile, nv, vf, cp, head_ok,
                             (a.scores_out && head_ok) ? a.scores_out + ((size_t)b * a.H_q + hq0 + hl) * a.L_max : nullptr);
            slot = slot + 1 == STAGES ? 0 : slot + 1;
            if (slot == 0) ring_parity ^= 1u;
            cursor_advance(a, cc, hgroups);
        }

        // ---- this warp's result for the unit: fold the weight and remainder columns ----
#pragma unroll
        for (int i = 0; i < DV / 16; ++i)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[i][k] += __shfl_xor_sync(0xffffffffu, acc[i][k], 2);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);

        __syncthreads();                                   // every warp is done with the tables
        if (q < 2) {
#pragma unroll
            for (int i = 0; i < DV / 16; ++i) {
                float *o = mg + (warp * 4 + 2 * q) * MG + 16 * i + n;
                o[0] = acc[i][0];              // (dv, head 2q)
                o[MG] = acc[i][1];             // (dv, head 2q+1)
                o[8] = acc[i][2];              // (dv + 8, head 2q)
                o[MG + 8] = acc[i][3];         // (dv + 8, head 2q+1)
            }
        }
        if (q == 0 && part == 0) {
            mg[(warp * 4 + hl) * MG + DV] = m_run;
            mg[(warp * 4 + hl) * MG + DV + 1] = l_run;
        }
        __syncthreads();

        // ---- merge the warps: one partial per (CTA, unit) ----
        const size_t pslot = (size_t)(c + unit) * 4;       // + head
        for (int idx = tid; idx < heads_here * DV; idx += kThreads) {
            const int h = idx / DV, dv = idx - h * DV;
            float M = kNegBig;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) M = fmaxf(M, mg[(w * 4 + h) * MG + DV]);
            float o = 0.f, l = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float f = ex2_approx(mg[(w * 4 + h) * MG + DV] - M);
                o += f * mg[(w * 4 + h) * MG + dv];
                l += f * mg[(w * 4 + h) * MG + DV + 1];
            }
            a.part_o[(pslot + h) * DV + dv] = o;
            if (dv == 0) {
                a.part_ml[(pslot + h) * 2] = M;
                a.part_ml[(pslot + h) * 2 + 1] = l;
            }
        }

        // ---- the CTA that completes a unit merges the unit's partials into the output ----
        long long c_lo, c_hi;
        if (a.splits_per_unit > 0) {
            c_lo = (long long)unit * a.splits_per_unit;
            c_hi = c_lo + a.splits_per_unit - 1;
        } else {
            c_lo = (long long)unit * a.tiles_per_unit / a.tiles_per_cta;
            c_hi = ((long long)(unit + 1) * a.tiles_per_unit - 1) / a.tiles_per_cta;
        }
        __threadfence();                                   // this thread's partial writes are visible
        __syncthreads();
        if (tid == 0) {
            const unsigned arrived = atomicAdd(a.tickets + unit, 1u);
            s_last = arrived == (unsigned)(c_hi - c_lo);
            if (s_last) a.tickets[unit] = 0u;              // ready for the next launch
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            for (int idx = tid; idx < heads_here * DV; idx += kThreads) {
                const int h = idx / DV, dv = idx - h * DV;
                float M = kNegBig;
                for (long long cp2 = c_lo; cp2 <= c_hi; ++cp2)
                    M = fmaxf(M, __ldcg(a.part_ml + ((size_t)(cp2 + unit) * 4 + h) * 2));
                float o = 0.f, l = 0.f;
                for (long long cp2 = c_lo; cp2 <= c_hi; ++cp2) {
                    const size_t pp = (size_t)(cp2 + unit) * 4 + h;
                    const float f = ex2_approx(__ldcg(a.part_ml + pp * 2) - M);
                    l += f * __ldcg(a.part_ml + pp * 2 + 1);
                    o += f * __ldcg(a.part_o + pp * DV + dv);
                }
                a.out[((size_t)b * a.H_q + hq0 + h) * DV + dv] = l > 0.f ? o / l : 0.f;
            }
        }
    }
    cp_async_wait<0>();
}

// Any shape.  One CTA per (chunk, query head, batch row); 128 threads.
constexpr int kMultiMaxTiles = 512;     // tiles per unit up to which attend_multi_kernel is used
constexpr int kGenThreads = 128;
constexpr int kGenBlockTokens = 1024;

__global__ void __launch_bounds__(kGenThreads) attend_generic_kernel(AttendArgs a)
{
    __shared__ float xs[kGenBlockTokens];
    __shared__ float red[kGenThreads / 32];
    __shared__ float bcast;

    const int split = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x;
    const int kvh = hq / a.g;
    const int seq_len = (int)min((long long)(a.seq_lens ? a.seq_lens[b] : a.uniform_len), a.L_max);
    const long long chunk_lo = (long long)split * a.chunk;
    const long long chunk_hi = min((long long)seq_len, chunk_lo + a.chunk);

    const float *lut = a.lut + ((size_t)b * a.H_q + hq) * a.m * a.K;
    const size_t kv_row = (size_t)b * a.H_kv + kvh;
    const uint8_t *codes = a.codes + kv_row * a.L_max * a.m;
    const __half *v = a.v + kv_row * a.L_max * a.d_v;
    float *scores_row = a.scores_out ? a.scores_out + ((size_t)b * a.H_q + hq) * a.L_max : nullptr;

    const int n_dv = (a.d_v + kGenThreads - 1) / kGenThreads;   // value columns per thread (<= 8)
    float o[8];
    for (int i = 0; i < 8; ++i) o[i] = 0.f;
    float M = kNegBig, l = 0.f;

    for (long long blk = chunk_lo; blk < chunk_hi; blk += kGenBlockTokens) {
        const int cnt = (int)min((long long)kGenBlockTokens, chunk_hi - blk);
        float mloc = -INFINITY;
        for (int t = tid; t < cnt; t += kGenThreads) {
            const uint8_t *cd = codes + (blk + t) * a.m;
            float s = 0.f;
            for (int j = 0; j < a.m; ++j) s += __ldg(lut + j * a.K + LOOKAT_CHECKED_CODE((int)cd[j], a.K, a.status));
            if (scores_row) scores_row[blk + t] = s;
            const float x = s * a.scale_log2;
            xs[t] = x;
            mloc = fmaxf(mloc, x);
        }
        for (int d = 16; d; d >>= 1) mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, d));
        if ((tid & 31) == 0) red[tid >> 5] = mloc;
        __syncthreads();
        if (tid == 0) {
            float mm = red[0];
            for (int w = 1; w < kGenThreads / 32; ++w) mm = fmaxf(mm, red[w]);
            bcast = mm;
        }
        __syncthreads();
        const float M_new = fmaxf(M, bcast);
        const float alpha = ex2_approx(M - M_new);
        float lloc = 0.f;
        for (int t = tid; t < cnt; t += kGenThreads) {
            const float p = ex2_approx(xs[t] - M_new);
            xs[t] = p;
            lloc += p;
        }
        for (int d = 16; d; d >>= 1) lloc += __shfl_xor_sync(0xffffffffu, lloc, d);
        __syncthreads();                       // bcast consumed by all, xs holds the weights
        if ((tid & 31) == 0) red[tid >> 5] = lloc;
        __syncthreads();
        float lsum = 0.f;
        for (int w = 0; w < kGenThreads / 32; ++w) lsum += red[w];
        l = l * alpha + lsum;
        M = M_new;
        for (int i = 0; i < n_dv; ++i) {
            const int dv = tid + i * kGenThreads;
            if (dv < a.d_v) {
                float accv = 0.f;
                for (int t = 0; t < cnt; ++t) accv += xs[t] * __half2float(v[(blk + t) * a.d_v + dv]);
                o[i] = o[i] * alpha + accv;
            }
        }
        __syncthreads();                       // before xs / red are overwritten
    }

    const size_t row = ((size_t)b * a.H_q + hq) * a.n_splits + split;
    for (int i = 0; i < n_dv; ++i) {
        const int dv = tid + i * kGenThreads;
        if (dv < a.d_v) a.part_o[row * a.d_v + dv] = o[i];
    }
    if (tid == 0) {
        a.part_ml[row * 2] = M;
        a.part_ml[row * 2 + 1] = l;
    }
}

// Merge of the generic kernel's chunk partials.
__global__ void combine_generic_kernel(AttendArgs a)
{
    const size_t row = blockIdx.x;                      // b * H_q + hq
    const float *ml = a.part_ml + row * a.n_splits * 2;
    float M = kNegBig;
    for (int i = 0; i < a.n_splits; ++i) M = fmaxf(M, ml[2 * i]);
    float l = 0.f;
    for (int i = 0; i < a.n_splits; ++i) l += ml[2 * i + 1] * ex2_approx(ml[2 * i] - M);
    const float inv = l > 0.f ? 1.f / l : 0.f;
    for (int dv = threadIdx.x; dv < a.d_v; dv += blockDim.x) {
        float o = 0.f;
        for (int i = 0; i < a.n_splits; ++i)
            o += a.part_o[(row * a.n_splits + i) * a.d_v + dv] * ex2_approx(ml[2 * i] - M);
        a.out[row * a.d_v + dv] = o * inv;
    }
}

// ---- host side: kernel choice, decomposition, launches ----
bool stream_shape_ok(const Ctx *ctx, const AttendArgs &a)
{
    const lookat_config &c = ctx->cfg;
    const bool m_ok = c.m == 1 || c.m == 2 || c.m == 4 || c.m == 8 || c.m == 16;
    const bool dv_ok = c.d_v == 64 || c.d_v == 128;
    // rows of the code cache and of V must start on 16-byte boundaries for the 16-byte copies
    const bool rows_ok = (a.L_max * c.m) % 16 == 0 && ((uintptr_t)a.codes % 16) == 0 &&
                         ((uintptr_t)a.v % 16) == 0 && ((uintptr_t)a.lut % 16) == 0;
    return m_ok && dv_ok && rows_ok;
}

size_t stream_smem_bytes(const AttendArgs &a, int stages)
{
    const int heads = a.g < 4 ? a.g : 4;
    const size_t lut_bytes = ((size_t)heads * (a.m * kTableStride + kHeadPad) * 4 + 15) & ~(size_t)15;
    const size_t merge_bytes = (size_t)kWarps * 4 * (a.d_v + 2) * 4;
    const size_t region0 = lut_bytes > merge_bytes ? lut_bytes : merge_bytes;
    const size_t q_bytes = a.fused_lut ? (size_t)4 * a.d_k * 8 : 0;
    const size_t slot = (size_t)kTile * (a.d_v * 2 + 16) + (size_t)kTile * a.m;
    if (a.bulk)   // V boxes (1024-byte aligned, hence the slack), codes, slot barriers
        return region0 + q_bytes + 1024 + (size_t)kWarps * stages * ((size_t)(a.d_v / 64) * 2048 + (size_t)kTile * a.m + 8);
    return region0 + q_bytes + (size_t)kWarps * stages * slot;
}

int stream_stages(const Ctx *ctx, const AttendArgs &a)
{
    const int options[2] = {4, 2};
    for (int s : options)
        if (stream_smem_bytes(a, s) <= (size_t)ctx->max_smem_optin) return s;
    return 0;
}

template <int M_SUB, int DV, int STAGES>
lookat_status stream_kernel_ready(Ctx *ctx, const AttendArgs &a, int *ctas_per_sm)
{
    auto kern = a.bulk ? attend_stream_kernel<M_SUB, DV, STAGES, true> : attend_stream_kernel<M_SUB, DV, STAGES, false>;
    const size_t smem = stream_smem_bytes(a, STAGES);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "attend: shared-memory opt-in");
    int nb = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, kThreads, smem) != cudaSuccess || nb < 1)
        return set_error(ctx, LOOKAT_ERR_CUDA, "attend: the streaming kernel does not fit on an SM");
    *ctas_per_sm = nb;
    return LOOKAT_OK;
}

template <int M_SUB, int DV, int STAGES>
lookat_status stream_launch(Ctx *ctx, const AttendArgs &a)
{
    CUtensorMap v_map;
    memset(&v_map, 0, sizeof(v_map));
    if (a.bulk) {
        // V as [all cache rows][d_v] fp16: boxes of 16 rows x 64 halfs, 128-byte swizzle, zeros beyond the last row
        if (!make_tile_map_f16(&v_map, a.v, (unsigned long long)a.d_v, (unsigned long long)a.B * a.H_kv * a.L_max, 64, kTile))
            return set_error(ctx, LOOKAT_ERR_CUDA, "attend: the tensor map of the value cache was rejected");
        attend_stream_kernel<M_SUB, DV, STAGES, true><<<a.n_ctas, kThreads, stream_smem_bytes(a, STAGES), ctx->stream>>>(a, v_map);
    } else {
        attend_stream_kernel<M_SUB, DV, STAGES, false><<<a.n_ctas, kThreads, stream_smem_bytes(a, STAGES), ctx->stream>>>(a, v_map);
    }
    return check_launch(ctx, "attend_stream_kernel");
}

// Calls f.template operator()<M_SUB, DV, STAGES>() for the runtime (m, d_v, stages).
template <typename F>
lookat_status dispatch_stream(int m, int d_v, int stages, F &&f)
{
#define LOOKAT_CASE(M, D, S) \
    if (m == M && d_v == D && stages == S) return f.template operator()<M, D, S>();
#define LOOKAT_CASES(M) \
    LOOKAT_CASE(M, 64, 4) LOOKAT_CASE(M, 64, 2) LOOKAT_CASE(M, 128, 4) LOOKAT_CASE(M, 128, 2)
    LOOKAT_CASES(1) LOOKAT_CASES(2) LOOKAT_CASES(4) LOOKAT_CASES(8) LOOKAT_CASES(16)
#undef LOOKAT_CASES
#undef LOOKAT_CASE
    return LOOKAT_ERR_UNSUPPORTED;
}

}  // namespace

lookat_status plan_attend(Ctx *ctx, AttendArgs &a, int n_splits, size_t *part_o_floats, size_t *part_ml_floats)
{
    a.fused_lut = (!a.lut && a.d_k <= 256) ? 1 : 0;    // tables built inside the streaming kernel
    // tiles by the bulk-copy engine where the driver provides tensor maps and the row coordinate fits 32 bits
    // (LOOKAT_NO_TENSOR_MAPS in the environment forces the 16-byte cp.async ring, which otherwise runs only where the
    // driver has no tensor-map entry point or the caches have 2^31 rows or more: a switch for tests of that path)
    a.bulk = (tile_maps_available() && (long long)a.B * a.H_kv * a.L_max < (1ll << 31) && !getenv("LOOKAT_NO_TENSOR_MAPS")) ? 1 : 0;
    const int stages = stream_shape_ok(ctx, a) ? stream_stages(ctx, a) : 0;
    if (!stages) a.fused_lut = 0;
    if (stages) {
        const int hgroups = (a.g + 3) / 4;
        const long long units = (long long)a.B * a.H_kv * hgroups;
        // the flat tile sequence covers the tokens that exist: where the host knows the length (no seq_lens), tiles
        // beyond it are left out, so a cache with spare capacity still spreads over every CTA; L_max stays the row stride
        const long long len_plan = a.seq_lens ? a.L_max : (a.uniform_len < a.L_max ? (long long)a.uniform_len : a.L_max);
        const long long tpu = len_plan > 0 ? (len_plan + kTile - 1) / kTile : 1;
        if (units > (1ll << 30) || units * tpu > (1ll << 40))
            return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend: problem too large");
        // rows of up to 8192 tokens go to the kernel that keeps several units' tables resident (attend_multi.cu)
        a.multi = (tpu <= kMultiMaxTiles && units * tpu < (1ll << 30) && multi_fits(ctx, a)) ? 1 : 0;
        int per_sm = 1;
        if (!a.multi) {
            lookat_status st = dispatch_stream(a.m, a.d_v, stages, [&]<int M, int D, int S>() {
                return stream_kernel_ready<M, D, S>(ctx, a, &per_sm);
            });
            if (st != LOOKAT_OK) return st;
        }
        a.stream = 1;
        a.n_units = (int)units;
        a.tiles_per_unit = (int)tpu;
        if (n_splits > 0) {
            long long splits = n_splits < tpu ? n_splits : tpu;
            a.tiles_per_cta = (tpu + splits - 1) / splits;
            splits = (tpu + a.tiles_per_cta - 1) / a.tiles_per_cta;
            if (units * splits > (1ll << 30)) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend: too many chunks");
            a.splits_per_unit = (int)splits;
            a.n_ctas = (int)(units * splits);
        } else {
            const long long total = units * tpu;
            long long ctas = (long long)per_sm * ctx->sm_count;
            if (ctas > total) ctas = total;
            a.tiles_per_cta = (total + ctas - 1) / ctas;
            // short rows that would be cut into less than a unit per CTA: whole units instead (no partials to merge
            // across CTAs; as many 16-tile rounds per warp, or nearly)
            if (a.multi && tpu <= 64 && a.tiles_per_cta <= tpu) a.tiles_per_cta = tpu;
            a.splits_per_unit = 0;
            a.n_ctas = (int)((total + a.tiles_per_cta - 1) / a.tiles_per_cta);
            // ranges that do not cross from one KV head into the next (a CTA stages one head's codebooks): each head's
            // tiles are cut among floor(CTAs / heads) CTAs of its own, where that leaves few SMs idle
            const long long cph = ctas / a.H_kv, tph = (long long)hgroups * a.B * tpu;
            if (a.multi && a.H_kv > 1 && a.tiles_per_cta > tpu && cph >= 1 && cph * a.H_kv * 10 >= ctas * 9) {
                a.tiles_per_cta = (tph + cph - 1) / cph;
                // whole units per CTA where that lengthens the longest range by less than 15 %: no unit is shared, so no
                // partial goes through global memory and no CTA waits on a counter before it may write its rows
                const long long whole = (a.tiles_per_cta + tpu - 1) / tpu * tpu;
                if (whole * 100 <= a.tiles_per_cta * 115) a.tiles_per_cta = whole;
                a.ctas_per_head = (int)((tph + a.tiles_per_cta - 1) / a.tiles_per_cta);
                a.n_ctas = a.ctas_per_head * a.H_kv;
            }
        }
        if (a.multi) {
            // the most units a CTA's range can touch
            const long long span = a.splits_per_unit > 0 ? 1
                                   : (a.tiles_per_cta % tpu == 0 ? a.tiles_per_cta / tpu : (a.tiles_per_cta + tpu - 2) / tpu + 1);
            lookat_status st = plan_multi(ctx, a, (int)(span < kMaxRoundUnits ? span : kMaxRoundUnits));
            if (st != LOOKAT_OK) return st;
        }
        const size_t slots = (size_t)a.n_ctas + (size_t)a.n_units;     // slot of (CTA c, unit u) = c + u
        *part_o_floats = slots * 4 * a.d_v;
        *part_ml_floats = slots * 4 * 2;
        return LOOKAT_OK;
    }
    // generic kernel: chunks of whole 16-token groups, at least 256 tokens unless asked otherwise
    a.stream = 0;
    long long splits = n_splits;
    if (splits <= 0) {
        const long long rows = (long long)a.B * a.H_q;
        splits = (4ll * ctx->sm_count + rows - 1) / rows;
        const long long max_splits = a.L_max / 256 > 0 ? a.L_max / 256 : 1;
        if (splits > max_splits) splits = max_splits;
    }
    if (splits > a.L_max) splits = a.L_max;
    long long chunk = (a.L_max + splits - 1) / splits;
    chunk = (chunk + 15) / 16 * 16;
    splits = (a.L_max + chunk - 1) / chunk;
    if (splits > 65535) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend: more than 65535 chunks");
    a.chunk = (int)chunk;
    a.n_splits = (int)splits;
    *part_o_floats = (size_t)a.B * a.H_q * splits * a.d_v;
    *part_ml_floats = (size_t)a.B * a.H_q * splits * 2;
    return LOOKAT_OK;
}

lookat_status launch_attend(Ctx *ctx, const AttendArgs &a)
{
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    const bool timed = ctx->timing && ctx->ev_count < ctx->ev_cap;     // launches beyond the room asked for go untimed
    if (timed) {
        e0 = ctx->ev0[ctx->ev_count];
        e1 = ctx->ev1[ctx->ev_count];
        cudaEventRecord(e0, ctx->stream);
    }
    lookat_status st;
    if (a.stream && a.multi) {
        st = launch_multi(ctx, a);
    } else if (a.stream) {
        st = dispatch_stream(a.m, a.d_v, stream_stages(ctx, a), [&]<int M, int D, int S>() {
            return stream_launch<M, D, S>(ctx, a);
        });
    } else {
        dim3 grid(a.n_splits, a.H_q, a.B);
        attend_generic_kernel<<<grid, kGenThreads, 0, ctx->stream>>>(a);
        st = check_launch(ctx, "attend_generic_kernel");
    }
    if (timed) {
        cudaEventRecord(e1, ctx->stream);
        ctx->ev_count += 1;
    }
    return st;
}


lookat_status launch_combine(Ctx *ctx, const AttendArgs &a)
{
    // the streaming kernel merges its partials itself; only the generic kernel needs this pass
    int threads = a.d_v < 32 ? 32 : (a.d_v > 256 ? 256 : ((a.d_v + 31) / 32) * 32);
    combine_generic_kernel<<<a.B * a.H_q, threads, 0, ctx->stream>>>(a);
    return check_launch(ctx, "combine_generic_kernel");
}

}  // namespace lookat
