// Multi-query causal attention over the compressed keys (prefill): Algorithm 1
// for a tile of TQ consecutive queries of one head at a time.  Query i stands at
// position q_pos0 + i and attends tokens 0 .. q_pos0 + i.
//
// One CTA per (query tile, query head, batch row), 512 threads:
//   * the tile's lookup tables (Section 3.5 "Precomputation Lookup Tables") are
//     built once into shared memory, query-minor: lut[j][c][ql], so one 16-byte
//     read serves one token for 4 queries (fp64 accumulation, one rounding, as
//     everywhere in this library),
//   * the CTA's two halves (8 warps each, each with its own hardware barrier)
//     share the tables and walk alternate chunks of CHUNK tokens on their own,
//     so one half's copies, gathers, softmax and value sum overlap the other's;
//     each half keeps its own running maximum, sum and accumulators, merged at
//     the end,
//   * per chunk: codes and V rows are copied to shared memory (cp.async), every
//     (query, token) pair is scored by m gathers (Section 3.5 "Lookup and Sum")
//     and masked causally, one warp per query row updates the online softmax
//     (base 2) and writes the weights as two fp16 planes (the rounding and what
//     it left over, ~22 bits), and the weighted value sum
//     O[TQ x d_v] += P[TQ x CHUNK] . V[CHUNK x d_v] runs on the tensor cores
//     (mma.sync m16n8k16, fp32 accumulate), once per plane; a warp owns 8-column
//     slices of the output, the V operand comes from the row-major rows by
//     ldmatrix with transpose.
// The cost is bound by the shared-memory gathers (m per pair); the tables cost
// K*d_k multiply-adds per query.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kPfWarps = 16;
constexpr int kPfThreads = kPfWarps * 32;
constexpr int kPfGroupWarps = 8;                  // warps per half
constexpr int kPfGroupThreads = kPfGroupWarps * 32;
constexpr int kPfMaxSlices = 4;                   // 8-column output slices per warp (d_v <= 256)
constexpr float kPfNegBig = -1.0e30f;

// tokens per chunk (64 or 128): fp32 score rows are padded by one float, fp16 weight rows by 16 bytes
__host__ __device__ constexpr int pf_s_pitch(int chunk) { return chunk + 1; }
__host__ __device__ constexpr int pf_p_pitch(int chunk) { return chunk + 8; }
__host__ __device__ inline size_t pf_align16(size_t x) { return (x + 15) & ~(size_t)15; }

// Shared-memory map; the per-half regions are `*_bytes` apart.
struct PfLayout {
    unsigned lut, qd, codes, v, s, p_hi, p_lo, state, total;
    unsigned codes_bytes, v_bytes, s_bytes, p_bytes, state_bytes;
    unsigned v_pitch;      // bytes per staged V row (row + 16 bytes)
    unsigned code_pitch;   // bytes per staged code row (m rounded up to 4)
};

PfLayout pf_layout(int tq, int chunk, int d_k, int d_v, int m, int K)
{
    PfLayout l;
    size_t off = 0;
    l.v_pitch = (unsigned)(d_v * 2 + 16);
    l.code_pitch = (unsigned)((m + 3) & ~3);
    l.codes_bytes = (unsigned)pf_align16((size_t)chunk * l.code_pitch);
    l.v_bytes = (unsigned)pf_align16((size_t)chunk * l.v_pitch);
    l.s_bytes = (unsigned)pf_align16((size_t)tq * pf_s_pitch(chunk) * 4);
    l.p_bytes = (unsigned)pf_align16((size_t)16 * pf_p_pitch(chunk) * 2);
    l.state_bytes = (unsigned)pf_align16((size_t)3 * 16 * 4);
    l.lut = (unsigned)off;   off += pf_align16((size_t)m * K * tq * 4);
    l.qd = (unsigned)off;    off += pf_align16((size_t)tq * d_k * 8);
    l.codes = (unsigned)off; off += 2 * (size_t)l.codes_bytes;
    l.v = (unsigned)off;     off += 2 * (size_t)l.v_bytes;
    l.s = (unsigned)off;     off += 2 * (size_t)l.s_bytes;
    l.p_hi = (unsigned)off;  off += 2 * (size_t)l.p_bytes;
    l.p_lo = (unsigned)off;  off += 2 * (size_t)l.p_bytes;
    l.state = (unsigned)off; off += 2 * (size_t)l.state_bytes;
    l.total = (unsigned)off;
    return l;
}

__device__ __forceinline__ void pf_cp_async16(unsigned dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void pf_cp_async4(unsigned dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void pf_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void pf_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// hardware barrier of one half of the CTA (ids 1 and 2; id 0 is __syncthreads)
__device__ __forceinline__ void pf_group_barrier(int group)
{
    asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "n"(kPfGroupThreads) : "memory");
}

__device__ __forceinline__ void pf_ldmatrix_x4(uint32_t (&r)[4], unsigned src)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(src));
}
__device__ __forceinline__ void pf_ldmatrix_x2_trans(uint32_t (&r)[2], unsigned src)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];"
                 : "=r"(r[0]), "=r"(r[1])
                 : "r"(src));
}
__device__ __forceinline__ void pf_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int TQ, int CHUNK>
__global__ void __launch_bounds__(kPfThreads, 1) attend_prefill_kernel(PrefillArgs a, PfLayout lay)
{
    constexpr int S_PITCH = pf_s_pitch(CHUNK), P_PITCH = pf_p_pitch(CHUNK);
    extern __shared__ __align__(16) unsigned char smem[];
    const unsigned smem_s = (unsigned)__cvta_generic_to_shared(smem);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grp = warp / kPfGroupWarps;                             // which half of the CTA
    const int gw = warp % kPfGroupWarps, gtid = tid % kPfGroupThreads;
    const int qtile = gridDim.x - 1 - blockIdx.x;                     // long tiles first
    const int hq = blockIdx.y, b = blockIdx.z;
    const int kvh = hq / a.g;
    const long long q0 = (long long)qtile * TQ;
    const int nq = (int)min((long long)TQ, a.L_q - q0);
    const int d_sub = a.d_k / a.m;

    float *lut = reinterpret_cast<float *>(smem + lay.lut);                          // [m][K][TQ]
    double *qd = reinterpret_cast<double *>(smem + lay.qd);                          // [TQ][d_k]
    // this half's regions
    unsigned char *codes_s = smem + lay.codes + grp * lay.codes_bytes;               // [CHUNK][code_pitch]
    unsigned char *v_sm = smem + lay.v + grp * lay.v_bytes;                          // [CHUNK][v_pitch]
    float *s_s = reinterpret_cast<float *>(smem + lay.s + grp * lay.s_bytes);        // [TQ][S_PITCH]
    __half *p_hi = reinterpret_cast<__half *>(smem + lay.p_hi + grp * lay.p_bytes);  // [16][P_PITCH]
    __half *p_lo = reinterpret_cast<__half *>(smem + lay.p_lo + grp * lay.p_bytes);
    float *m_run = reinterpret_cast<float *>(smem + lay.state + grp * lay.state_bytes);   // [16] each
    float *l_run = m_run + 16;
    float *alpha_s = l_run + 16;

    // ---- queries of the tile, widened; weight planes start as zeros (rows TQ..15 stay zero) ----
    const __half *qrow = a.q + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.d_k;
    for (int i = tid; i < TQ * a.d_k; i += kPfThreads)
        qd[i] = (i / a.d_k) < nq ? (double)__half2float(qrow[i]) : 0.0;
    for (int i = gtid; i < 16 * P_PITCH; i += kPfGroupThreads) {
        p_hi[i] = __float2half(0.f);
        p_lo[i] = __float2half(0.f);
    }
    if (gtid < 16) {
        m_run[gtid] = kPfNegBig;
        l_run[gtid] = 0.f;
        alpha_s[gtid] = 1.f;
    }
    __syncthreads();

    // ---- tables of the tile: lut[j][c][ql] = q_ql^(j) . C_j[c], fp64 accumulation ----
    const float *book = a.codebooks + (size_t)kvh * a.m * a.K * d_sub;
    for (int e = tid; e < a.m * a.K; e += kPfThreads) {
        const int j = e / a.K;
        const float *cen = book + (size_t)e * d_sub;
        const double *qj = qd + j * d_sub;
        double t[TQ];
#pragma unroll
        for (int ql = 0; ql < TQ; ++ql) t[ql] = 0.0;
        for (int i = 0; i < d_sub; ++i) {
            const double cv = (double)__ldg(cen + i);
#pragma unroll
            for (int ql = 0; ql < TQ; ++ql) t[ql] = fma(qj[ql * a.d_k + i], cv, t[ql]);
        }
#pragma unroll
        for (int ql = 0; ql < TQ; ql += 4)
            *reinterpret_cast<float4 *>(lut + (size_t)e * TQ + ql) =
                make_float4((float)t[ql], (float)t[ql + 1], (float)t[ql + 2], (float)t[ql + 3]);
    }
    __syncthreads();

    const size_t kv_row = (size_t)b * a.H_kv + kvh;
    const uint8_t *codes = a.codes + kv_row * a.L_max * a.m;
    const unsigned char *vrow = reinterpret_cast<const unsigned char *>(a.v + kv_row * a.L_max * a.d_v);
    const long long pos0 = a.q_pos0 + q0;                             // position of the tile's first query
    const long long n_tok = pos0 + nq;                                // tokens the tile's last query sees
    const int v_vec = a.d_v / 8;                                      // 16-byte pieces per V row
    const bool codes_by_word = (a.m & 3) == 0;
    const int n_slices = a.d_v / 8;                                   // 8-column output slices
    float *scores_base =
        a.scores_out ? a.scores_out + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.L_max : nullptr;

    // value-sum ownership: warp gw of a half accumulates output slices gw, gw+8, gw+16, gw+24
    float acc[kPfMaxSlices][4];
#pragma unroll
    for (int t = 0; t < kPfMaxSlices; ++t) acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
    // ldmatrix lane addresses: weights (rows lane&15, tokens 8*(lane>>4)); V (tokens lane&15 of a
    // 16-token step; lanes 16..31 repeat valid addresses that are not used)
    const unsigned p_lane = (unsigned)(((lane & 15) * P_PITCH + (lane >> 4) * 8) * 2);
    const unsigned v_lane = (unsigned)((lane & 15) * lay.v_pitch);
    const unsigned p_hi_s = smem_s + lay.p_hi + grp * lay.p_bytes, p_lo_s = smem_s + lay.p_lo + grp * lay.p_bytes;
    const unsigned v_s = smem_s + lay.v + grp * lay.v_bytes;
    const unsigned codes_ss = smem_s + lay.codes + grp * lay.codes_bytes;

    // ---- this half's chunks: grp, grp+2, grp+4, ... ----
    for (long long c0 = (long long)grp * CHUNK; c0 < n_tok; c0 += 2 * CHUNK) {
        const int n = (int)min((long long)CHUNK, n_tok - c0);
        // ---- copy the chunk's codes and V rows; rows beyond its tokens are zeros ----
        if (codes_by_word) {
            const int words = a.m >> 2;
            for (int i = gtid; i < CHUNK * words; i += kPfGroupThreads) {
                if (i / words < n) pf_cp_async4(codes_ss + i * 4, codes + c0 * a.m + (size_t)i * 4);
                else reinterpret_cast<uint32_t *>(codes_s)[i] = 0u;
            }
        } else {
            for (int i = gtid; i < CHUNK * a.m; i += kPfGroupThreads) {
                const int tl = i / a.m, j = i - tl * a.m;
                codes_s[tl * lay.code_pitch + j] = tl < n ? codes[(c0 + tl) * a.m + j] : 0;
            }
        }
        {
            const int tl0 = gtid / v_vec, piece = gtid - tl0 * v_vec;     // threads walk rows in steps
            const int rows_per_pass = kPfGroupThreads / v_vec;
            const unsigned char *src = vrow + ((size_t)(c0 + tl0) * v_vec + piece) * 16;
            if (tl0 < rows_per_pass)
                for (int tl = tl0; tl < CHUNK; tl += rows_per_pass, src += (size_t)rows_per_pass * v_vec * 16) {
                    if (tl < n) pf_cp_async16(v_s + tl * lay.v_pitch + piece * 16, src);
                    else *reinterpret_cast<uint4 *>(v_sm + tl * lay.v_pitch + piece * 16) = make_uint4(0, 0, 0, 0);
                }
        }
        pf_commit();
        pf_wait_all();
        pf_group_barrier(grp);                // the chunk has landed for the whole half

        // ---- lookup-and-sum for every (query, token) pair of the chunk, causal mask;
        //      a thread scores one token for 4 consecutive queries: every gather is one 16-byte read ----
        for (int idx = gtid; idx < (TQ / 4) * CHUNK; idx += kPfGroupThreads) {
            const int qg = idx % (TQ / 4), tl = idx / (TQ / 4);
            const unsigned char *cd = codes_s + tl * lay.code_pitch;
            const float4 *row = reinterpret_cast<const float4 *>(lut) + qg;     // + entry * (TQ/4)
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            auto add = [&](int entry) {
                const float4 t = row[entry * (TQ / 4)];
                s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
            };
            if (codes_by_word) {
                for (int j4 = 0; j4 < a.m; j4 += 4) {
                    const uint32_t wd = *reinterpret_cast<const uint32_t *>(cd + j4);
                    add((j4 + 0) * a.K + (int)(wd & 0xff));
                    add((j4 + 1) * a.K + (int)((wd >> 8) & 0xff));
                    add((j4 + 2) * a.K + (int)((wd >> 16) & 0xff));
                    add((j4 + 3) * a.K + (int)(wd >> 24));
                }
            } else {
                for (int j = 0; j < a.m; ++j) add(j * a.K + cd[j]);
            }
            const float sv[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int ql = qg * 4 + k;
                const bool valid = ql < nq && tl < n && c0 + tl <= pos0 + ql;
                if (scores_base && valid) scores_base[(size_t)ql * a.L_max + c0 + tl] = sv[k];
                s_s[ql * S_PITCH + tl] = valid ? sv[k] * a.scale_log2 : -INFINITY;
            }
        }
        pf_group_barrier(grp);

        // ---- online softmax, one warp per query row; weights as fp16 rounding + remainder ----
        for (int r = gw; r < TQ; r += kPfGroupWarps) {
            constexpr int PER = CHUNK / 32;                           // values per lane
            float x[PER], p[PER];
            float mx = -INFINITY;
#pragma unroll
            for (int k = 0; k < PER; ++k) {
                x[k] = s_s[r * S_PITCH + lane + 32 * k];
                mx = fmaxf(mx, x[k]);
            }
            for (int d = 16; d; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
            const float m_old = m_run[r];
            const float m_new = fmaxf(m_old, mx);
            float sum = 0.f;
#pragma unroll
            for (int k = 0; k < PER; ++k) {
                p[k] = ex2_approx(x[k] - m_new);
                sum += p[k];
            }
            for (int d = 16; d; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
#pragma unroll
            for (int k = 0; k < PER; ++k) {
                const __half h = __float2half_rn(p[k]);
                p_hi[r * P_PITCH + lane + 32 * k] = h;
                p_lo[r * P_PITCH + lane + 32 * k] = __float2half_rn(p[k] - __half2float(h));
            }
            if (lane == 0) {
                const float al = ex2_approx(m_old - m_new);
                alpha_s[r] = al;
                l_run[r] = l_run[r] * al + sum;
                m_run[r] = m_new;
            }
        }
        pf_group_barrier(grp);

        // ---- O += P V on the tensor cores: this warp's output slices ----
        const float al0 = alpha_s[lane >> 2], al1 = alpha_s[(lane >> 2) + 8];
#pragma unroll
        for (int t = 0; t < kPfMaxSlices; ++t) {
            const int nt = gw + t * kPfGroupWarps;
            if (nt < n_slices) {
                acc[t][0] *= al0; acc[t][1] *= al0; acc[t][2] *= al1; acc[t][3] *= al1;
#pragma unroll
                for (int ks = 0; ks < CHUNK / 16; ++ks) {
                    uint32_t vb[2], ph[4], pl[4];                     // V: tokens 16ks..+7 and +8..15, 8 columns
                    pf_ldmatrix_x2_trans(vb, v_s + (ks * 16) * lay.v_pitch + v_lane + nt * 16);
                    pf_ldmatrix_x4(ph, p_hi_s + p_lane + ks * 32);
                    pf_ldmatrix_x4(pl, p_lo_s + p_lane + ks * 32);
                    pf_mma(acc[t], ph, vb[0], vb[1]);
                    pf_mma(acc[t], pl, vb[0], vb[1]);
                }
            }
        }
        pf_group_barrier(grp);                // before the next chunk overwrites V, scores and weights
    }

    // ---- merge the two halves: M = max, l and O rescaled (accumulator rows lane/4 and lane/4 + 8) ----
    __syncthreads();
    float *xch = reinterpret_cast<float *>(smem + lay.v);             // the copy areas are free now
    const float *m_a = reinterpret_cast<const float *>(smem + lay.state);
    const float *m_b = reinterpret_cast<const float *>(smem + lay.state + lay.state_bytes);
    const int r0 = lane >> 2, r1 = r0 + 8, col = 2 * (lane & 3);
    if (grp == 1) {
#pragma unroll
        for (int t = 0; t < kPfMaxSlices; ++t)
#pragma unroll
            for (int k = 0; k < 4; ++k) xch[((gw * kPfMaxSlices + t) * 4 + k) * 32 + lane] = acc[t][k];
    }
    __syncthreads();
    if (grp == 0) {
        const float M0 = fmaxf(m_a[r0], m_b[r0]), M1 = fmaxf(m_a[r1], m_b[r1]);
        const float fa0 = ex2_approx(m_a[r0] - M0), fb0 = ex2_approx(m_b[r0] - M0);
        const float fa1 = ex2_approx(m_a[r1] - M1), fb1 = ex2_approx(m_b[r1] - M1);
        const float l0 = fa0 * m_a[16 + r0] + fb0 * m_b[16 + r0];     // l_run sits 16 floats after m_run
        const float l1 = fa1 * m_a[16 + r1] + fb1 * m_b[16 + r1];
#pragma unroll
        for (int t = 0; t < kPfMaxSlices; ++t) {
            const int nt = gw + t * kPfGroupWarps;
            if (nt < n_slices) {
                float o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float other = xch[((gw * kPfMaxSlices + t) * 4 + k) * 32 + lane];
                    o[k] = (k < 2 ? fa0 : fa1) * acc[t][k] + (k < 2 ? fb0 : fb1) * other;
                }
                float *dst = a.out + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.d_v + nt * 8 + col;
                if (r0 < nq)                                          // token 0 is always visible: l > 0
                    *reinterpret_cast<float2 *>(dst + (size_t)r0 * a.d_v) = make_float2(o[0] / l0, o[1] / l0);
                if (r1 < nq)
                    *reinterpret_cast<float2 *>(dst + (size_t)r1 * a.d_v) = make_float2(o[2] / l1, o[3] / l1);
            }
        }
    }
}

template <int TQ, int CHUNK>
lookat_status launch_pf(Ctx *ctx, const PrefillArgs &a)
{
    const PfLayout lay = pf_layout(TQ, CHUNK, a.d_k, a.d_v, a.m, a.K);
    auto kern = attend_prefill_kernel<TQ, CHUNK>;
    if (lay.total > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lay.total) != cudaSuccess)
        return check_launch(ctx, "prefill: shared-memory opt-in");
    dim3 grid((unsigned)((a.L_q + TQ - 1) / TQ), a.H_q, a.B);
    kern<<<grid, kPfThreads, lay.total, ctx->stream>>>(a, lay);
    return check_launch(ctx, "attend_prefill_kernel");
}

}  // namespace

lookat_status launch_prefill(Ctx *ctx, const PrefillArgs &a)
{
    // contraction form (tcgen05) where it applies
    const bool want = ctx->prefill_form == LOOKAT_PREFILL_CONTRACTION;
    const bool auto_pick = ctx->prefill_form == LOOKAT_PREFILL_AUTO && a.L_q >= 32;
    if (want || auto_pick) {
        if (prefill_umma_covers(ctx, a)) return launch_prefill_umma(ctx, a);
        if (want)
            return set_error(ctx, LOOKAT_ERR_UNSUPPORTED,
                             "attend_prefill: the contraction form needs d_k, d_v in {64, 128}, d_sub 4 or a multiple of 8, L_max * m a "
                             "multiple of 4, a positive scale and K * d_k * 4 bytes of shared memory for the codebooks");
    }
    if (a.d_v % 8 != 0 || a.d_v > 256 || ((uintptr_t)a.v & 15) != 0 || ((uintptr_t)a.codes & 3) != 0)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_prefill: d_v must be a multiple of 8, at most 256");
    // 16 queries per tile when their tables fit in shared memory, else 8; 128-token chunks when they fit
    const size_t cap = (size_t)ctx->max_smem_optin;
    if (pf_layout(16, 128, a.d_k, a.d_v, a.m, a.K).total <= cap) return launch_pf<16, 128>(ctx, a);
    if (pf_layout(16, 64, a.d_k, a.d_v, a.m, a.K).total <= cap) return launch_pf<16, 64>(ctx, a);
    if (pf_layout(8, 128, a.d_k, a.d_v, a.m, a.K).total <= cap) return launch_pf<8, 128>(ctx, a);
    if (pf_layout(8, 64, a.d_k, a.d_v, a.m, a.K).total <= cap) return launch_pf<8, 64>(ctx, a);
    return set_error(ctx, LOOKAT_ERR_UNSUPPORTED,
                     "attend_prefill: the tables of 8 queries (m*K*32 bytes) do not fit in shared memory");
}

}  // namespace lookat
