// Multi-query causal attention over the compressed keys (prefill): Algorithm 1
// for a tile of TQ consecutive queries of one head at a time.  Query i stands at
// position q_pos0 + i and attends tokens 0 .. q_pos0 + i.
//
// One CTA per (query tile, query head, batch row), 256 threads:
//   * the tile's lookup tables (Section 3.5 "Precomputation Lookup Tables") are
//     built once into shared memory, query-minor: lut[j][c][ql], so the TQ
//     lanes that score one token for the TQ queries read one contiguous row,
//   * tokens are walked in chunks of 64: codes and V rows of the chunk are
//     staged in shared memory, every (query, token) pair is scored by m
//     gathers (Section 3.5 "Lookup and Sum") and masked causally,
//   * per query row an online softmax (running maximum and sum, base 2), then
//     the weighted value sum with fp32 accumulators (CUDA cores in this
//     version: 16 or 32 threads per query, each a slice of d_v).
// The cost is dominated by the shared-memory gathers (m per pair) and the
// d_v multiply-adds per pair; the tables cost K*d_k multiply-adds per query.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kPfThreads = 256;
constexpr int kPfChunk = 64;
constexpr int kPfPitch = kPfChunk + 1;      // score rows are padded by one float
constexpr float kPfNegBig = -1.0e30f;

size_t pf_align16(size_t x) { return (x + 15) & ~(size_t)15; }

struct PfLayout {
    size_t lut, qd, codes, v, s, state, total;
};

PfLayout pf_layout(int tq, int d_k, int d_v, int m, int K)
{
    PfLayout l;
    size_t off = 0;
    l.lut = off;   off += pf_align16((size_t)m * K * tq * 4);
    l.qd = off;    off += pf_align16((size_t)tq * d_k * 8);
    l.codes = off; off += pf_align16((size_t)kPfChunk * m);
    l.v = off;     off += pf_align16((size_t)kPfChunk * d_v * 2);
    l.s = off;     off += pf_align16((size_t)tq * kPfPitch * 4);
    l.state = off; off += pf_align16((size_t)3 * tq * 4);
    l.total = off;
    return l;
}

template <int TQ>
__global__ void __launch_bounds__(kPfThreads) attend_prefill_kernel(PrefillArgs a, PfLayout lay)
{
    extern __shared__ __align__(16) unsigned char smem[];
    float *lut = reinterpret_cast<float *>(smem + lay.lut);           // [m][K][TQ]
    double *qd = reinterpret_cast<double *>(smem + lay.qd);           // [TQ][d_k]
    unsigned char *codes_s = smem + lay.codes;                        // [64][m]
    __half *v_s = reinterpret_cast<__half *>(smem + lay.v);           // [64][d_v]
    float *s_s = reinterpret_cast<float *>(smem + lay.s);             // [TQ][65]
    float *m_run = reinterpret_cast<float *>(smem + lay.state);       // [TQ]
    float *l_run = m_run + TQ;
    float *alpha_s = l_run + TQ;

    constexpr int TPQ = kPfThreads / TQ;                              // threads per query in the value sum
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int qtile = gridDim.x - 1 - blockIdx.x;                     // long tiles first
    const int hq = blockIdx.y, b = blockIdx.z;
    const int kvh = hq / a.g;
    const long long q0 = (long long)qtile * TQ;
    const int nq = (int)min((long long)TQ, a.L_q - q0);
    const int d_sub = a.d_k / a.m;
    const int dvt = a.d_v / TPQ;                                      // value columns per thread (<= 8)

    // ---- queries of the tile, widened ----
    const __half *qrow = a.q + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.d_k;
    for (int i = tid; i < TQ * a.d_k; i += kPfThreads)
        qd[i] = (i / a.d_k) < nq ? (double)__half2float(qrow[i]) : 0.0;
    if (tid < TQ) {
        m_run[tid] = kPfNegBig;
        l_run[tid] = 0.f;
    }
    __syncthreads();

    // ---- tables of the tile: lut[j][c][ql] = q_ql^(j) . C_j[c], fp64 accumulation ----
    const float *book = a.codebooks + (size_t)kvh * a.m * a.K * d_sub;
    for (int e = tid; e < a.m * a.K; e += kPfThreads) {
        const int j = e / a.K;
        const float *cen = book + (size_t)e * d_sub;
        const double *qj = qd + j * d_sub;
        double acc[TQ];
#pragma unroll
        for (int ql = 0; ql < TQ; ++ql) acc[ql] = 0.0;
        for (int i = 0; i < d_sub; ++i) {
            const double cv = (double)__ldg(cen + i);
#pragma unroll
            for (int ql = 0; ql < TQ; ++ql) acc[ql] = fma(qj[ql * a.d_k + i], cv, acc[ql]);
        }
#pragma unroll
        for (int ql = 0; ql < TQ; ql += 4)
            *reinterpret_cast<float4 *>(lut + (size_t)e * TQ + ql) =
                make_float4((float)acc[ql], (float)acc[ql + 1], (float)acc[ql + 2], (float)acc[ql + 3]);
    }
    __syncthreads();

    const size_t kv_row = (size_t)b * a.H_kv + kvh;
    const uint8_t *codes = a.codes + kv_row * a.L_max * a.m;
    const __half *vrow = a.v + kv_row * a.L_max * a.d_v;
    const long long pos0 = a.q_pos0 + q0;                             // position of the tile's first query
    const long long n_tok = pos0 + nq;                                // tokens the last query of the tile sees
    const int qr = tid / TPQ, dv0 = (tid % TPQ) * dvt;
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
    float *scores_base =
        a.scores_out ? a.scores_out + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.L_max : nullptr;

    for (long long c0 = 0; c0 < n_tok; c0 += kPfChunk) {
        const int n = (int)min((long long)kPfChunk, n_tok - c0);
        // ---- stage the chunk: codes and V rows; rows beyond the chunk's tokens are zeros ----
        for (int i = tid; i < kPfChunk * a.m; i += kPfThreads)
            codes_s[i] = i < n * a.m ? codes[c0 * a.m + i] : 0;
        const int v_vec = a.d_v / 8;                                  // 16-byte pieces per row
        for (int i = tid; i < kPfChunk * v_vec; i += kPfThreads) {
            uint4 x = make_uint4(0, 0, 0, 0);
            if (i / v_vec < n) x = __ldg(reinterpret_cast<const uint4 *>(vrow + c0 * a.d_v) + i);
            reinterpret_cast<uint4 *>(v_s)[i] = x;
        }
        __syncthreads();

        // ---- lookup-and-sum for every (query, token) pair of the chunk, causal mask ----
        for (int idx = tid; idx < TQ * kPfChunk; idx += kPfThreads) {
            const int ql = idx % TQ, tl = idx / TQ;
            const unsigned char *cd = codes_s + tl * a.m;
            float s = 0.f;
            for (int j = 0; j < a.m; ++j) s += lut[((size_t)j * a.K + cd[j]) * TQ + ql];
            const bool valid = ql < nq && tl < n && c0 + tl <= pos0 + ql;
            if (scores_base && valid) scores_base[(size_t)ql * a.L_max + c0 + tl] = s;
            s_s[ql * kPfPitch + tl] = valid ? s * a.scale_log2 : -INFINITY;
        }
        __syncthreads();

        // ---- online softmax, one warp per query row ----
        for (int r = warp; r < TQ; r += kPfThreads / 32) {
            const float x0 = s_s[r * kPfPitch + lane], x1 = s_s[r * kPfPitch + lane + 32];
            float mx = fmaxf(x0, x1);
            for (int d = 16; d; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
            const float m_old = m_run[r];
            const float m_new = fmaxf(m_old, mx);
            const float p0 = ex2_approx(x0 - m_new), p1 = ex2_approx(x1 - m_new);
            float sum = p0 + p1;
            for (int d = 16; d; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
            s_s[r * kPfPitch + lane] = p0;
            s_s[r * kPfPitch + lane + 32] = p1;
            if (lane == 0) {
                const float al = ex2_approx(m_old - m_new);
                alpha_s[r] = al;
                l_run[r] = l_run[r] * al + sum;
                m_run[r] = m_new;
            }
        }
        __syncthreads();

        // ---- weighted value sum: this thread's slice of one query's output ----
        {
            const float al = alpha_s[qr];
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] *= al;
            const float *prow = s_s + qr * kPfPitch;
            for (int tl = 0; tl < n; ++tl) {
                const float p = prow[tl];
                const __half *vr = v_s + tl * a.d_v + dv0;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (k < dvt) acc[k] = fmaf(p, __half2float(vr[k]), acc[k]);
            }
        }
        __syncthreads();
    }

    if (qr < nq) {
        const float inv = 1.f / l_run[qr];                            // token 0 is always visible: l > 0
        float *o = a.out + (((size_t)b * a.H_q + hq) * a.L_q + q0 + qr) * a.d_v + dv0;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (k < dvt) o[k] = acc[k] * inv;
    }
}

template <int TQ>
lookat_status launch_pf(Ctx *ctx, const PrefillArgs &a)
{
    const PfLayout lay = pf_layout(TQ, a.d_k, a.d_v, a.m, a.K);
    auto kern = attend_prefill_kernel<TQ>;
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
    // 16 queries per tile when the tables fit in shared memory, else 8
    for (int tq : {16, 8}) {
        const int tpq = kPfThreads / tq;
        if (a.d_v % tpq != 0 || a.d_v / tpq > 8) continue;
        if (pf_layout(tq, a.d_k, a.d_v, a.m, a.K).total > (size_t)ctx->max_smem_optin) continue;
        return tq == 16 ? launch_pf<16>(ctx, a) : launch_pf<8>(ctx, a);
    }
    return set_error(ctx, LOOKAT_ERR_UNSUPPORTED,
                     "attend_prefill: needs d_v a multiple of 32 up to 256 and tables of 8 queries "
                     "(m*K*32 bytes) within shared memory");
}

}  // namespace lookat
