// Multi-query causal attention over the compressed keys (prefill): Algorithm 1
// for a tile of TQ consecutive queries of one head at a time.  Query i stands at
// position q_pos0 + i and attends tokens 0 .. q_pos0 + i.
//
// One CTA per (query tile, query head, batch row), 512 threads:
//   * the tile's lookup tables (Section 3.5 "Precomputation Lookup Tables") are
//     built once into shared memory, query-minor: lut[j][c][ql], so the TQ
//     lanes that score one token for the TQ queries read one contiguous row
//     (fp64 accumulation, one rounding, as everywhere in this library),
//   * tokens are walked in chunks of 64; the codes and V rows of the next chunk
//     are copied (cp.async) while the current one is worked on,
//   * every (query, token) pair is scored by m gathers (Section 3.5 "Lookup and
//     Sum") and masked causally; one warp per query row keeps the online
//     softmax (running maximum and sum, base 2) and writes the weights as two
//     fp16 planes: the rounding and what the rounding left over (~22 bits),
//   * the weighted value sum O[TQ x d_v] += P[TQ x 64] . V[64 x d_v] runs on the
//     tensor cores (mma.sync m16n8k16, fp32 accumulate), once per plane; a warp
//     owns 8 output columns, the V operand comes from the row-major rows by
//     ldmatrix with transpose.
// The cost is bound by the shared-memory gathers (m per pair); the tables cost
// K*d_k multiply-adds per query.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kPfWarps = 16;
constexpr int kPfThreads = kPfWarps * 32;
constexpr int kPfChunk = 64;
constexpr int kPfSPitch = kPfChunk + 1;       // fp32 score rows, padded by one float
constexpr int kPfPPitch = kPfChunk + 8;       // fp16 weight rows, padded by 16 bytes
constexpr float kPfNegBig = -1.0e30f;

__host__ __device__ inline size_t pf_align16(size_t x) { return (x + 15) & ~(size_t)15; }

struct PfLayout {
    unsigned lut, qd, codes, v, s, p_hi, p_lo, state, total;
    unsigned v_pitch;      // bytes per staged V row (row + 16 bytes)
    unsigned code_pitch;   // bytes per staged code row (m rounded up to 4)
};

PfLayout pf_layout(int tq, int d_k, int d_v, int m, int K)
{
    PfLayout l;
    size_t off = 0;
    l.v_pitch = (unsigned)(d_v * 2 + 16);
    l.code_pitch = (unsigned)((m + 3) & ~3);
    l.lut = (unsigned)off;   off += pf_align16((size_t)m * K * tq * 4);
    l.qd = (unsigned)off;    off += pf_align16((size_t)tq * d_k * 8);
    l.codes = (unsigned)off; off += 2 * pf_align16((size_t)kPfChunk * l.code_pitch);
    l.v = (unsigned)off;     off += 2 * pf_align16((size_t)kPfChunk * l.v_pitch);
    l.s = (unsigned)off;     off += pf_align16((size_t)tq * kPfSPitch * 4);
    l.p_hi = (unsigned)off;  off += pf_align16((size_t)16 * kPfPPitch * 2);
    l.p_lo = (unsigned)off;  off += pf_align16((size_t)16 * kPfPPitch * 2);
    l.state = (unsigned)off; off += pf_align16((size_t)3 * 16 * 4);
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

template <int TQ>
__global__ void __launch_bounds__(kPfThreads, 1) attend_prefill_kernel(PrefillArgs a, PfLayout lay)
{
    extern __shared__ __align__(16) unsigned char smem[];
    float *lut = reinterpret_cast<float *>(smem + lay.lut);           // [m][K][TQ]
    double *qd = reinterpret_cast<double *>(smem + lay.qd);           // [TQ][d_k]
    float *s_s = reinterpret_cast<float *>(smem + lay.s);             // [TQ][65]
    __half *p_hi = reinterpret_cast<__half *>(smem + lay.p_hi);       // [16][72]
    __half *p_lo = reinterpret_cast<__half *>(smem + lay.p_lo);       // [16][72]
    float *m_run = reinterpret_cast<float *>(smem + lay.state);       // [16]
    float *l_run = m_run + 16;
    float *alpha_s = l_run + 16;
    const unsigned smem_s = (unsigned)__cvta_generic_to_shared(smem);
    const unsigned codes_bytes = (unsigned)pf_align16((size_t)kPfChunk * lay.code_pitch);
    const unsigned v_bytes = (unsigned)pf_align16((size_t)kPfChunk * lay.v_pitch);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int qtile = gridDim.x - 1 - blockIdx.x;                     // long tiles first
    const int hq = blockIdx.y, b = blockIdx.z;
    const int kvh = hq / a.g;
    const long long q0 = (long long)qtile * TQ;
    const int nq = (int)min((long long)TQ, a.L_q - q0);
    const int d_sub = a.d_k / a.m;

    // ---- queries of the tile, widened; weight planes start as zeros (rows TQ..15 stay zero) ----
    const __half *qrow = a.q + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.d_k;
    for (int i = tid; i < TQ * a.d_k; i += kPfThreads)
        qd[i] = (i / a.d_k) < nq ? (double)__half2float(qrow[i]) : 0.0;
    for (int i = tid; i < 16 * kPfPPitch; i += kPfThreads) {
        p_hi[i] = __float2half(0.f);
        p_lo[i] = __float2half(0.f);
    }
    if (tid < 16) {
        m_run[tid] = kPfNegBig;
        l_run[tid] = 0.f;
        alpha_s[tid] = 1.f;
    }

    const size_t kv_row = (size_t)b * a.H_kv + kvh;
    const uint8_t *codes = a.codes + kv_row * a.L_max * a.m;
    const unsigned char *vrow = reinterpret_cast<const unsigned char *>(a.v + kv_row * a.L_max * a.d_v);
    const long long pos0 = a.q_pos0 + q0;                             // position of the tile's first query
    const long long n_tok = pos0 + nq;                                // tokens the tile's last query sees
    const int v_vec = a.d_v / 8;                                      // 16-byte pieces per V row
    const bool codes_by_word = (a.m & 3) == 0 && ((uintptr_t)codes & 3) == 0;

    // copies of chunk `c0` into buffer `buf`; rows beyond the chunk's tokens are zeros
    auto stage = [&](long long c0, int buf) {
        const int n = (int)min((long long)kPfChunk, n_tok - c0);
        unsigned char *cdst = smem + lay.codes + buf * codes_bytes;
        const unsigned cdst_s = smem_s + lay.codes + buf * codes_bytes;
        if (codes_by_word) {
            const int words = a.m >> 2;
            for (int i = tid; i < kPfChunk * words; i += kPfThreads) {
                if (i / words < n) pf_cp_async4(cdst_s + i * 4, codes + c0 * a.m + (size_t)i * 4);
                else reinterpret_cast<uint32_t *>(cdst)[i] = 0u;
            }
        } else {
            for (int i = tid; i < kPfChunk * a.m; i += kPfThreads) {
                const int tl = i / a.m, j = i - tl * a.m;
                cdst[tl * lay.code_pitch + j] = tl < n ? codes[(c0 + tl) * a.m + j] : 0;
            }
        }
        unsigned char *vdst = smem + lay.v + buf * v_bytes;
        const unsigned vdst_s = smem_s + lay.v + buf * v_bytes;
        for (int i = tid; i < kPfChunk * v_vec; i += kPfThreads) {
            const int tl = i / v_vec, piece = i - tl * v_vec;
            if (tl < n) pf_cp_async16(vdst_s + tl * lay.v_pitch + piece * 16, vrow + ((size_t)(c0 + tl) * v_vec + piece) * 16);
            else *reinterpret_cast<uint4 *>(vdst + tl * lay.v_pitch + piece * 16) = make_uint4(0, 0, 0, 0);
        }
        pf_commit();
    };
    stage(0, 0);                                                       // overlaps the table build
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

    // value-sum ownership: warp w accumulates output columns 8*nt .. 8*nt+7 for nt = w, w+16
    float acc[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
    const int n_tiles = a.d_v / 8;
    float *scores_base =
        a.scores_out ? a.scores_out + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.L_max : nullptr;
    // ldmatrix lane addresses: weights (rows lane&15, tokens 8*(lane>>4)); V (tokens lane&15 of a
    // 16-token step, this warp's 8 columns; lanes 16..31 repeat valid addresses that are not used)
    const unsigned p_lane = (unsigned)(((lane & 15) * kPfPPitch + (lane >> 4) * 8) * 2);
    const unsigned v_lane = (unsigned)((lane & 15) * lay.v_pitch);

    int buf = 0;
    for (long long c0 = 0; c0 < n_tok; c0 += kPfChunk, buf ^= 1) {
        const int n = (int)min((long long)kPfChunk, n_tok - c0);
        pf_wait_all();
        __syncthreads();                      // chunk c0 has landed; the previous chunk's readers are done
        if (c0 + kPfChunk < n_tok) stage(c0 + kPfChunk, buf ^ 1);

        // ---- lookup-and-sum for every (query, token) pair of the chunk, causal mask ----
        const unsigned char *codes_s = smem + lay.codes + buf * codes_bytes;
        for (int idx = tid; idx < TQ * kPfChunk; idx += kPfThreads) {
            const int ql = idx % TQ, tl = idx / TQ;
            const unsigned char *cd = codes_s + tl * lay.code_pitch;
            float s = 0.f;
            if ((a.m & 3) == 0) {
                for (int j4 = 0; j4 < a.m; j4 += 4) {
                    const uint32_t wd = *reinterpret_cast<const uint32_t *>(cd + j4);
                    s += lut[((size_t)(j4 + 0) * a.K + (wd & 0xff)) * TQ + ql];
                    s += lut[((size_t)(j4 + 1) * a.K + ((wd >> 8) & 0xff)) * TQ + ql];
                    s += lut[((size_t)(j4 + 2) * a.K + ((wd >> 16) & 0xff)) * TQ + ql];
                    s += lut[((size_t)(j4 + 3) * a.K + (wd >> 24)) * TQ + ql];
                }
            } else {
                for (int j = 0; j < a.m; ++j) s += lut[((size_t)j * a.K + cd[j]) * TQ + ql];
            }
            const bool valid = ql < nq && tl < n && c0 + tl <= pos0 + ql;
            if (scores_base && valid) scores_base[(size_t)ql * a.L_max + c0 + tl] = s;
            s_s[ql * kPfSPitch + tl] = valid ? s * a.scale_log2 : -INFINITY;
        }
        __syncthreads();

        // ---- online softmax, one warp per query row; weights as fp16 rounding + remainder ----
        for (int r = warp; r < TQ; r += kPfWarps) {
            const float x0 = s_s[r * kPfSPitch + lane], x1 = s_s[r * kPfSPitch + lane + 32];
            float mx = fmaxf(x0, x1);
            for (int d = 16; d; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
            const float m_old = m_run[r];
            const float m_new = fmaxf(m_old, mx);
            const float p0 = ex2_approx(x0 - m_new), p1 = ex2_approx(x1 - m_new);
            float sum = p0 + p1;
            for (int d = 16; d; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
            const __half h0 = __float2half_rn(p0), h1 = __float2half_rn(p1);
            p_hi[r * kPfPPitch + lane] = h0;
            p_hi[r * kPfPPitch + lane + 32] = h1;
            p_lo[r * kPfPPitch + lane] = __float2half_rn(p0 - __half2float(h0));
            p_lo[r * kPfPPitch + lane + 32] = __float2half_rn(p1 - __half2float(h1));
            if (lane == 0) {
                const float al = ex2_approx(m_old - m_new);
                alpha_s[r] = al;
                l_run[r] = l_run[r] * al + sum;
                m_run[r] = m_new;
            }
        }
        __syncthreads();

        // ---- O += P V on the tensor cores: this warp's output columns ----
        const unsigned v_s = smem_s + lay.v + buf * v_bytes;
        const float al0 = alpha_s[lane >> 2], al1 = alpha_s[(lane >> 2) + 8];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int nt = warp + t * kPfWarps;
            if (nt < n_tiles) {
                acc[t][0] *= al0; acc[t][1] *= al0; acc[t][2] *= al1; acc[t][3] *= al1;
#pragma unroll
                for (int ks = 0; ks < kPfChunk / 16; ks += 2) {
                    // V operands of two 16-token steps: tokens 16ks..+7 and +8..15, 8 columns
                    uint32_t vb0[2], vb1[2];
                    pf_ldmatrix_x2_trans(vb0, v_s + (ks * 16) * lay.v_pitch + v_lane + nt * 16);
                    pf_ldmatrix_x2_trans(vb1, v_s + ((ks + 1) * 16) * lay.v_pitch + v_lane + nt * 16);
                    uint32_t ph[4], pl[4];
                    pf_ldmatrix_x4(ph, smem_s + lay.p_hi + p_lane + ks * 32);
                    pf_ldmatrix_x4(pl, smem_s + lay.p_lo + p_lane + ks * 32);
                    pf_mma(acc[t], ph, vb0[0], vb0[1]);
                    pf_mma(acc[t], pl, vb0[0], vb0[1]);
                    pf_ldmatrix_x4(ph, smem_s + lay.p_hi + p_lane + (ks + 1) * 32);
                    pf_ldmatrix_x4(pl, smem_s + lay.p_lo + p_lane + (ks + 1) * 32);
                    pf_mma(acc[t], ph, vb1[0], vb1[1]);
                    pf_mma(acc[t], pl, vb1[0], vb1[1]);
                }
            }
        }
        // the next iteration's barrier separates these reads from the following writes
    }

    // ---- normalise and store: accumulator rows lane/4 and lane/4 + 8, columns 2*(lane%4) + {0,1} ----
    const int r0 = lane >> 2, r1 = r0 + 8, col = 2 * (lane & 3);
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int nt = warp + t * kPfWarps;
        if (nt < n_tiles) {
            float *o = a.out + (((size_t)b * a.H_q + hq) * a.L_q + q0) * a.d_v + nt * 8 + col;
            if (r0 < nq) {
                const float inv = 1.f / l_run[r0];                    // token 0 is always visible: l > 0
                *reinterpret_cast<float2 *>(o + (size_t)r0 * a.d_v) = make_float2(acc[t][0] * inv, acc[t][1] * inv);
            }
            if (r1 < nq) {
                const float inv = 1.f / l_run[r1];
                *reinterpret_cast<float2 *>(o + (size_t)r1 * a.d_v) = make_float2(acc[t][2] * inv, acc[t][3] * inv);
            }
        }
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
    if (a.d_v % 8 != 0 || a.d_v > 256 || ((uintptr_t)a.v & 15) != 0)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_prefill: d_v must be a multiple of 8, at most 256");
    // 16 queries per tile when their tables fit in shared memory, else 8
    for (int tq : {16, 8}) {
        if (pf_layout(tq, a.d_k, a.d_v, a.m, a.K).total > (size_t)ctx->max_smem_optin) continue;
        return tq == 16 ? launch_pf<16>(ctx, a) : launch_pf<8>(ctx, a);
    }
    return set_error(ctx, LOOKAT_ERR_UNSUPPORTED,
                     "attend_prefill: the tables of 8 queries (m*K*32 bytes) do not fit in shared memory");
}

}  // namespace lookat
