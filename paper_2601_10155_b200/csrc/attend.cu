// Fused ADC scoring + online softmax + value accumulation (Section 3.5 "Lookup
// and Sum"; Algorithm 1, second loop and continuation), split over sequence
// chunks, plus the merge of the chunk partials.
//
// Streaming kernel (attend_stream_kernel), one CTA per (chunk, KV head x head
// group, batch row); each of its 8 warps walks 16-token tiles on its own:
//   * codes and V go from global memory straight to registers with 16-byte
//     loads, one tile ahead of the arithmetic (V is ~97 % of the bytes; nothing
//     is reused, so it is never staged in shared memory),
//   * the query group's tables sit in shared memory, one padded table set per
//     head; a lane scores two (token, head) pairs per tile by m gathers each,
//   * the weighted value sum  O^T[d_v x heads] += V^T[d_v x 16 tokens] . P[16 x heads]
//     runs on the tensor cores (mma.sync m16n8k16, fp16 in, fp32 accumulate).
//     The 8 columns hold the <= 4 heads of the group twice: the fp16 rounding of
//     each weight and the fp16 rounding of its remainder, so weights carry
//     ~22 bits.  The token-pair operand layout is produced from the row-major V
//     registers by byte permutes.
// Up to 4 query heads of a KV head share one pass over that head's codes and V.
//
// Generic kernel (attend_generic_kernel): any shape, plain loads, tables read
// from global memory; used where the streaming kernel's layout assumptions
// (d_v in {64,128}, m in {1,2,4,8,16}, 16-byte aligned rows) do not hold.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kTile = 16;           // tokens per warp step (the MMA's k extent)
constexpr int kHeadPad = 8;         // floats between the table sets of two heads (bank shift)
constexpr float kNegBig = -1.0e30f; // running-max start: finite, so differences never give NaN

__device__ __forceinline__ uint4 ldg_stream16(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                          uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// fp16 rounding of p (part 0) or of what that rounding left over (part 1).
__device__ __forceinline__ __half weight_part(float p, int part)
{
    __half h = __float2half_rn(p);
    if (part) h = __float2half_rn(p - __half2float(h));
    return h;
}

__device__ __forceinline__ uint32_t pack_half2(__half lo, __half hi)
{
    return (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
}

template <int M_SUB>
struct CodePair {                    // the codes of two consecutive tokens
    uint32_t w[(2 * M_SUB + 3) / 4];
};

template <int M_SUB>
__device__ __forceinline__ CodePair<M_SUB> load_code_pair(const uint8_t *p)
{
    CodePair<M_SUB> c;
    if constexpr (M_SUB == 16) {
        uint4 a = *reinterpret_cast<const uint4 *>(p);
        uint4 b = *reinterpret_cast<const uint4 *>(p + 16);
        c.w[0] = a.x; c.w[1] = a.y; c.w[2] = a.z; c.w[3] = a.w;
        c.w[4] = b.x; c.w[5] = b.y; c.w[6] = b.z; c.w[7] = b.w;
    } else if constexpr (M_SUB == 8) {
        uint4 a = *reinterpret_cast<const uint4 *>(p);
        c.w[0] = a.x; c.w[1] = a.y; c.w[2] = a.z; c.w[3] = a.w;
    } else if constexpr (M_SUB == 4) {
        uint2 a = *reinterpret_cast<const uint2 *>(p);
        c.w[0] = a.x; c.w[1] = a.y;
    } else if constexpr (M_SUB == 2) {
        c.w[0] = *reinterpret_cast<const uint32_t *>(p);
    } else {
        c.w[0] = *reinterpret_cast<const uint16_t *>(p);
    }
    return c;
}

template <int M_SUB>
__device__ __forceinline__ int code_at(const CodePair<M_SUB> &c, int token01, int j)
{
    int byte = token01 * M_SUB + j;
    return (c.w[byte >> 2] >> (8 * (byte & 3))) & 0xff;
}

template <int DV>
struct VTile {                       // 4 tokens x (DV/64) 16-byte pieces per lane
    uint4 r[DV / 64][4];
};

template <int M_SUB, int DV>
__global__ void __launch_bounds__(kThreads, 2) attend_stream_kernel(AttendArgs a)
{
    extern __shared__ __align__(16) float smem[];

    const int split = blockIdx.x;
    const int hgroups = (a.g + 3) >> 2;
    const int kvh = blockIdx.y / hgroups;
    const int hgrp = blockIdx.y % hgroups;
    const int b = blockIdx.z;
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int n = lane >> 2, q = lane & 3;
    const int heads_here = min(4, a.g - hgrp * 4);        // query heads this CTA serves
    const int hq0 = kvh * a.g + hgrp * 4;                 // first of them
    const int hl = n & 3;                                 // head this lane scores
    const int part = n >> 2;                              // 0: weight, 1: its fp16 remainder
    const bool head_ok = hl < heads_here;

    const int seq_len = (int)min((long long)(a.seq_lens ? a.seq_lens[b] : a.uniform_len), a.L_max);
    const long long chunk_lo = (long long)split * a.chunk;
    const long long chunk_hi = min((long long)seq_len, chunk_lo + a.chunk);

    const int table = M_SUB * a.K;                        // floats per head
    const int head_stride = table + kHeadPad;

    // ---- stage the tables of this head group ----
    if (chunk_lo < chunk_hi) {
        for (int h = 0; h < heads_here; ++h) {
            const float *src = a.lut + ((size_t)b * a.H_q + hq0 + h) * table;
            float *dst = smem + h * head_stride;
            if ((table & 3) == 0) {
                for (int i = tid; i < (table >> 2); i += kThreads)
                    reinterpret_cast<float4 *>(dst)[i] = reinterpret_cast<const float4 *>(src)[i];
            } else {
                for (int i = tid; i < table; i += kThreads) dst[i] = src[i];
            }
        }
    }
    __syncthreads();

    const size_t kv_row = (size_t)b * a.H_kv + kvh;
    const uint8_t *codes = a.codes + kv_row * a.L_max * M_SUB;
    const __half *vbase = a.v + kv_row * a.L_max * DV;
    const float *my_table = smem + hl * head_stride;
    float *scores_row =
        (a.scores_out && head_ok) ? a.scores_out + ((size_t)b * a.H_q + hq0 + hl) * a.L_max : nullptr;

    float acc[DV / 16][4];
#pragma unroll
    for (int i = 0; i < DV / 16; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
    float m_run = kNegBig, l_run = 0.f;

    // token offsets inside a tile: the two this lane scores, the four whose V it holds
    const int ts_off = 2 * q + 8 * part;
    const int tv_off[4] = {2 * q, 2 * q + 1, 2 * q + 8, 2 * q + 9};

    auto load_tile = [&](long long t0, VTile<DV> &vt, CodePair<M_SUB> &cp) {
        const bool full = t0 + kTile <= chunk_hi;
        if (full) {
            cp = load_code_pair<M_SUB>(codes + (t0 + ts_off) * M_SUB);
#pragma unroll
            for (int gI = 0; gI < DV / 64; ++gI)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    vt.r[gI][k] = ldg_stream16(vbase + (t0 + tv_off[k]) * DV + gI * 64 + n * 8);
        } else {
            // ragged tail: never read a token at or beyond chunk_hi
            if (t0 + ts_off + 1 < chunk_hi) {
                cp = load_code_pair<M_SUB>(codes + (t0 + ts_off) * M_SUB);
            } else {
#pragma unroll
                for (int i = 0; i < (2 * M_SUB + 3) / 4; ++i) cp.w[i] = 0;
                if (t0 + ts_off < chunk_hi) {
                    const uint8_t *p = codes + (t0 + ts_off) * M_SUB;
#pragma unroll
                    for (int j = 0; j < M_SUB; ++j) cp.w[j >> 2] |= (uint32_t)p[j] << (8 * (j & 3));
                }
            }
#pragma unroll
            for (int gI = 0; gI < DV / 64; ++gI)
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (t0 + tv_off[k] < chunk_hi)
                        vt.r[gI][k] = ldg_stream16(vbase + (t0 + tv_off[k]) * DV + gI * 64 + n * 8);
                    else
                        vt.r[gI][k] = make_uint4(0, 0, 0, 0);
                }
        }
    };

    auto process_tile = [&](long long t0, const VTile<DV> &vt, const CodePair<M_SUB> &cp) {
        // ---- lookup-and-sum for this lane's two (token, head) pairs ----
        float s0 = 0.f, s1 = 0.f;
        if (head_ok) {
#pragma unroll
            for (int j = 0; j < M_SUB; ++j) {
                s0 += my_table[j * a.K + code_at<M_SUB>(cp, 0, j)];
                s1 += my_table[j * a.K + code_at<M_SUB>(cp, 1, j)];
            }
        }
        const long long ts = t0 + ts_off;
        const bool ok0 = head_ok && ts < chunk_hi, ok1 = head_ok && ts + 1 < chunk_hi;
        if (scores_row) {
            if (ok0) scores_row[ts] = s0;
            if (ok1) scores_row[ts + 1] = s1;
        }
        const float x0 = ok0 ? s0 * a.scale_log2 : -INFINITY;
        const float x1 = ok1 ? s1 * a.scale_log2 : -INFINITY;

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
        const uint32_t b0 = pack_half2(weight_part(w0, part), weight_part(w1, part));
        const uint32_t b1 = pack_half2(weight_part(w2, part), weight_part(w3, part));

        // ---- O^T += V^T P on the tensor cores ----
#pragma unroll
        for (int gI = 0; gI < DV / 64; ++gI) {
            const uint32_t x[4] = {vt.r[gI][0].x, vt.r[gI][0].y, vt.r[gI][0].z, vt.r[gI][0].w};
            const uint32_t y[4] = {vt.r[gI][1].x, vt.r[gI][1].y, vt.r[gI][1].z, vt.r[gI][1].w};
            const uint32_t z[4] = {vt.r[gI][2].x, vt.r[gI][2].y, vt.r[gI][2].z, vt.r[gI][2].w};
            const uint32_t w[4] = {vt.r[gI][3].x, vt.r[gI][3].y, vt.r[gI][3].z, vt.r[gI][3].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t a0 = __byte_perm(x[i], y[i], 0x5410);   // dv even, tokens 2q,2q+1
                const uint32_t a1 = __byte_perm(x[i], y[i], 0x7632);   // dv odd
                const uint32_t a2 = __byte_perm(z[i], w[i], 0x5410);   // tokens 2q+8,2q+9
                const uint32_t a3 = __byte_perm(z[i], w[i], 0x7632);
                mma_16816(acc[gI * 4 + i], a0, a1, a2, a3, b0, b1);
            }
        }
    };

    // ---- walk this warp's tiles, loads one tile ahead ----
    const long long stride = (long long)kWarps * kTile;
    long long t0 = chunk_lo + (long long)warp * kTile;
    VTile<DV> vA, vB;
    CodePair<M_SUB> cA, cB;
    if (t0 < chunk_hi) load_tile(t0, vA, cA);
    while (t0 < chunk_hi) {
        const long long t1 = t0 + stride;
        if (t1 < chunk_hi) load_tile(t1, vB, cB);
        process_tile(t0, vA, cA);
        if (t1 >= chunk_hi) break;
        const long long t2 = t1 + stride;
        if (t2 < chunk_hi) load_tile(t2, vA, cA);
        process_tile(t1, vB, cB);
        t0 = t2;
    }

    // ---- fold the weight and remainder columns, reduce l over the head's lanes ----
#pragma unroll
    for (int i = 0; i < DV / 16; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[i][k] += __shfl_xor_sync(0xffffffffu, acc[i][k], 2);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);

    // ---- merge the 8 warps through shared memory (the tables are no longer needed) ----
    __syncthreads();
    float *w_o = smem;                                   // [kWarps][4][DV]
    float *w_m = smem + kWarps * 4 * DV;                 // [kWarps][4]
    float *w_l = w_m + kWarps * 4;                       // [kWarps][4]
    if (q < 2) {
#pragma unroll
        for (int i = 0; i < DV / 16; ++i) {
            const int dv = (i >> 2) * 64 + n * 8 + 2 * (i & 3);
            float *o = w_o + (warp * 4 + 2 * q) * DV + dv;
            o[0] = acc[i][0];          // (dv, head 2q)
            o[DV] = acc[i][1];         // (dv, head 2q+1)
            o[1] = acc[i][2];          // (dv+1, head 2q)
            o[DV + 1] = acc[i][3];     // (dv+1, head 2q+1)
        }
    }
    if (q == 0 && part == 0) {
        w_m[warp * 4 + hl] = m_run;
        w_l[warp * 4 + hl] = l_run;
    }
    __syncthreads();

    for (int idx = tid; idx < heads_here * DV; idx += kThreads) {
        const int h = idx / DV, dv = idx % DV;
        float M = kNegBig;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, w_m[w * 4 + h]);
        float o = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float f = ex2_approx(w_m[w * 4 + h] - M);
            o += f * w_o[(w * 4 + h) * DV + dv];
            l += f * w_l[w * 4 + h];
        }
        const size_t row = ((size_t)b * a.H_q + hq0 + h) * a.n_splits + split;
        a.part_o[row * DV + dv] = o;
        if (dv == 0) {
            a.part_ml[row * 2] = M;
            a.part_ml[row * 2 + 1] = l;
        }
    }
}

// Any shape.  One CTA per (chunk, query head, batch row); 128 threads.
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
            const uint8_t *c = codes + (blk + t) * a.m;
            float s = 0.f;
            for (int j = 0; j < a.m; ++j) s += __ldg(lut + j * a.K + c[j]);
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

// Merge of the chunk partials: M = max_i M_i, l = sum l_i 2^(M_i-M),
// o = sum o_i 2^(M_i-M) / l.  A chunk without tokens carries l = 0 and adds nothing.
__global__ void combine_kernel(AttendArgs a)
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

template <int M_SUB, int DV>
lookat_status launch_stream(Ctx *ctx, const AttendArgs &a)
{
    const int hgroups = (a.g + 3) / 4;
    const int heads = a.g < 4 ? a.g : 4;
    size_t lut_bytes = (size_t)heads * (M_SUB * a.K + kHeadPad) * sizeof(float);
    size_t merge_bytes = (size_t)(kWarps * 4 * DV + 2 * kWarps * 4) * sizeof(float);
    size_t smem = lut_bytes > merge_bytes ? lut_bytes : merge_bytes;
    auto kern = attend_stream_kernel<M_SUB, DV>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return check_launch(ctx, "attend: shared-memory opt-in");
    }
    dim3 grid(a.n_splits, a.H_kv * hgroups, a.B);
    kern<<<grid, kThreads, smem, ctx->stream>>>(a);
    return check_launch(ctx, "attend_stream_kernel");
}

template <int M_SUB>
lookat_status launch_stream_dv(Ctx *ctx, const AttendArgs &a)
{
    if (a.d_v == 64) return launch_stream<M_SUB, 64>(ctx, a);
    return launch_stream<M_SUB, 128>(ctx, a);
}

}  // namespace

bool attend_fast_path(const Ctx *ctx, const void *codes, const void *v, long long L_max)
{
    const lookat_config &c = ctx->cfg;
    const bool m_ok = c.m == 1 || c.m == 2 || c.m == 4 || c.m == 8 || c.m == 16;
    const bool dv_ok = c.d_v == 64 || c.d_v == 128;
    const int heads = c.n_q_heads / c.n_kv_heads < 4 ? c.n_q_heads / c.n_kv_heads : 4;
    const size_t lut_bytes = (size_t)heads * (c.m * c.K + kHeadPad) * sizeof(float);
    // rows of the code cache must start on a 16-byte boundary for the vector loads
    const bool rows_ok = (L_max * c.m) % 16 == 0 && ((uintptr_t)codes % 16) == 0 && ((uintptr_t)v % 16) == 0;
    return m_ok && dv_ok && rows_ok && lut_bytes <= (size_t)ctx->max_smem_optin;
}

int attend_auto_splits(const Ctx *ctx, int B, long long L_max)
{
    const lookat_config &c = ctx->cfg;
    const int g = c.n_q_heads / c.n_kv_heads;
    const long long units = (long long)B * c.n_kv_heads * ((g + 3) / 4);
    const long long resident = 2LL * ctx->sm_count;            // CTAs resident at once
    long long max_splits = L_max / 256;                         // keep chunks >= 256 tokens
    if (max_splits < 1) max_splits = 1;
    long long want = (8 * resident + units - 1) / units;        // about 8 waves of CTAs
    if (want < 1) want = 1;
    long long n = want < max_splits ? want : max_splits;
    // prefer a CTA count that is a whole number of waves
    for (long long cand = n; cand <= max_splits && cand <= n + 8; ++cand)
        if ((units * cand) % resident == 0) { n = cand; break; }
    if (n > 4096) n = 4096;
    return (int)n;
}

lookat_status launch_attend(Ctx *ctx, const AttendArgs &a)
{
    const bool fast = attend_fast_path(ctx, a.codes, a.v, a.L_max);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (ctx->timing) {
        const int s = ctx->ev_next;
        if (ctx->ev_used[s]) {
            float ms = 0.f;
            cudaEventSynchronize(ctx->ev1[s]);
            if (cudaEventElapsedTime(&ms, ctx->ev0[s], ctx->ev1[s]) == cudaSuccess) {
                ctx->timed_ms += ms;
                ctx->timed_n += 1;
            }
            ctx->ev_used[s] = 0;
        }
        e0 = ctx->ev0[s];
        e1 = ctx->ev1[s];
        cudaEventRecord(e0, ctx->stream);
    }
    lookat_status st;
    if (fast) {
        switch (a.m) {
            case 1: st = launch_stream_dv<1>(ctx, a); break;
            case 2: st = launch_stream_dv<2>(ctx, a); break;
            case 4: st = launch_stream_dv<4>(ctx, a); break;
            case 8: st = launch_stream_dv<8>(ctx, a); break;
            default: st = launch_stream_dv<16>(ctx, a); break;
        }
    } else {
        dim3 grid(a.n_splits, a.H_q, a.B);
        attend_generic_kernel<<<grid, kGenThreads, 0, ctx->stream>>>(a);
        st = check_launch(ctx, "attend_generic_kernel");
    }
    if (ctx->timing) {
        cudaEventRecord(e1, ctx->stream);
        ctx->ev_used[ctx->ev_next] = 1;
        ctx->ev_next = (ctx->ev_next + 1) % kTimingSlots;
    }
    return st;
}

lookat_status launch_combine(Ctx *ctx, const AttendArgs &a)
{
    int threads = a.d_v < 32 ? 32 : (a.d_v > 256 ? 256 : ((a.d_v + 31) / 32) * 32);
    combine_kernel<<<a.B * a.H_q, threads, 0, ctx->stream>>>(a);
    return check_launch(ctx, "combine_kernel");
}

}  // namespace lookat
