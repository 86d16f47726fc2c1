// Pieces shared by the streaming attend kernels (attend.cu, attend_multi.cu): tile geometry, the
// asynchronous-copy and tensor-core instructions they issue, and the packed codes of a token pair.
#pragma once

#include "common.cuh"

namespace lookat {
namespace {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kTile = 16;           // tokens per warp step (the MMA's k extent)
constexpr int kHeadPad = 8;         // floats between the table sets of two heads (bank shift)
constexpr int kTableStride = 256;   // shared-memory entries per subspace table (codes are bytes)
constexpr float kNegBig = -1.0e30f; // running-max start: finite, so differences never give NaN
constexpr int kMaxRoundUnits = 8;   // attend_multi_kernel: units whose tables are resident together

__host__ __device__ inline MultiLayout multi_layout(int m, int d_v, int d_k, int K, int g, int ut, int stage_book,
                                                    int stages)
{
    MultiLayout l;
    const int heads_max = g < 4 ? g : 4;
    const int qh = stage_book ? (g == 1 ? 1 : (g == 2 ? 2 : 4)) : 4;
    l.set_floats = heads_max * (m * kTableStride + kHeadPad);
    int off = 0;
    l.tables = off;
    off += ut * l.set_floats * 4;
    off = (off + 15) & ~15;
    l.partials = off;
    off += ut * kWarps * heads_max * (d_v + 2) * 4;
    off = (off + 15) & ~15;
    l.q = off;
    off += ut * d_k * qh * 8;
    off = (off + 15) & ~15;
    l.xk = off;
    off += ut * d_k * 4;
    off = (off + 15) & ~15;
    l.newc = off;
    off += ut * 16;
    l.book = off;
    off += stage_book ? K * d_k * 4 : 0;
    off = (off + 15) & ~15;
    l.ring = off;
    off += kWarps * stages * (kTile * (d_v * 2 + 16) + kTile * m);
    l.total = off;
    return l;
}

__device__ __forceinline__ void cp_async16(unsigned smem_dst, const void *gmem_src)
{
    asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
// Four 8x8 fp16 matrices, transposed on the way: lane l gives the address of one 16-byte matrix row.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], unsigned smem_src)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
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

// Two weights as packed fp16: their roundings (part 0) or what the roundings left over (part 1).
__device__ __forceinline__ uint32_t weight_pair(float w0, float w1, int part)
{
    const __half2 h = __floats2half2_rn(w0, w1);
    const float2 f = __half22float2(h);
    const __half2 r = __floats2half2_rn(w0 - f.x, w1 - f.y);
    const __half2 out = part ? r : h;
    return *reinterpret_cast<const uint32_t *>(&out);
}

template <int M_SUB>
struct CodePair {                    // the codes of two consecutive tokens
    uint32_t w[(2 * M_SUB + 3) / 4];
};

template <int M_SUB>
__device__ __forceinline__ CodePair<M_SUB> read_code_pair(const unsigned char *p)
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

// the same from a shared-memory address (32-bit), so that no generic pointer to the slot has to stay live
template <int M_SUB>
__device__ __forceinline__ CodePair<M_SUB> read_code_pair_s(unsigned p)
{
    CodePair<M_SUB> c;
    if constexpr (M_SUB == 16) {
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(c.w[0]), "=r"(c.w[1]), "=r"(c.w[2]), "=r"(c.w[3]) : "r"(p));
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(c.w[4]), "=r"(c.w[5]), "=r"(c.w[6]), "=r"(c.w[7]) : "r"(p + 16));
    } else if constexpr (M_SUB == 8) {
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(c.w[0]), "=r"(c.w[1]), "=r"(c.w[2]), "=r"(c.w[3]) : "r"(p));
    } else if constexpr (M_SUB == 4) {
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(c.w[0]), "=r"(c.w[1]) : "r"(p));
    } else if constexpr (M_SUB == 2) {
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(c.w[0]) : "r"(p));
    } else {
        unsigned short v;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(p));
        c.w[0] = v;
    }
    return c;
}

template <int M_SUB>
__device__ __forceinline__ int code_at(const CodePair<M_SUB> &c, int token01, int j)
{
    const int byte = token01 * M_SUB + j;
    return (int)__byte_perm(c.w[byte >> 2], 0u, 0x4440u | (unsigned)(byte & 3));
}

// The table entries of one unit, out of line: its registers are its own, so the next entry's centroid can be
// requested ahead without touching the allocation of the streaming loop.  With xk (a key of d_k floats in shared
// memory) the fp32 squared distance of every centroid to its sub-vector of the key goes to dist[j * kTableStride + c],
// formed as the warp search of encode_warp.cuh forms it: the append's search rides on the centroids read here.
template <bool DIST>
__device__ __noinline__ void build_unit_tables(const float *book, const double *q_s, float *lut_s, int table, int K,
                                               int d_sub, int heads_here, int head_stride, int tid, const float *xk, float *dist)
{
    const bool vec16 = d_sub == 16;
    float4 pre[4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
        pre[u] = (vec16 && tid < table) ? __ldg(reinterpret_cast<const float4 *>(book + (size_t)tid * 16) + u) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int e = tid; e < table; e += kThreads) {
        const float *cen = book + (size_t)e * d_sub;
        const int j = e / K;
        const int es = j * kTableStride + (e - j * K);
        const double *qj = q_s + 4 * j * d_sub;
        double t0 = 0.0, t1 = 0.0, t2 = 0.0, t3 = 0.0;
        float dacc = 0.f;
        const float *xj = DIST ? xk + j * d_sub : nullptr;
        auto step = [&](int i, float cf) {
            if constexpr (DIST) {
                const float t = xj[i] - cf;
                dacc = fmaf(t, t, dacc);
            }
            const double cv = (double)cf;
            const double2 q01 = *reinterpret_cast<const double2 *>(qj + 4 * i);
            const double2 q23 = *reinterpret_cast<const double2 *>(qj + 4 * i + 2);
            t0 = fma(q01.x, cv, t0), t1 = fma(q01.y, cv, t1);
            t2 = fma(q23.x, cv, t2), t3 = fma(q23.y, cv, t3);
        };
        if (vec16) {
            float4 nxt[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                nxt[u] = e + kThreads < table ? __ldg(reinterpret_cast<const float4 *>(cen + (size_t)kThreads * 16) + u) : pre[u];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                step(4 * u, pre[u].x); step(4 * u + 1, pre[u].y); step(4 * u + 2, pre[u].z); step(4 * u + 3, pre[u].w);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) pre[u] = nxt[u];
        } else if ((d_sub & 3) == 0) {
            for (int i = 0; i < d_sub; i += 4) {
                const float4 c4 = __ldg(reinterpret_cast<const float4 *>(cen + i));
                step(i, c4.x); step(i + 1, c4.y); step(i + 2, c4.z); step(i + 3, c4.w);
            }
        } else {
            for (int i = 0; i < d_sub; ++i) step(i, __ldg(cen + i));
        }
        lut_s[es] = (float)t0;
        if (heads_here > 1) lut_s[head_stride + es] = (float)t1;
        if (heads_here > 2) lut_s[2 * head_stride + es] = (float)t2;
        if (heads_here > 3) lut_s[3 * head_stride + es] = (float)t3;
        if constexpr (DIST) dist[es] = dacc;
    }
}

}  // namespace
}  // namespace lookat
