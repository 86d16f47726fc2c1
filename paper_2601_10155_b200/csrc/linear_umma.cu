// Linear layers of the GPT-2 decoder harness (Section 4.1 of the paper names the model; these products are not part of
// the paper's method, they are what surrounds its attention in BASELINE config 2):
//     out = act(x W + b) [+ residual],      W stored transposed, w_t [N][K] fp16 (K-major), x [M][K].
//
// linear_umma_kernel (prompt-sized M): one CTA per 128 x 128 output tile.  Both operands come K-major through 2-D
// tensor maps (TMA tiles of 128 rows x 64 halfs with the 128-byte swizzle the MMA descriptors expect; rows or columns
// beyond the matrix read as zeros), three stages of 32 KB, so two CTAs share an SM and one's epilogue overlaps the
// other's main loop.  One thread issues the copies, one thread issues tcgen05.mma (128 x 128 x 16, fp16 in, fp32
// accumulate in 128 columns of tensor memory) and commits each stage back to the copier; four warps read the
// accumulator with tcgen05.ld (thread r = row r of the tile) and apply bias, the tanh-form GELU, the residual and the
// output conversion, or scatter the q / k / v thirds of the fused projection into head-major buffers.
// Every mbarrier wait is bounded; a wait that runs out raises the context's time-out flag, the CTA drains, frees its
// tensor memory and returns.
//
// linear_skinny_kernel (M <= 32: one decode step of the whole batch): the product is bound by reading W once, and at
// these sizes by latency.  A CTA owns 8 or 32 output columns and a slice of K; its 4 warps stream rows of w_t over
// quarters of the slice with 16-byte loads straight into mma.sync.m16n8k16 B fragments (the k order inside a 32-wide
// block is permuted the same way for both operands, so no shuffle is needed); two 16-row tiles cover the batch; the
// quarters meet in shared memory, the slices in the shared memory of the first CTA of a thread-block cluster.
#include <cuda.h>           // CUtensorMap and its enums only; the driver entry point is looked up at run time

#include <cooperative_groups.h>

#include <cstring>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace lookat {

namespace {

constexpr int kLnBM = 128, kLnBN = 128, kLnBK = 64, kLnStages = 3;
constexpr int kLnTileBytes = kLnBM * kLnBK * 2;            // 16 KB per operand tile
constexpr int kLnStageBytes = 2 * kLnTileBytes;
constexpr int kLnThreads = 192;                             // warp 0: copies, warp 1: MMA, warps 2..5: epilogue
constexpr int kLnPolls = 1 << 20;                           // bound of every mbarrier wait
constexpr int kLnSmem = kLnStages * kLnStageBytes + 1024 /* alignment slack */ + 128 /* barriers */;

__device__ __forceinline__ uint32_t ln_smem(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ln_bar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool ln_bar_wait(uint32_t bar, uint32_t parity)
{
    for (int it = 0; it < kLnPolls; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void ln_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void ln_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D (tensor memory) = or += A . B, both operands in shared memory (64-bit descriptors)
__device__ __forceinline__ void ln_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void ln_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ln_ld32(uint32_t (&r)[32], uint32_t taddr)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}

// GPT-2's activation: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
__device__ __forceinline__ float gelu_tanh(float x)
{
    return 0.5f * x * (1.f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}

// 32 consecutive output columns [col0, col0+32) of row `row`, as fp32 in acc[]: bias, activation, residual, store.
// In the q/k/v form the columns are one half of a head's 64 dims of one of the three thirds.
__device__ __forceinline__ void linear_store32(const LinearArgs &p, long long row, int col0, float (&acc)[32])
{
    if (row >= p.M) return;
    const int ncol = min(32, p.N - col0);
    if (ncol <= 0) return;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        if (i < ncol) {
            float v = acc[i] + (p.bias ? __half2float(p.bias[col0 + i]) : 0.f);
            if (p.gelu) v = gelu_tanh(v);
            acc[i] = v;
        }
    }
    if (p.qkv) {
        const int d_model = p.N / 3;
        const int sel = col0 / d_model, c = col0 - sel * d_model, h = c >> 6, d0 = c & 63;
        const long long b = row / p.T, t = row - b * p.T;
        __half *dst = p.dst[sel] + (((size_t)b * p.n_head + h) * p.cap[sel] + p.off[sel] + t) * 64 + d0;
#pragma unroll
        for (int i = 0; i < 32; i += 8) {                      // d_model is a multiple of 64: whole 32-column pieces
            uint4 w;
            __half2 h0 = __floats2half2_rn(acc[i], acc[i + 1]), h1 = __floats2half2_rn(acc[i + 2], acc[i + 3]);
            __half2 h2 = __floats2half2_rn(acc[i + 4], acc[i + 5]), h3 = __floats2half2_rn(acc[i + 6], acc[i + 7]);
            w.x = *reinterpret_cast<uint32_t *>(&h0); w.y = *reinterpret_cast<uint32_t *>(&h1);
            w.z = *reinterpret_cast<uint32_t *>(&h2); w.w = *reinterpret_cast<uint32_t *>(&h3);
            *reinterpret_cast<uint4 *>(dst + i) = w;
        }
        return;
    }
    const size_t at = (size_t)row * p.N + col0;
    if (p.residual) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < ncol) acc[i] += p.residual[at + i];
    }
    if (ncol == 32 && (p.N & 7) == 0) {
        if (p.out_fp16) {
            __half *o = static_cast<__half *>(p.out) + at;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
                uint4 w;
                __half2 h0 = __floats2half2_rn(acc[i], acc[i + 1]), h1 = __floats2half2_rn(acc[i + 2], acc[i + 3]);
                __half2 h2 = __floats2half2_rn(acc[i + 4], acc[i + 5]), h3 = __floats2half2_rn(acc[i + 6], acc[i + 7]);
                w.x = *reinterpret_cast<uint32_t *>(&h0); w.y = *reinterpret_cast<uint32_t *>(&h1);
                w.z = *reinterpret_cast<uint32_t *>(&h2); w.w = *reinterpret_cast<uint32_t *>(&h3);
                *reinterpret_cast<uint4 *>(o + i) = w;
            }
        } else {
            float *o = static_cast<float *>(p.out) + at;
#pragma unroll
            for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4 *>(o + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (i < ncol) {
                if (p.out_fp16) static_cast<__half *>(p.out)[at + i] = __float2half_rn(acc[i]);
                else static_cast<float *>(p.out)[at + i] = acc[i];
            }
        }
    }
}

__global__ void __launch_bounds__(kLnThreads, 2)
linear_umma_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map, LinearArgs p)
{
    extern __shared__ unsigned char ln_raw[];
    const uint32_t raw0 = ln_smem(ln_raw);
    const uint32_t sm0 = (raw0 + 1023u) & ~1023u;               // operand tiles want 1024-byte alignment
    unsigned char *const sm = ln_raw + (sm0 - raw0);
    uint64_t *const bars = reinterpret_cast<uint64_t *>(sm + kLnStages * kLnStageBytes);
    uint32_t *const tmem_slot = reinterpret_cast<uint32_t *>(bars + 8);
    const uint32_t bar_full = ln_smem(bars), bar_empty = bar_full + 8 * kLnStages, bar_acc = bar_full + 16 * kLnStages;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile_n = blockIdx.x, tile_m = blockIdx.y;
    const int num_k = (p.K + kLnBK - 1) / kLnBK;

    if (tid == 0) {
        for (int s = 0; s < kLnStages; ++s) {
            ln_bar_init(bar_full + 8 * s, 1);                   // one arrival (the copier's expect_tx) plus the bytes
            ln_bar_init(bar_empty + 8 * s, 1);                  // one arrival: the commit of the stage's MMAs
        }
        ln_bar_init(bar_acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ln_smem(tmem_slot)), "n"(kLnBN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    ln_fence_before();
    __syncthreads();
    ln_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool dead = false;

    if (warp == 0) {
        if (lane == 0) {
            // =================== copies: stage s gets the x tile and the w tile of k-block kb ===================
            for (int kb = 0; kb < num_k; ++kb) {
                const int s = kb % kLnStages;
                if (kb >= kLnStages && !ln_bar_wait(bar_empty + 8 * s, ((kb / kLnStages) - 1) & 1)) { dead = true; break; }
                const uint32_t full = bar_full + 8 * s, dst = sm0 + s * kLnStageBytes;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full), "r"(kLnStageBytes) : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                    "l"(reinterpret_cast<uint64_t>(&x_map)), "r"(kb * kLnBK), "r"(tile_m * kLnBM), "r"(full)
                    : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                        dst + kLnTileBytes),
                    "l"(reinterpret_cast<uint64_t>(&w_map)), "r"(kb * kLnBK), "r"(tile_n * kLnBN), "r"(full)
                    : "memory");
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // =================== MMA: D[128 x 128] += X[128 x 16] . W^T[16 x 128], four per stage ===================
            // descriptors: K-major, 8-row groups 1024 bytes apart, version 1, 128-byte swizzle; the start address
            // (16-byte units) advances by 32 bytes per 16 halfs of k inside the swizzled row
            const uint64_t desc_hi = (uint64_t)((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
            const uint32_t idesc = (1u << 4) | ((uint32_t)(kLnBN >> 3) << 17) | ((uint32_t)(kLnBM >> 4) << 24);
            for (int kb = 0; kb < num_k; ++kb) {
                const int s = kb % kLnStages;
                if (!ln_bar_wait(bar_full + 8 * s, (kb / kLnStages) & 1)) { dead = true; break; }
                ln_fence_after();
                const uint32_t a_lo = ((sm0 + s * kLnStageBytes) >> 4) | (1u << 16);
                const uint32_t b_lo = ((sm0 + s * kLnStageBytes + kLnTileBytes) >> 4) | (1u << 16);
#pragma unroll
                for (int ks = 0; ks < kLnBK / 16; ++ks)
                    ln_mma_ss(tmem, desc_hi | (a_lo + ks * 2), desc_hi | (b_lo + ks * 2), idesc, (kb | ks) != 0 ? 1u : 0u);
                ln_commit(bar_empty + 8 * s);                   // the stage is free once these MMAs have read it
            }
            if (!dead) ln_commit(bar_acc);                      // ... and the tile is complete once all of them are done
        }
    } else {
        // =================== epilogue: thread r of the four warps = row r of the tile = tensor-memory lane r ===================
        const int quarter = warp & 3;                           // a warp may read the 32 lanes of its own quarter
        if (!ln_bar_wait(bar_acc, 0)) dead = true;
        dead = __any_sync(0xffffffffu, dead);
        if (!dead) {
            ln_fence_after();
            const long long row = (long long)tile_m * kLnBM + quarter * 32 + lane;
#pragma unroll 1
            for (int part = 0; part < kLnBN / 32; ++part) {
                uint32_t r[32];
                ln_ld32(r, tmem + ((uint32_t)(quarter * 32) << 16) + part * 32);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                float acc[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[i] = __uint_as_float(r[i]);
                linear_store32(p, row, tile_n * kLnBN + part * 32, acc);
            }
        }
    }
    if (dead && p.timeout_flag) atomicExch(p.timeout_flag, 1);
    ln_fence_before();
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kLnBN) : "memory");
}

// ---------------------------------------------------------------------------------------------------------------
// One decode step's products: M <= 32 rows, bound by reading w_t once, and small enough that latency decides: what
// counts is how many 16-byte loads are in flight over the whole GPU.  A CTA of 4 warps owns 8 NT output columns and one
// slice of K (about 384 wide); a thread-block cluster of up to 8 CTAs covers K.  Warp w takes a quarter of the slice --
// three 32-wide k-blocks, unrolled, so all its loads are requested before the first MMA -- the quarters meet in shared
// memory, and the slices meet in the shared memory of the cluster's first CTA (read through distributed shared
// memory), which applies bias, activation and residual and stores.  x is read from global memory as it is needed (at
// most 192 KB, resident in L2); NT = 4 for wide outputs, where re-reading x per 8 columns would cost more than w_t.
constexpr int kSkThreads = 128, kSkWarps = 4, kSkSlice = 384, kSkMaxCluster = 8;

__device__ __forceinline__ void sk_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 8 consecutive elements of x row `r` from column k as four packed half pairs (zeros for rows >= M)
template <bool X_FP32>
__device__ __forceinline__ uint4 sk_x8(const void *x, int r, int M, int K, int k)
{
    if (r >= M) return make_uint4(0u, 0u, 0u, 0u);
    if (X_FP32) {
        const float4 *src = reinterpret_cast<const float4 *>(static_cast<const float *>(x) + (size_t)r * K + k);
        const float4 f0 = src[0], f1 = src[1];
        __half2 h0 = __floats2half2_rn(f0.x, f0.y), h1 = __floats2half2_rn(f0.z, f0.w);
        __half2 h2 = __floats2half2_rn(f1.x, f1.y), h3 = __floats2half2_rn(f1.z, f1.w);
        return make_uint4(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1), *reinterpret_cast<uint32_t *>(&h2),
                          *reinterpret_cast<uint32_t *>(&h3));
    }
    return *reinterpret_cast<const uint4 *>(static_cast<const __half *>(x) + (size_t)r * K + k);
}

// grid (column groups, K slices); the CTAs of one column group form a cluster (gridDim.y of them)
template <bool X_FP32, int NT>
__global__ void __launch_bounds__(kSkThreads) linear_skinny_kernel(const void *__restrict__ x, const __half *__restrict__ w_t, LinearArgs p,
                                                                   int slice)
{
    constexpr int kVals = NT * 2 * 4 * 32;                      // partial sums of a CTA: [n-tile][row tile][accumulator][lane]
    __shared__ float part[kSkWarps][kVals];
    __shared__ float mine[kVals];                               // this CTA's slice, summed over its warps
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int n0 = blockIdx.x * (8 * NT);
    const int M = (int)p.M, K = p.K;
    // this warp's share of the CTA's slice: whole 32-wide blocks
    const int per = ((slice >> 5) + kSkWarps - 1) / kSkWarps;
    const int k_end = min(K, ((int)blockIdx.y + 1) * slice);
    const int k_lo = min(k_end, (int)blockIdx.y * slice + warp * per * 32), k_hi = min(k_end, k_lo + per * 32);
    float acc[NT][2][4] = {};
    // lane (g, t) streams row n0 + 8 nt + g of w_t, 8 halfs at k = kk + 8 t of every 32-wide block (columns beyond N read row N - 1).
    // Inside such a block the MMA's k index is a relabelling of the true one: the lane with t supplies true k = 8 t .. 8 t + 7
    // -- (8t, 8t+1 | 8t+2, 8t+3) to the first MMA, (8t+4, 8t+5 | 8t+6, 8t+7) to the second -- for both operands alike.
    const __half *wrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) wrow[nt] = w_t + (size_t)min(n0 + nt * 8 + g, p.N - 1) * K;
#pragma unroll 3
    for (int kk = k_lo; kk < k_hi; kk += 32) {
        const int k = kk + 8 * t;
        uint4 wv[NT], xa[2][2];
        const bool in = k < K;                                  // K is a multiple of 8
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) wv[nt] = in ? __ldg(reinterpret_cast<const uint4 *>(wrow[nt] + k)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            xa[mt][0] = in ? sk_x8<X_FP32>(x, mt * 16 + g, M, K, k) : make_uint4(0u, 0u, 0u, 0u);
            xa[mt][1] = in ? sk_x8<X_FP32>(x, mt * 16 + g + 8, M, K, k) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                sk_mma(acc[nt][mt], xa[mt][0].x, xa[mt][1].x, xa[mt][0].y, xa[mt][1].y, wv[nt].x, wv[nt].y);
                sk_mma(acc[nt][mt], xa[mt][0].z, xa[mt][1].z, xa[mt][0].w, xa[mt][1].w, wv[nt].z, wv[nt].w);
            }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) part[warp][((nt * 2 + mt) * 4 + i) * 32 + lane] = acc[nt][mt][i];
    __syncthreads();
    for (int e = tid; e < kVals; e += kSkThreads) mine[e] = part[0][e] + part[1][e] + part[2][e] + part[3][e];
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();                                             // every slice of the column group is summed and visible
    if (blockIdx.y == 0) {
        const unsigned n_slices = gridDim.y;
        // value e: n-tile e >> 8, row tile (e >> 7) & 1, accumulator (e >> 5) & 3 of lane e & 31:
        // row mt * 16 + g + 8 * (i >> 1), column n0 + 8 nt + 2 t + (i & 1)
        for (int e = tid; e < kVals; e += kSkThreads) {
            const int ln = e & 31, i = (e >> 5) & 3, mt = (e >> 7) & 1, nt = e >> 8;
            const int row = mt * 16 + (ln >> 2) + 8 * (i >> 1), col = n0 + nt * 8 + 2 * (ln & 3) + (i & 1);
            float v = mine[e];
            for (unsigned r = 1; r < n_slices; ++r) v += cluster.map_shared_rank(mine, r)[e];
            if (row >= M || col >= p.N) continue;
            v += p.bias ? __half2float(p.bias[col]) : 0.f;
            if (p.gelu) v = gelu_tanh(v);
            if (p.qkv) {
                const int d_model = p.N / 3;
                const int sel = col / d_model, c = col - sel * d_model, h = c >> 6, d = c & 63;
                const int b = row / p.T, tt = row - b * p.T;
                p.dst[sel][(((size_t)b * p.n_head + h) * p.cap[sel] + p.off[sel] + tt) * 64 + d] = __float2half_rn(v);
            } else {
                const size_t at = (size_t)row * p.N + col;
                if (p.residual) v += p.residual[at];
                if (p.out_fp16) static_cast<__half *>(p.out)[at] = __float2half_rn(v);
                else static_cast<float *>(p.out)[at] = v;
            }
        }
    }
    cluster.sync();                                             // the other CTAs' shared memory stays until it has been read
}

typedef CUresult (*tensor_map_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                         const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                         CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

tensor_map_encode_fn tensor_map_encoder()
{
    static tensor_map_encode_fn encode = nullptr;
    static bool looked = false;
    if (!looked) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            encode = reinterpret_cast<tensor_map_encode_fn>(fn);
        else
            cudaGetLastError();
        looked = true;
    }
    return encode;
}

// [rows][K] fp16, row-major: tiles of 128 rows x 64 halfs, 128-byte swizzle, zeros outside
bool make_operand_map(CUtensorMap *map, const void *base, long long rows, int K)
{
    tensor_map_encode_fn encode = tensor_map_encoder();
    if (!encode) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kLnBK, (cuuint32_t)kLnBM}, estr[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tile_maps_available() { return tensor_map_encoder() != nullptr; }

bool make_tile_map_f16(void *map, const void *base, unsigned long long inner, unsigned long long rows, unsigned box_inner,
                       unsigned box_rows)
{
    tensor_map_encode_fn encode = tensor_map_encoder();
    if (!encode) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows}, estr[2] = {1, 1};
    return encode(static_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

lookat_status launch_linear(Ctx *ctx, const void *x, int x_fp32, const __half *w_t, LinearArgs p)
{
    p.timeout_flag = ctx->timeout_flag;
    if (p.M <= 32) {
        // K in slices of about kSkSlice, at most kSkMaxCluster of them (one cluster per column group), whole 32-wide blocks
        int slices = (p.K + kSkSlice - 1) / kSkSlice;
        if (slices > kSkMaxCluster) slices = kSkMaxCluster;
        if (slices < 1) slices = 1;
        const int slice = ((p.K + slices - 1) / slices + 31) / 32 * 32;
        slices = (p.K + slice - 1) / slice;
        // 32 columns per CTA where that still fills the GPU twice over, else 8
        const bool wide = (long long)((p.N + 31) / 32) * slices >= 2ll * ctx->sm_count;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)((p.N + (wide ? 31 : 7)) / (wide ? 32 : 8)), (unsigned)slices, 1);
        cfg.blockDim = dim3(kSkThreads, 1, 1);
        cfg.stream = ctx->stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 1;
        attr.val.clusterDim.y = (unsigned)slices;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        cudaError_t err;
        if (wide)
            err = x_fp32 ? cudaLaunchKernelEx(&cfg, linear_skinny_kernel<true, 4>, x, w_t, p, slice)
                         : cudaLaunchKernelEx(&cfg, linear_skinny_kernel<false, 4>, x, w_t, p, slice);
        else
            err = x_fp32 ? cudaLaunchKernelEx(&cfg, linear_skinny_kernel<true, 1>, x, w_t, p, slice)
                         : cudaLaunchKernelEx(&cfg, linear_skinny_kernel<false, 1>, x, w_t, p, slice);
        if (err != cudaSuccess) return check_launch(ctx, "linear_skinny_kernel (cluster launch)");
        return check_launch(ctx, "linear_skinny_kernel");
    }
    if (x_fp32) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "linear: fp32 input is taken for M <= 32 only");
    if (ctx->timeout_flag && *(volatile int *)ctx->timeout_flag) {
        *(volatile int *)ctx->timeout_flag = 0;
        return set_error(ctx, LOOKAT_ERR_TIMEOUT, "an earlier kernel gave up a bounded barrier wait; its output is not valid");
    }
    CUtensorMap x_map, w_map;
    if (!make_operand_map(&x_map, x, p.M, p.K) || !make_operand_map(&w_map, w_t, p.N, p.K))
        return set_error(ctx, LOOKAT_ERR_CUDA, "linear: cuTensorMapEncodeTiled is not available or rejected the operands");
    if (cudaFuncSetAttribute(linear_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLnSmem) != cudaSuccess)
        return check_launch(ctx, "linear: shared-memory opt-in");
    dim3 grid((unsigned)((p.N + kLnBN - 1) / kLnBN), (unsigned)((p.M + kLnBM - 1) / kLnBM));
    linear_umma_kernel<<<grid, kLnThreads, kLnSmem, ctx->stream>>>(x_map, w_map, p);
    return check_launch(ctx, "linear_umma_kernel");
}

}  // namespace lookat
