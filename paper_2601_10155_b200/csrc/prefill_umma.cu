// Multi-query causal attention over the compressed keys, contraction form, on the 5th-generation tensor
// cores (Algorithm 1 applied to two tiles of 128 queries at a time).  The score of Section 3.4,
//     s[q][t] = sum_j LUT_j[code[t][j]],   LUT_j[c] = q^(j) . C_j[c],
// is the inner product of q with the key rebuilt from its codes, k^[t] = (C_1[code[t][1]], ...,
// C_m[code[t][m]]).  A table pays when one query meets many keys; in prefill many queries meet each key,
// so the centroids named by a chunk of 64 tokens are gathered ONCE per CTA into shared memory (the codes
// stay the only stored form of the keys; nothing is written back to HBM) and all 256 queries take their
// scores from them with tcgen05.mma: S = Q . K^^T (fp32 in tensor memory), online softmax by one thread
// per query row, O += P . V with P read from tensor memory.  q (fp16) is an exact operand; every fp32
// centroid is split into two fp16 planes (rounding + remainder), which carries s to ~2^-22 relative.
//
// A CTA works on two tiles of 128 queries against the same chunks, one behind the other: while the softmax
// threads of one tile work, the tensor pipe runs the other tile's MMAs, and every rebuilt chunk serves 256 queries.
// The two tiles are consecutive row tiles of one query head, or (grouped heads) the same rows of two query heads
// that share the KV head.
// Roles in a CTA of 15 warps (one CTA per SM; the shared memory is full):
//   warps 0-3 / 4-7  softmax of tile 0 / tile 1: thread r owns query row r of its tile = tensor-memory lane r;
//   warps 8-11  key producers: rebuild the next chunk's key rows from the codebook image in shared memory
//               (16-byte items placed so that gathers and stores are free of bank conflicts whatever the codes are);
//   warps 12-13 fetch the V rows of the chunk after next, on their own schedule: whole chunks by TMA (tiled bulk
//               copies with the 128-byte swizzle of the MMA operand), the last partial chunk by cp.async;
//   warp 14     one thread issues every MMA and commits them to mbarriers.
// Tensor memory (512 columns): per tile the scores of one chunk (64; the fp16 weights overwrite their first
// half), O (d_v) and the query rows as the A operand of the score MMA (d_k / 2).
// Hand-offs go through mbarriers, one per buffer where a buffer is reused, so that no waiter can fall two
// phases behind; every wait gives up after a bounded number of polls, raises the context's timeout flag and
// lets the CTA drain and free its tensor memory.
#include <cuda.h>           // CUtensorMap and its enums only; the driver entry point is looked up at run time

#include <type_traits>

#include "common.cuh"

namespace lookat {

namespace {

constexpr int kUmRows = 128;                   // queries per tile = rows of one MMA
constexpr int kUmChunk = 64;                   // tokens per chunk = columns of the score MMA
constexpr int kUmTiles = 2;                    // query tiles per CTA
constexpr int kUmSoftmax = kUmTiles * kUmRows, kUmProducers = 128, kUmVLoaders = 64;
constexpr int kUmThreads = kUmSoftmax + kUmProducers + kUmVLoaders + 32;
constexpr float kUmSlack = 8.f;                // how far a row maximum may run ahead of the softmax reference point
constexpr int kUmPolls = 1 << 20;              // bound of every mbarrier wait

__device__ __forceinline__ uint32_t um_smem(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void um_bar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void um_bar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// false after `polls` unsuccessful polls
__device__ __forceinline__ bool um_bar_wait(uint32_t bar, uint32_t parity, int polls = kUmPolls)
{
    for (int it = 0; it < polls; ++it) {
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
// one poll that never suspends the thread (try_wait may park it for a while, which would starve the other condition
// the MMA thread is watching)
__device__ __forceinline__ bool um_bar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    return ok != 0;
}
// One thread polls, the named barrier hands its verdict to the whole group (key producers: barrier 1, V loaders:
// barrier 2): nobody leaves a loop alone.
template <int BARRIER, int THREADS>
__device__ __forceinline__ bool um_group_wait(bool poller, uint32_t bar, uint32_t parity)
{
    const uint32_t failed = poller ? (um_bar_wait(bar, parity) ? 0u : 1u) : 0u;
    uint32_t any;
    asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 p, %1, 0;\nbar.red.or.pred q, %2, %3, p;\nselp.u32 %0, 1, 0, q;\n}"
                 : "=r"(any)
                 : "r"(failed), "n"(BARRIER), "n"(THREADS)
                 : "memory");
    return any == 0;
}
__device__ __forceinline__ void um_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void um_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void um_fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// D (tensor memory) = or += A (tensor memory) . B (shared memory, descriptor given as its two words)
template <bool ACCUMULATE>
__device__ __forceinline__ void um_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc)
{
    asm volatile(
        "{\n.reg .pred p;\n.reg .b64 bd;\nsetp.ne.b32 p, %5, 0;\nmov.b64 bd, {%2, %3};\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "n"(ACCUMULATE ? 1 : 0)
        : "memory");
}
__device__ __forceinline__ void um_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void um_cp_async16(unsigned dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// 32 consecutive 32-bit columns of this thread's tensor-memory lane; the registers are valid after um_wait_ld()
__device__ __forceinline__ void um_ld32(uint32_t (&r)[32], uint32_t taddr)
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
__device__ __forceinline__ void um_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void um_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(
            taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
        "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void um_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory image of one head's codebooks as two fp16 planes, hi = fp16(c), lo = fp16(c - hi):
// halfs [plane][d_k/64][K][8 pieces][8]: the 16-byte piece of 8-dim group gi sits in bank group gi mod 8.
__global__ void um_codebook_image_kernel(const float *__restrict__ books, __half *__restrict__ images, int H_kv, int m, int K,
                                         int d_sub)
{
    const int d_k = m * d_sub;
    const size_t n = (size_t)H_kv * K * d_k;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % d_sub), c = (int)(i / d_sub % K), j = (int)(i / ((size_t)d_sub * K) % m);
        const int h = (int)(i / ((size_t)d_sub * K * m));
        const int dim = j * d_sub + e, gi = dim >> 3, blocks = d_k / 64;
        const float v = books[i];
        const __half hi = __float2half_rn(v), lo = __float2half_rn(v - __half2float(hi));
        __half *img = images + (size_t)h * K * d_k * 2;
        const size_t at = (((size_t)(gi >> 3) * K + c) * 8 + (gi & 7)) * 8 + (dim & 7);
        img[at] = hi;
        img[at + (size_t)blocks * K * 64] = lo;
    }
}

template <int D_K, int D_V>
struct UmLayout {
    static constexpr int kKb = D_K / 64, kNb = D_V / 64;               // 128-byte blocks per key row / V row
    static constexpr int kKeys = kKb * 2 * kUmChunk * 128;             // [kb][64 hi rows, 64 lo rows][128 B]
    static constexpr int kV = kNb * kUmChunk * 128;                    // [nb][64 tokens][128 B]
    static constexpr int kOffKeys = 0, kOffV = 2 * kKeys, kOffBook = kOffV + 2 * kV;   // two key buffers, two V buffers
    static constexpr int kIds = D_K / 4;                               // 16-byte items per key row, both planes
    static constexpr int kItems = kUmChunk * kIds / kUmProducers;      // items rebuilt per producer thread per chunk
    static_assert(kUmChunk * kIds % kUmProducers == 0, "whole items per thread");
    static size_t book_bytes(int K) { return (size_t)K * D_K * 4; }
    // operands, codebook image, then barriers (256 B) and the codes of two chunks (2 KB)
    static size_t bytes(int K) { return (size_t)kOffBook + book_bytes(K) + 256 + 2048; }
    // tensor-memory columns: S of tile 0, 1 (64 each; P over their first halves) | O of tile 0, 1 | Q of tile 0, 1
    static constexpr int kColO = kUmTiles * kUmChunk, kColQ = kColO + kUmTiles * D_V;
    static constexpr int kTmemCols = kColQ + kUmTiles * (D_K / 2) <= 256 ? 256 : 512;
    static_assert(kColQ + kUmTiles * (D_K / 2) <= 512, "tensor memory");
    // instruction descriptors: fp32 accumulate, fp16 operands, N >> 3 at bit 17, M >> 4 at bit 24; bit 16: B is MN-major
    static constexpr uint32_t kIdescS = (1u << 4) | ((uint32_t)(kUmChunk >> 3) << 17) | ((uint32_t)(kUmRows >> 4) << 24);
    static constexpr uint32_t kIdescO = (1u << 4) | (1u << 16) | ((uint32_t)(D_V >> 3) << 17) | ((uint32_t)(kUmRows >> 4) << 24);
};

template <int D_K, int D_V, bool SCORES>
__global__ void __launch_bounds__(kUmThreads, 1)
attend_prefill_umma_kernel(PrefillArgs a, const __half *__restrict__ images, int *__restrict__ timeout_flag,
                           const __grid_constant__ CUtensorMap v_map, int use_tma, int pair_heads)
{
    using Lay = UmLayout<D_K, D_V>;
    extern __shared__ __align__(1024) unsigned char um_raw[];
    unsigned char *const sm = um_raw;                          // operands want 1024-byte alignment (checked below)
    const uint32_t sm0 = um_smem(sm);
    const uint32_t book_bytes = (uint32_t)a.K * D_K * 4;
    unsigned char *const book = sm + Lay::kOffBook;
    uint64_t *const bars = reinterpret_cast<uint64_t *>(book + book_bytes);
    uint32_t *const tmem_slot = reinterpret_cast<uint32_t *>(bars + 30);
    uint8_t *const codes_s = reinterpret_cast<uint8_t *>(bars + 32);  // [2][1024]: the codes of two chunks
    // barriers: k_ready[buf], v_ready[buf] (keys / V of a chunk staged); per tile s_full[t][buf] (scores done),
    // pv_done[t][buf] (value MMA done), p_ready[t] (weights stored)
    const uint32_t bar0 = um_smem(bars);
    const uint32_t bar_k = bar0, bar_v = bar0 + 16, bar_s = bar0 + 32, bar_pv = bar0 + 64, bar_p = bar0 + 96;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The two tiles of a CTA are two query heads of one KV head over the same 128 rows where heads come in groups
    // (pair_heads: same keys, same causal limits), else two consecutive tiles of 128 rows of one head.
    const int rows_per_cta = pair_heads ? kUmRows : kUmTiles * kUmRows;
    const int n_super = (int)((a.L_q + rows_per_cta - 1) / rows_per_cta);
    const int super = n_super - 1 - (int)blockIdx.x;           // longest first
    const int hq_first = pair_heads ? 2 * (int)blockIdx.y : (int)blockIdx.y, b = blockIdx.z, h = hq_first / a.g;
    const int d_sub = D_K / a.m;

    const long long row0 = (long long)super * rows_per_cta;
    const long long t_end = a.q_pos0 + (row0 + rows_per_cta < a.L_q ? row0 + rows_per_cta : a.L_q);   // tokens the CTA sees
    const int n_chunks = (int)((t_end + kUmChunk - 1) / kUmChunk);     // both tiles walk all of them (row tiles: tile 0 has up to two all masked)

    // ---- prologue, all threads: codebook image into shared memory, barriers, tensor memory ----
    {
        const unsigned char *img = reinterpret_cast<const unsigned char *>(images) + (size_t)h * book_bytes;
        for (uint32_t i = tid * 16; i < book_bytes; i += kUmThreads * 16) um_cp_async16(sm0 + Lay::kOffBook + i, img + i);
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (tid == 0) {
            for (int i = 0; i < 2; ++i) {
                um_bar_init(bar_k + 8 * i, kUmProducers);
                um_bar_init(bar_v + 8 * i, 1);                 // one arrival: the thread that issued the copies
                for (int t = 0; t < kUmTiles; ++t) {
                    um_bar_init(bar_s + 16 * t + 8 * i, 1);
                    um_bar_init(bar_pv + 16 * t + 8 * i, 1);
                }
                um_bar_init(bar_p + 8 * i, kUmRows);           // i as the tile index here
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        if (warp == 0) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(um_smem(tmem_slot)),
                         "n"(Lay::kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        um_fence_async_smem();
        um_fence_before();
        __syncthreads();
        um_fence_after();
    }
    const uint32_t tmem = *tmem_slot;
    bool dead = (sm0 & 1023u) != 0;                            // a wait ran out (or the base is misaligned): leave, free, return

    // ---- the query rows go to tensor memory as the A operand of the score MMA: lane r = row r, two halfs per column ----
    if (warp < kUmSoftmax / 32) {                              // one thread per row of each tile
        const int t = warp >> 2, r = (warp & 3) * 32 + lane;
        const long long want = row0 + (pair_heads ? 0 : t * kUmRows) + r;
        const long long qr = want < a.L_q ? want : a.L_q - 1;  // rows beyond L_q repeat the last one
        const int hq = hq_first + (pair_heads ? t : 0);
        const uint4 *src = reinterpret_cast<const uint4 *>(a.q + ((size_t)(b * a.H_q + hq) * a.L_q + qr) * D_K);
#pragma unroll
        for (int part = 0; part < D_K / 64; ++part) {
            uint32_t w[32];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint4 x = src[part * 8 + i];
                w[4 * i] = x.x;
                w[4 * i + 1] = x.y;
                w[4 * i + 2] = x.z;
                w[4 * i + 3] = x.w;
            }
            um_st32(tmem + Lay::kColQ + t * (D_K / 2) + part * 32 + ((uint32_t)((warp & 3) * 32) << 16), w);
        }
        um_wait_st();
    }
    um_fence_before();
    __syncthreads();
    um_fence_after();

    if (dead) {
        // misaligned shared-memory base: nothing runs
    } else if (warp >= (kUmSoftmax + kUmProducers + kUmVLoaders) / 32) {
        // =================== the MMA thread ===================
        if (lane == 0) {
            // descriptors: stride 1024 B, version 1, 128-byte swizzle in the high word; the low word holds the start
            // address and the leading offset (16-byte units) and is all that changes from one MMA to the next
            const uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t keys_lo = ((sm0 + Lay::kOffKeys) >> 4) | (1u << 16);                    // leading offset unused (16 B)
            const uint32_t v_lo = ((sm0 + Lay::kOffV) >> 4) | ((uint32_t)(kUmChunk * 128 / 16) << 16);   // between 64-column blocks
            auto score_mma = [&](int t, int c) {               // S(t) = Q(t) . K^(c)^T: the hi plane, then the lo plane on top
                const int buf = c & 1;
                const uint32_t lo = keys_lo + buf * (Lay::kKeys >> 4), d = tmem + t * kUmChunk, q = tmem + Lay::kColQ + t * (D_K / 2);
#pragma unroll
                for (int plane = 0; plane < 2; ++plane)
#pragma unroll
                    for (int ks = 0; ks < D_K / 16; ++ks) {
                        const uint32_t off = ((ks >> 2) * (2 * kUmChunk * 128) + plane * (kUmChunk * 128) + (ks & 3) * 32) >> 4;
                        if (plane == 0 && ks == 0) um_mma_ts<false>(d, q + ks * 8, lo + off, desc_hi, Lay::kIdescS);
                        else um_mma_ts<true>(d, q + ks * 8, lo + off, desc_hi, Lay::kIdescS);
                    }
                um_commit(bar_s + 16 * t + 8 * buf);
            };
            auto value_mma = [&](int t, int c) {               // O(t) += P(t, c) . V(c), P read from the first half of S(t)
                const int buf = c & 1;
                const uint32_t lo = v_lo + buf * (Lay::kV >> 4), pa = tmem + t * kUmChunk, d = tmem + Lay::kColO + t * D_V;
#pragma unroll
                for (int kt = 0; kt < kUmChunk / 16; ++kt) {   // 16 tokens: 8 columns of weights, two 8-token groups of V
                    if (kt == 0 && c == 0) um_mma_ts<false>(d, pa + kt * 8, lo + kt * (2048 >> 4), desc_hi, Lay::kIdescO);
                    else um_mma_ts<true>(d, pa + kt * 8, lo + kt * (2048 >> 4), desc_hi, Lay::kIdescO);
                }
                um_commit(bar_pv + 16 * t + 8 * buf);
            };
            // Per tile strictly scores(c) -> [softmax] -> value(c) -> scores(c + 1) (the weights overwrite the scores);
            // the two tiles take turns, so the pipe has the other tile's MMAs while one tile's softmax runs.
            int next_qk[kUmTiles] = {0, 0}, next_pv[kUmTiles] = {0, 0};
            long long polls = 0;
            while (next_pv[0] < n_chunks || next_pv[1] < n_chunks) {
                bool progress = false;
#pragma unroll
                for (int t = 0; t < kUmTiles; ++t) {           // value MMAs first: they release a tile's next scores
                    const int cp = next_pv[t];
                    if (cp < next_qk[t] && um_bar_test(bar_p + 8 * t, cp & 1) && um_bar_test(bar_v + 8 * (cp & 1), (cp >> 1) & 1)) {
                        um_fence_after();
                        value_mma(t, cp);
                        next_pv[t] = cp + 1;
                        progress = true;
                    }
                    const int cq = next_qk[t];
                    if (cq < n_chunks && next_pv[t] == cq && um_bar_test(bar_k + 8 * (cq & 1), (cq >> 1) & 1)) {
                        um_fence_after();
                        score_mma(t, cq);
                        next_qk[t] = cq + 1;
                        progress = true;
                    }
                }
                if (progress) polls = 0;
                else if (++polls > kUmPolls) { dead = true; break; }
            }
        }
    } else if (warp >= kUmSoftmax / 32 && warp < (kUmSoftmax + kUmProducers) / 32) {
        // =================== key producers ===================
        const int ptid = tid - kUmSoftmax;
        const uint8_t *codes = a.codes + (size_t)(b * a.H_kv + h) * a.L_max * a.m;
        // item p = ptid + i * producers of a chunk: token p / kIds, id = p % kIds = plane * (D_K/8) + gi (fixed per thread)
        const int my_id = ptid % Lay::kIds, my_plane = my_id / (D_K / 8), my_gi = my_id % (D_K / 8);
        const int my_j = (my_gi * 8) / d_sub;                  // the (first) subspace of this thread's 8-dim group
        const bool pair = d_sub == 4;                          // ... which holds two sub-vectors when they have 4 dims
        const unsigned char *my_src = book + (uint32_t)my_plane * (book_bytes / 2) + (uint32_t)(my_gi >> 3) * a.K * 128 + ((my_gi & 7) << 4);
        unsigned char *my_dst = sm + Lay::kOffKeys + (my_gi >> 3) * (2 * kUmChunk * 128) + my_plane * (kUmChunk * 128);   // + buf * kKeys
        const int tl0 = ptid / Lay::kIds;                      // this thread's tokens of a chunk: tl0 + i * (producers / kIds)
        constexpr int kTokStep = kUmProducers / Lay::kIds;
        const int code_bytes = kUmChunk * a.m;                 // codes of one chunk, staged in shared memory a chunk ahead
        auto fetch_codes = [&](int c) {                        // 4-byte cp.async pieces; pieces beyond the CTA's tokens stay unread
            // a piece that starts below the limit is read whole: with m < 4 it can reach past the CTA's last token, never
            // past the row (L_max * m is a multiple of 4); tokens past the limit are zeroed when the keys are rebuilt
            const long long first = (long long)c * code_bytes, limit = t_end * a.m;
            for (int o = ptid * 4; o < code_bytes; o += kUmProducers * 4)
                if (first + o < limit)
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(um_smem(codes_s) + (c & 1) * 1024 + o),
                                 "l"(codes + first + o)
                                 : "memory");
        };
        // key rows of chunk c into key buffer c & 1: one 16-byte item of the codebook image per (token, 8-dim group, plane)
        auto rebuild_keys_as = [&](auto pair_c, int c) {
            constexpr bool PAIR = decltype(pair_c)::value;
            const int buf = c & 1;
            const bool whole = (long long)(c + 1) * kUmChunk <= t_end;   // every token of the chunk is visible to the CTA
            const uint8_t *cs = codes_s + buf * 1024 + my_j;
#pragma unroll
            for (int half = 0; half < 2; ++half) {             // in two batches: all loads of a batch before its stores
                uint32_t code[Lay::kItems / 2], code_b[PAIR ? Lay::kItems / 2 : 1];
                uint4 item[Lay::kItems / 2];
#pragma unroll
                for (int i = 0; i < Lay::kItems / 2; ++i) {
                    const uint8_t *ct = cs + (tl0 + (half * (Lay::kItems / 2) + i) * kTokStep) * a.m;
                    code[i] = ct[0];
                    if constexpr (PAIR) code_b[i] = ct[1];
                }
#pragma unroll
                for (int i = 0; i < Lay::kItems / 2; ++i) {
                    item[i] = make_uint4(0u, 0u, 0u, 0u);
                    if (whole || (long long)c * kUmChunk + tl0 + (half * (Lay::kItems / 2) + i) * kTokStep < t_end) {
                        if constexpr (!PAIR) {
                            item[i] = *reinterpret_cast<const uint4 *>(my_src + code[i] * 128);
                        } else {
                            // sub-vectors of 4 dims: the group's first half from the centroid of subspace 2 gi, its second
                            // half from the centroid of subspace 2 gi + 1 (the image holds both at the same place of their rows)
                            const uint2 lo = *reinterpret_cast<const uint2 *>(my_src + code[i] * 128);
                            const uint2 hi = *reinterpret_cast<const uint2 *>(my_src + code_b[i] * 128 + 8);
                            item[i] = make_uint4(lo.x, lo.y, hi.x, hi.y);
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < Lay::kItems / 2; ++i) {
                    const int tl = tl0 + (half * (Lay::kItems / 2) + i) * kTokStep;
                    *reinterpret_cast<uint4 *>(my_dst + buf * Lay::kKeys + tl * 128 + (((my_gi & 7) ^ (tl & 7)) << 4)) = item[i];
                }
            }
            um_fence_async_smem();                             // generic-proxy writes before the MMA's reads
            um_bar_arrive(bar_k + 8 * buf);
        };
        auto rebuild_keys = [&](int c) {
            if constexpr (D_K == 64) {                         // (16 subspaces at most: sub-vectors of 4 dims only on 64-dim heads)
                if (pair) {
                    rebuild_keys_as(std::true_type{}, c);
                    return;
                }
            }
            rebuild_keys_as(std::false_type{}, c);
        };
        fetch_codes(0);
        if (n_chunks > 1) fetch_codes(1);
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("bar.sync 1, %0;" ::"n"(kUmProducers) : "memory");
        rebuild_keys(0);
        asm volatile("bar.sync 1, %0;" ::"n"(kUmProducers) : "memory");   // everyone is done with the codes of chunk 0
        // keys of chunk c into the buffer that the score MMAs of chunk c - 2 (both tiles) have released
        for (int c = 1; c < n_chunks; ++c) {
            if (c >= 2) {
                bool ok = true;
#pragma unroll
                for (int t = 0; t < kUmTiles; ++t)
                    ok = um_group_wait<1, kUmProducers>(ptid == 0, bar_s + 16 * t + 8 * (c & 1), ((c - 2) >> 1) & 1) && ok;
                if (!ok) { dead = true; break; }
            }
            rebuild_keys(c);
            if (c + 1 < n_chunks) fetch_codes(c + 1);          // into the code buffer the keys of chunk c - 1 were built from
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            asm volatile("bar.sync 1, %0;" ::"n"(kUmProducers) : "memory");   // those codes are visible to all key producers
        }
    } else if (warp >= (kUmSoftmax + kUmProducers) / 32) {
        // =================== V loaders ===================
        const int vtid = tid - kUmSoftmax - kUmProducers;
        const __half *vsrc = a.v + (size_t)(b * a.H_kv + h) * a.L_max * D_V;
        constexpr int kPieces = kUmChunk * (D_V / 8) / kUmVLoaders;
        for (int c = 0; c < n_chunks; ++c) {
            const int buf = c & 1;
            // the V buffer of chunk c - 2 is free once both tiles' value MMAs of that chunk are done
            if (c >= 2) {
                bool ok = true;
#pragma unroll
                for (int t = 0; t < kUmTiles; ++t)
                    ok = um_group_wait<2, kUmVLoaders>(vtid == 0, bar_pv + 16 * t + 8 * buf, ((c - 2) >> 1) & 1) && ok;
                if (!ok) { dead = true; break; }
            }
            // V rows as [nb][token][128 B] with the 16-byte pieces swizzled by token.  A whole chunk comes by TMA (one
            // tiled bulk copy per 64-column block, 128-byte swizzle, completion counted in bytes on the barrier);
            // the last, partial chunk by cp.async with the rows the CTA does not see zeroed.
            const bool whole = (long long)(c + 1) * kUmChunk <= t_end;
            if (whole && use_tma) {
                if (vtid == 0) {
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_v + 8 * buf), "r"(Lay::kV) : "memory");
#pragma unroll
                    for (int nb = 0; nb < Lay::kNb; ++nb)
                        asm volatile(
                            "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                                sm0 + Lay::kOffV + buf * Lay::kV + nb * (kUmChunk * 128)),
                            "l"(reinterpret_cast<uint64_t>(&v_map)), "r"(nb * 64), "r"(c * kUmChunk), "r"(b * a.H_kv + h), "r"(bar_v + 8 * buf)
                            : "memory");
                }
            } else {
#pragma unroll
                for (int i = 0; i < kPieces; ++i) {
                    const int p = vtid + i * kUmVLoaders, tl = p / (D_V / 8), pc = p % (D_V / 8);
                    const uint32_t off = Lay::kOffV + buf * Lay::kV + (pc >> 3) * (kUmChunk * 128) + tl * 128 + (((pc & 7) ^ (tl & 7)) << 4);
                    if (whole || (long long)c * kUmChunk + tl < t_end)
                        um_cp_async16(sm0 + off, vsrc + ((size_t)c * kUmChunk + tl) * D_V + pc * 8);
                    else
                        *reinterpret_cast<uint4 *>(sm + off) = make_uint4(0u, 0u, 0u, 0u);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                um_fence_async_smem();
                asm volatile("bar.sync 2, %0;" ::"n"(kUmVLoaders) : "memory");   // every loader's rows have landed
                if (vtid == 0) um_bar_arrive(bar_v + 8 * buf);
            }
        }
    } else {
        // =================== softmax of tile t: thread r owns query row r of the tile (tensor-memory lane r) ===================
        const int t = warp >> 2, rq = warp & 3, r = rq * 32 + lane;
        const long long row = row0 + (pair_heads ? 0 : t * kUmRows) + r;
        const int hq = hq_first + (pair_heads ? t : 0);
        const long long vis_end = a.q_pos0 + (row < a.L_q ? row : a.L_q - 1) + 1;    // tokens this row sees
        const uint32_t lane_base = (uint32_t)(rq * 32) << 16;
        const uint32_t tm_s = tmem + t * kUmChunk + lane_base, tm_o = tmem + Lay::kColO + t * D_V + lane_base;
        float m_run = -INFINITY, l_run = 0.f;                  // reference point (base-2 exponent units) and row sum
        for (int c = 0; c < n_chunks; ++c) {
            const int buf = c & 1;
            const long long tok0 = (long long)c * kUmChunk;
            if (!__all_sync(0xffffffffu, um_bar_wait(bar_s + 16 * t + 8 * buf, (c >> 1) & 1))) { dead = true; break; }   // warp-uniform
            um_fence_after();
            float sc[kUmChunk];                                // raw scores
            {
                uint32_t s0[32], s1[32];
                um_ld32(s0, tm_s);
                um_ld32(s1, tm_s + 32);
                um_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    sc[i] = __uint_as_float(s0[i]);
                    sc[32 + i] = __uint_as_float(s1[i]);
                }
            }
            if (SCORES && a.scores_out && row < a.L_q) {
                float *dst = a.scores_out + ((size_t)(b * a.H_q + hq) * a.L_q + row) * a.L_max + tok0;
#pragma unroll
                for (int i = 0; i < kUmChunk; ++i)
                    if (tok0 + i < vis_end) dst[i] = sc[i];
            }
            if (tok0 + kUmChunk > vis_end) {                   // the chunk crosses (or lies beyond) this row's causal limit
#pragma unroll
                for (int i = 0; i < kUmChunk; ++i)
                    if (tok0 + i >= vis_end) sc[i] = -INFINITY;
            }
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < kUmChunk; ++i) mx = fmaxf(mx, sc[i]);
            // The reference point m_run of the exponentials follows the row maximum lazily: it moves only when the
            // maximum has grown by more than kUmSlack (base-2 units), so weights stay below 2^kUmSlack (fine in fp16
            // and in the fp32 sums) and O is rescaled rarely.  Any reference gives the same normalised result.
            const float m_cand = mx * a.scale_log2;             // the scale is positive; finite in chunk 0 (token 0 is visible)
            const bool move = m_cand > m_run + kUmSlack;
            const float alpha = move ? ex2_approx(m_run - m_cand) : 1.f;
            m_run = move ? m_cand : m_run;
            uint32_t pk[32];
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float p0 = ex2_approx(fmaf(sc[2 * i], a.scale_log2, -m_run));
                const float p1 = ex2_approx(fmaf(sc[2 * i + 1], a.scale_log2, -m_run));
                const __half2 h01 = __floats2half2_rn(p0, p1);
                pk[i] = *reinterpret_cast<const uint32_t *>(&h01);
                const float2 b01 = __half22float2(h01);        // the row sum takes the weights as the MMA sees them:
                sum += b01.x + b01.y;                          // their rounding cancels in the normalised result
            }
            l_run = l_run * alpha + sum;
            // The tile's previous value MMA is complete: the commit behind s_full covers every MMA its thread issued
            // before, and value(c - 1) was issued before scores(c).  So O may be rescaled right away.
            if (c >= 1 && __any_sync(0xffffffffu, alpha != 1.f)) {   // a reference point moved in this warp's rows
#pragma unroll 1
                for (int part = 0; part < D_V / 32; ++part) {
                    uint32_t o[32];
                    um_ld32(o, tm_o + part * 32);
                    um_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    um_st32(tm_o + part * 32, o);
                }
            }
            um_st32(tm_s, pk);                                 // the 64 weights over the first half of the scores, two per column
            um_wait_st();
            um_fence_before();
            um_bar_arrive(bar_p + 8 * t);
        }
        if (!dead && __all_sync(0xffffffffu, um_bar_wait(bar_pv + 16 * t + 8 * ((n_chunks - 1) & 1), ((n_chunks - 1) >> 1) & 1))) {
            um_fence_after();
            const float inv = 1.f / l_run;
#pragma unroll 1
            for (int part = 0; part < D_V / 32; ++part) {
                uint32_t o[32];
                um_ld32(o, tm_o + part * 32);
                um_wait_ld();
                if (row < a.L_q) {
                    float4 *dst = reinterpret_cast<float4 *>(a.out + ((size_t)(b * a.H_q + hq) * a.L_q + row) * D_V + part * 32);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[i] = make_float4(__uint_as_float(o[4 * i]) * inv, __uint_as_float(o[4 * i + 1]) * inv,
                                             __uint_as_float(o[4 * i + 2]) * inv, __uint_as_float(o[4 * i + 3]) * inv);
                }
            }
        } else {
            dead = true;
        }
    }

    if (dead) atomicExch(timeout_flag, 1);
    um_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(Lay::kTmemCols) : "memory");
}

// A wait that nothing will ever satisfy, with a short limit: exercises the path wait-ran-out -> flag -> host status
// without hanging anything (the bounded loop ends by itself after 4096 polls).
__global__ void um_timeout_selftest_kernel(int *__restrict__ timeout_flag)
{
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        um_bar_init(um_smem(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!um_bar_wait(um_smem(&bar), 0, 4096)) atomicExch(timeout_flag, 1);
    }
}

template <int D_K, int D_V>
lookat_status launch_um(Ctx *ctx, const PrefillArgs &a)
{
    using Lay = UmLayout<D_K, D_V>;
    // the codebooks as shared-memory images of two fp16 planes, rewritten at every call (the caller may have refitted them)
    const size_t elems = (size_t)a.H_kv * a.K * a.d_k;
    lookat_status st = ensure(ctx, (void **)&ctx->split_books, &ctx->split_cap, 2 * elems * sizeof(__half), "codebook planes");
    if (st != LOOKAT_OK) return st;
    um_codebook_image_kernel<<<(unsigned)((elems + 1023) / 1024), 256, 0, ctx->stream>>>(a.codebooks, ctx->split_books, a.H_kv,
                                                                                         a.m, a.K, a.d_k / a.m);
    st = check_launch(ctx, "um_codebook_image_kernel");
    if (st != LOOKAT_OK) return st;

    // tensor map of V as [row * head][token][d_v] for tiled bulk copies of 64 tokens x 64 columns with the 128-byte
    // swizzle the MMA operand wants; without the driver entry point the loaders use cp.async for every chunk
    CUtensorMap v_map;
    memset(&v_map, 0, sizeof(v_map));
    int use_tma = 0;
    {
        typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                      const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        static encode_fn encode = nullptr;
        static bool looked = false;
        if (!looked) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult q;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
                q == cudaDriverEntryPointSuccess)
                encode = reinterpret_cast<encode_fn>(fn);
            else
                cudaGetLastError();
            looked = true;
        }
        if (encode) {
            const cuuint64_t dims[3] = {(cuuint64_t)D_V, (cuuint64_t)a.L_max, (cuuint64_t)a.B * a.H_kv};
            const cuuint64_t strides[2] = {(cuuint64_t)D_V * 2, (cuuint64_t)a.L_max * D_V * 2};
            const cuuint32_t box[3] = {64, (cuuint32_t)kUmChunk, 1}, estr[3] = {1, 1, 1};
            use_tma = encode(&v_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half *>(a.v), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        }
    }

    // grouped heads: a CTA takes two query heads of a KV head over 128 rows; else two row tiles of one head
    const int pair_heads = a.g % 2 == 0 ? 1 : 0;
    const int rows_per_cta = pair_heads ? kUmRows : kUmTiles * kUmRows;
    const int n_tiles = (int)((a.L_q + rows_per_cta - 1) / rows_per_cta);
    const int smem = (int)Lay::bytes(a.K);
    dim3 grid((unsigned)n_tiles, (unsigned)(pair_heads ? a.H_q / 2 : a.H_q), (unsigned)a.B);
    auto launch = [&](auto kern) -> lookat_status {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return check_launch(ctx, "prefill (tcgen05 form): shared-memory opt-in");
        kern<<<grid, kUmThreads, smem, ctx->stream>>>(a, ctx->split_books, ctx->timeout_flag, v_map, use_tma, pair_heads);
        return check_launch(ctx, "attend_prefill_umma_kernel");
    };
    if (a.scores_out) return launch(attend_prefill_umma_kernel<D_K, D_V, true>);
    return launch(attend_prefill_umma_kernel<D_K, D_V, false>);
}

}  // namespace

bool prefill_umma_covers(const Ctx *ctx, const PrefillArgs &a)
{
    const int d_sub = a.d_k / a.m;
    // (m <= 16: the codes of a chunk are staged in 1 KB of shared memory)
    const bool shape = (a.d_k == 64 || a.d_k == 128) && (a.d_v == 64 || a.d_v == 128) && (d_sub % 8 == 0 || d_sub == 4) && a.m <= 16;
    const bool aligned = ((uintptr_t)a.q & 15) == 0 && ((uintptr_t)a.v & 15) == 0 && ((uintptr_t)a.codes & 3) == 0 &&
                         (a.L_max * a.m) % 4 == 0;
    // the row maxima are taken on the raw scores, which needs a positive softmax scale
    if (!shape || !aligned || a.H_q > 65535 || a.B > 65535 || !(a.scale_log2 > 0.f) || !ctx->timeout_flag) return false;
    const size_t operands = 2 * (size_t)kUmChunk * a.d_k * 4 + 2 * (size_t)kUmChunk * a.d_v * 2;   // two key tiles (two planes), two V tiles
    return operands + (size_t)a.K * a.d_k * 4 + 256 + 2048 <= (size_t)ctx->max_smem_optin;
}

lookat_status launch_timeout_selftest(Ctx *ctx)
{
    if (!ctx->timeout_flag) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "no time-out flag on this context");
    um_timeout_selftest_kernel<<<1, 32, 0, ctx->stream>>>(ctx->timeout_flag);
    return check_launch(ctx, "um_timeout_selftest_kernel");
}

lookat_status launch_prefill_umma(Ctx *ctx, const PrefillArgs &a)
{
    if (a.d_k == 128) return a.d_v == 128 ? launch_um<128, 128>(ctx, a) : launch_um<128, 64>(ctx, a);
    return a.d_v == 128 ? launch_um<64, 128>(ctx, a) : launch_um<64, 64>(ctx, a);
}

}  // namespace lookat
