// Multi-query causal attention over the compressed keys, contraction form (Algorithm 1 applied to a
// tile of queries).  The score of Section 3.4,
//     s[q][t] = sum_j LUT_j[code[t][j]],   LUT_j[c] = q^(j) . C_j[c],
// is the inner product of q with the key rebuilt from its codes, k^[t] = (C_1[code[t][1]], ...,
// C_m[code[t][m]]).  A table pays when one query meets many keys; in prefill many queries meet each
// key, so this kernel gathers the centroids of a chunk of tokens ONCE per CTA into shared memory (the
// codes stay the only stored form of the keys; nothing is written back to HBM) and lets 128 queries
// take their scores from it on the tensor cores: S = Q . K^^T, online softmax, O += P . V, all with
// mma.sync.m16n8k16 and fp32 accumulation.  q (fp16) is an exact operand; every fp32 centroid is
// split into two fp16 planes (rounding + remainder), which carries s to ~2^-22 relative.
//
//
// One CTA: one (batch row, query head), 128 consecutive queries (8 warps x 16 rows), 64-token chunks up
// to the causal limit of the tile.  Both planes of the head's codebooks (K x d_k x 4 bytes, 128 KB at
// d_k = 128) stay in shared memory for the life of the CTA, in an order that makes the gathers free of
// bank conflicts whatever the codes are: the 16-byte item of (8-dim group gi, plane p, centroid c)
// lives in bank group (2 gi + p) mod 8, and the 8 lanes of a quarter-warp always fetch 8 different
// (gi, p).  split_codebook_kernel writes that image once per call; a CTA copies it in with cp.async.
// Per chunk: the next chunk's V rows arrive by cp.async and its key rows are rebuilt (one 16-byte
// shared load and store per item) while this chunk's MMAs run; the codes are read one chunk further
// ahead; one barrier per chunk.  Key and V tiles are XOR-swizzled (16-byte piece index ^ token mod 8)
// instead of padded, so that everything fits in 224 KB.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kPmWarps = 8;
constexpr int kPmThreads = kPmWarps * 32;
constexpr int kPmRows = kPmWarps * 16;        // queries per CTA
constexpr int kPmChunk = 64;                  // tokens per chunk

__device__ __forceinline__ void pm_cp_async16(unsigned dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void pm_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void pm_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void pm_ldmatrix_x4(uint32_t (&r)[4], unsigned src)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(src));
}
__device__ __forceinline__ void pm_ldmatrix_x4_trans(uint32_t (&r)[4], unsigned src)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(src));
}
__device__ __forceinline__ void pm_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pm_pack(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}


// Shared-memory image of one head's codebooks as two fp16 planes, hi = fp16(c), lo = fp16(c - hi):
// halfs [d_k/32][K][8 slots][8], slot = 2 (gi mod 4) + plane for the 8-dim group gi of the key row.
__global__ void split_codebook_kernel(const float *__restrict__ books, __half *__restrict__ images, int H_kv, int m, int K,
                                      int d_sub)
{
    const int d_k = m * d_sub;
    const size_t n = (size_t)H_kv * K * d_k;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        // i indexes books [h][j][c][e]
        const int e = (int)(i % d_sub), c = (int)(i / d_sub % K), j = (int)(i / ((size_t)d_sub * K) % m);
        const int h = (int)(i / ((size_t)d_sub * K * m));
        const int dim = j * d_sub + e, gi = dim >> 3;
        const float v = books[i];
        const __half hi = __float2half_rn(v), lo = __float2half_rn(v - __half2float(hi));
        __half *img = images + (size_t)h * K * d_k * 2;
        const size_t at = (((size_t)(gi >> 2) * K + c) * 8 + (gi & 3) * 2) * 8 + (dim & 7);
        img[at] = hi;
        img[at + 8] = lo;
    }
}

template <int D_K, int D_V>
struct PmLayout {
    static constexpr int kRowK = D_K * 2;                              // bytes per rebuilt key row (one plane)
    static constexpr int kRowV = D_V * 2;
    static constexpr int kPlane = kPmChunk * kRowK;
    static constexpr int kVTile = kPmChunk * kRowV;
    static constexpr int kStage = 2 * kPlane + kVTile;                 // hi plane, lo plane, V
    static constexpr int kIds = D_K / 4;                               // 16-byte items per key row, both planes
    static constexpr int kItems = kPmChunk * kIds / kPmThreads;        // items rebuilt per thread per chunk
    static_assert(kPmChunk * kIds % kPmThreads == 0, "whole items per thread");
    static size_t book_bytes(int K) { return (size_t)K * D_K * 4; }
    static size_t bytes(int K) { return book_bytes(K) + 2 * kStage; }
};

template <int D_K, int D_V, bool SCORES, bool SPLIT_P>
__global__ void __launch_bounds__(kPmThreads, 1)
attend_prefill_mma_kernel(PrefillArgs a, const __half *__restrict__ images)
{
    using Lay = PmLayout<D_K, D_V>;
    extern __shared__ __align__(128) unsigned char pm_smem[];
    const unsigned smem0 = (unsigned)__cvta_generic_to_shared(pm_smem);
    const unsigned book_bytes = (unsigned)a.K * D_K * 4;
    unsigned char *const stages = pm_smem + book_bytes;
    const unsigned stages0 = smem0 + book_bytes;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int n_tiles = (int)((a.L_q + kPmRows - 1) / kPmRows);
    const int tile = n_tiles - 1 - (int)blockIdx.x;            // longest tiles first
    const int hq = blockIdx.y, b = blockIdx.z, h = hq / a.g;
    const int d_sub = D_K / a.m;

    const long long row0 = (long long)tile * kPmRows;
    const long long t_end = a.q_pos0 + (row0 + kPmRows < a.L_q ? row0 + kPmRows : a.L_q);   // tokens the tile sees
    const int n_chunks = (int)((t_end + kPmChunk - 1) / kPmChunk);

    const uint8_t *codes = a.codes + (size_t)(b * a.H_kv + h) * a.L_max * a.m;
    const __half *vsrc = a.v + (size_t)(b * a.H_kv + h) * a.L_max * D_V;

    // ---- the head's codebook image: a flat copy ----
    {
        const unsigned char *img = reinterpret_cast<const unsigned char *>(images) + (size_t)h * book_bytes;
        for (unsigned i = tid * 16; i < book_bytes; i += kPmThreads * 16) pm_cp_async16(smem0 + i, img + i);
    }

    // ---- this thread's two query rows (clamped copies beyond L_q are computed and dropped) ----
    long long row[2], vis_end[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        row[i] = row0 + warp * 16 + g + 8 * i;
        const long long rc = row[i] < a.L_q ? row[i] : a.L_q - 1;
        vis_end[i] = a.q_pos0 + rc + 1;
    }
    const long long warp_first = row0 + warp * 16, warp_last = warp_first + 15;
    const long long w_min_end = a.q_pos0 + (warp_first < a.L_q ? warp_first : a.L_q - 1) + 1;
    const long long w_max_end = a.q_pos0 + (warp_last < a.L_q ? warp_last : a.L_q - 1) + 1;

    uint32_t qa[D_K / 16][4];
    {
        const __half *qb = a.q + (size_t)(b * a.H_q + hq) * a.L_q * D_K;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const __half *qr = qb + (size_t)(vis_end[i] - 1 - a.q_pos0) * D_K;
#pragma unroll
            for (int ks = 0; ks < D_K / 16; ++ks) {
                qa[ks][i] = *reinterpret_cast<const uint32_t *>(qr + ks * 16 + 2 * t);
                qa[ks][2 + i] = *reinterpret_cast<const uint32_t *>(qr + ks * 16 + 2 * t + 8);
            }
        }
    }

    // ---- staging of one chunk ----
    auto stage_v = [&](int c, int buf) {                        // V rows by cp.async, pieces swizzled by token
        constexpr int per_row = D_V * 2 / 16;
        const unsigned vo = buf * Lay::kStage + 2 * Lay::kPlane;
#pragma unroll
        for (int i = 0; i < kPmChunk * per_row / kPmThreads; ++i) {
            const int p = tid + i * kPmThreads, tl = p / per_row, piece = p % per_row;
            const long long tok = (long long)c * kPmChunk + tl;
            const unsigned off = vo + tl * Lay::kRowV + ((piece ^ (tl & 7)) << 4);
            if (tok < t_end)
                pm_cp_async16(stages0 + off, vsrc + (size_t)tok * D_V + piece * 8);
            else
                *reinterpret_cast<uint4 *>(stages + off) = make_uint4(0u, 0u, 0u, 0u);
        }
        pm_commit();
    };
    // item p = tid + i * threads of a chunk: token p / kIds, id = p % kIds = 2 gi + plane
    const int my_id = tid % Lay::kIds, my_gi = my_id >> 1, my_plane = my_id & 1;
    const int my_j = (my_gi * 8) / d_sub;
    const unsigned my_src = (unsigned)(my_gi >> 2) * a.K * 128 + (((my_gi & 3) * 2 + my_plane) << 4);   // + c * 128
    uint32_t cd[Lay::kItems];                                   // codes of this thread's items; 0xffffffff = token not seen
    auto load_codes = [&](int c) {
#pragma unroll
        for (int i = 0; i < Lay::kItems; ++i) {
            const int tl = (tid + i * kPmThreads) / Lay::kIds;
            const long long tok = (long long)c * kPmChunk + tl;
            cd[i] = tok < t_end ? (uint32_t)codes[(size_t)tok * a.m + my_j] : 0xffffffffu;
        }
    };
    auto rebuild_keys = [&](int buf) {                          // uses cd[]: the chunk whose codes were loaded last
#pragma unroll
        for (int i = 0; i < Lay::kItems; ++i) {
            const int tl = (tid + i * kPmThreads) / Lay::kIds;
            uint4 item = make_uint4(0u, 0u, 0u, 0u);
            if (cd[i] != 0xffffffffu) item = *reinterpret_cast<const uint4 *>(pm_smem + my_src + cd[i] * 128);
            *reinterpret_cast<uint4 *>(stages + buf * Lay::kStage + my_plane * Lay::kPlane + tl * Lay::kRowK +
                                       ((my_gi ^ (tl & 7) ^ (my_plane << 2)) << 4)) = item;
        }
    };

    load_codes(0);
    stage_v(0, 0);                                              // commits the codebook copy as well
    pm_wait_all();
    __syncthreads();
    rebuild_keys(0);
    if (n_chunks > 1) load_codes(1);
    __syncthreads();

    float o[D_V / 8][4];
#pragma unroll
    for (int nd = 0; nd < D_V / 8; ++nd) o[nd][0] = o[nd][1] = o[nd][2] = o[nd][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};                    // running maxima, in units of the base-2 exponent
    float l_acc[4] = {0.f, 0.f, 0.f, 0.f};                      // running row sums: P times a block of ones
    constexpr uint32_t kOnes = 0x3c003c00u;                     // half2(1, 1)

    // ldmatrix lane addresses.  Keys: token lane&7 of an 8-token group, 16-byte piece (lane>>3) of a 32-dim
    // group; the lo plane's pieces are swizzled with one more bit (^4).  V: token (lane&7) + 8 ((lane>>3)&1),
    // piece lane>>4 of a 16-column group.
    const int r7 = lane & 7;
    const unsigned k_row = r7 * Lay::kRowK;
    const unsigned v_row = (r7 + ((lane >> 3) & 1) * 8) * Lay::kRowV;

    for (int c = 0; c < n_chunks; ++c) {
        const int buf = c & 1;
        const bool more = c + 1 < n_chunks;
        const long long tok0 = (long long)c * kPmChunk;
        const bool active = tok0 < w_max_end;                  // warp-uniform: some row of this warp sees the chunk
        float s[kPmChunk / 8][4];
        if (active) {
            const unsigned kh = stages0 + buf * Lay::kStage + k_row;
#pragma unroll
            for (int nt = 0; nt < kPmChunk / 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < D_K / 32; ++kp) {
                const unsigned piece = (unsigned)(((kp * 4 + (lane >> 3)) ^ r7) << 4);
#pragma unroll
                for (int nt = 0; nt < kPmChunk / 8; ++nt) {
                    uint32_t bh[4], bl[4];
                    pm_ldmatrix_x4(bh, kh + nt * 8 * Lay::kRowK + piece);
                    pm_ldmatrix_x4(bl, kh + Lay::kPlane + nt * 8 * Lay::kRowK + (piece ^ 64u));
                    pm_mma(s[nt], qa[2 * kp], bh[0], bh[1]);
                    pm_mma(s[nt], qa[2 * kp + 1], bh[2], bh[3]);
                    pm_mma(s[nt], qa[2 * kp], bl[0], bl[1]);
                    pm_mma(s[nt], qa[2 * kp + 1], bl[2], bl[3]);
                }
            }
        }

        if (more) stage_v(c + 1, buf ^ 1);                     // issued while the score MMAs drain

        if (active) {
            // ---- raw scores out (validation), causal mask, online softmax in base 2 ----
            const bool masked = tok0 + kPmChunk > w_min_end;
            if (SCORES && a.scores_out) {
#pragma unroll
                for (int nt = 0; nt < kPmChunk / 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const long long tok = tok0 + nt * 8 + 2 * t + (e & 1);
                        const int i = e >> 1;
                        if (row[i] < a.L_q && tok < vis_end[i])
                            a.scores_out[((size_t)(b * a.H_q + hq) * a.L_q + row[i]) * a.L_max + tok] = s[nt][e];
                    }
            }
            float mx[2] = {-INFINITY, -INFINITY};               // row maxima of the raw scores (scale > 0)
#pragma unroll
            for (int nt = 0; nt < kPmChunk / 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (masked && tok0 + nt * 8 + 2 * t + (e & 1) >= vis_end[e >> 1]) s[nt][e] = -INFINITY;
                    mx[e >> 1] = fmaxf(mx[e >> 1], s[nt][e]);
                }
            float alpha[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 1));
                mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 2));
                const float m_new = fmaxf(m_run[i], mx[i] * a.scale_log2);   // finite from chunk 0 on: token 0 is visible to every row
                alpha[i] = ex2_approx(m_run[i] - m_new);
                m_run[i] = m_new;
            }
            if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {   // a maximum moved: rescale
#pragma unroll
                for (int nd = 0; nd < D_V / 8; ++nd) {
                    o[nd][0] *= alpha[0];
                    o[nd][1] *= alpha[0];
                    o[nd][2] *= alpha[1];
                    o[nd][3] *= alpha[1];
                }
                l_acc[0] *= alpha[0];
                l_acc[1] *= alpha[0];
                l_acc[2] *= alpha[1];
                l_acc[3] *= alpha[1];
            }
            // ---- weights as fp16 operands (two planes when SPLIT_P) ----
            uint32_t ph[kPmChunk / 8][2], pl[SPLIT_P ? kPmChunk / 8 : 1][2];
#pragma unroll
            for (int nt = 0; nt < kPmChunk / 8; ++nt)
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float p0 = ex2_approx(fmaf(s[nt][2 * i], a.scale_log2, -m_run[i]));
                    const float p1 = ex2_approx(fmaf(s[nt][2 * i + 1], a.scale_log2, -m_run[i]));
                    const __half2 hh = __floats2half2_rn(p0, p1);
                    ph[nt][i] = *reinterpret_cast<const uint32_t *>(&hh);
                    if (SPLIT_P) {
                        const float2 back = __half22float2(hh);
                        pl[nt][i] = pm_pack(p0 - back.x, p1 - back.y);
                    }
                }
            const unsigned vs = stages0 + buf * Lay::kStage + 2 * Lay::kPlane + v_row;
#pragma unroll
            for (int kt = 0; kt < kPmChunk / 16; ++kt) {
                const uint32_t pa[4] = {ph[2 * kt][0], ph[2 * kt][1], ph[2 * kt + 1][0], ph[2 * kt + 1][1]};
                pm_mma(l_acc, pa, kOnes, kOnes);                // row sums of exactly the weights the value sum uses
                if (SPLIT_P) {
                    const uint32_t pb[4] = {pl[2 * kt][0], pl[2 * kt][1], pl[2 * kt + 1][0], pl[2 * kt + 1][1]};
                    pm_mma(l_acc, pb, kOnes, kOnes);
                }
#pragma unroll
                for (int np = 0; np < D_V / 16; ++np) {
                    uint32_t vb[4];
                    pm_ldmatrix_x4_trans(vb, vs + kt * 16 * Lay::kRowV + (((np * 2 + (lane >> 4)) ^ r7) << 4));
                    pm_mma(o[2 * np], pa, vb[0], vb[1]);
                    pm_mma(o[2 * np + 1], pa, vb[2], vb[3]);
                    if (SPLIT_P) {
                        const uint32_t pb[4] = {pl[2 * kt][0], pl[2 * kt][1], pl[2 * kt + 1][0], pl[2 * kt + 1][1]};
                        pm_mma(o[2 * np], pb, vb[0], vb[1]);
                        pm_mma(o[2 * np + 1], pb, vb[2], vb[3]);
                    }
                }
            }
        }
        if (more) {
            rebuild_keys(buf ^ 1);                              // chunk c+1: its codes arrived during this step
            if (c + 2 < n_chunks) load_codes(c + 2);
        }
        pm_wait_all();
        __syncthreads();
    }

    // ---- normalise and store ----
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        if (row[i] >= a.L_q) continue;
        const float inv = 1.f / l_acc[2 * i];                   // every column of the ones block holds the row sum
        float *dst = a.out + ((size_t)(b * a.H_q + hq) * a.L_q + row[i]) * D_V + 2 * t;
#pragma unroll
        for (int nd = 0; nd < D_V / 8; ++nd)
            *reinterpret_cast<float2 *>(dst + nd * 8) = make_float2(o[nd][2 * i] * inv, o[nd][2 * i + 1] * inv);
    }
}

template <int D_K, int D_V>
lookat_status launch_pm(Ctx *ctx, const PrefillArgs &a)
{
    using Lay = PmLayout<D_K, D_V>;
    // the codebooks as shared-memory images of two fp16 planes, rewritten at every call (the caller may have refitted them)
    const size_t elems = (size_t)a.H_kv * a.K * a.d_k;
    lookat_status st = ensure(ctx, (void **)&ctx->split_books, &ctx->split_cap, 2 * elems * sizeof(__half), "codebook planes");
    if (st != LOOKAT_OK) return st;
    split_codebook_kernel<<<(unsigned)((elems + 1023) / 1024), 256, 0, ctx->stream>>>(a.codebooks, ctx->split_books, a.H_kv,
                                                                                      a.m, a.K, a.d_k / a.m);
    st = check_launch(ctx, "split_codebook_kernel");
    if (st != LOOKAT_OK) return st;

    const int n_tiles = (int)((a.L_q + kPmRows - 1) / kPmRows);
    const int smem = (int)Lay::bytes(a.K);
    dim3 grid((unsigned)n_tiles, (unsigned)a.H_q, (unsigned)a.B);
    auto launch = [&](auto kern) -> lookat_status {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return check_launch(ctx, "prefill (contraction form): shared-memory opt-in");
        kern<<<grid, kPmThreads, smem, ctx->stream>>>(a, ctx->split_books);
        return check_launch(ctx, "attend_prefill_mma_kernel");
    };
    if (a.scores_out) return launch(attend_prefill_mma_kernel<D_K, D_V, true, false>);
    return launch(attend_prefill_mma_kernel<D_K, D_V, false, false>);
}

}  // namespace

bool prefill_mma_covers(const Ctx *ctx, const PrefillArgs &a)
{
    const int d_sub = a.d_k / a.m;
    const bool shape = (a.d_k == 64 || a.d_k == 128) && (a.d_v == 64 || a.d_v == 128) && d_sub % 8 == 0;
    const bool aligned = ((uintptr_t)a.q & 3) == 0 && ((uintptr_t)a.v & 15) == 0;
    // the row maxima are taken on the raw scores, which needs a positive softmax scale
    if (!shape || !aligned || a.H_q > 65535 || a.B > 65535 || !(a.scale_log2 > 0.f)) return false;
    const size_t stage = (size_t)kPmChunk * (4 * a.d_k + 2 * a.d_v);
    return (size_t)a.K * a.d_k * 4 + 2 * stage <= (size_t)ctx->max_smem_optin;
}

lookat_status launch_prefill_mma(Ctx *ctx, const PrefillArgs &a)
{
    if (a.d_k == 128) return a.d_v == 128 ? launch_pm<128, 128>(ctx, a) : launch_pm<128, 64>(ctx, a);
    return a.d_v == 128 ? launch_pm<64, 128>(ctx, a) : launch_pm<64, 64>(ctx, a);
}

}  // namespace lookat
