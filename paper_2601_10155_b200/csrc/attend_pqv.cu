// Decode attention with product-quantised VALUES as well.  The paper leaves value compression to future work
// (Section 5.2); this formulation is this build's own and has no counterpart there.  The weights are those of
// Algorithm 1 (scores = sums of table entries named by the key codes, stable softmax); the output
//     o = sum_t alpha_t v^_t,   v^_t = (C^V_1[vcode[t][1]], ..., C^V_mv[vcode[t][mv]])
// is taken per value subspace as  o^(j) = sum_c w[j][c] C^V_j[c]  with the weight histogram
// w[j][c] = sum of alpha_t over the tokens whose value code in subspace j is c.  Nothing but codes is read per
// token: m + m_v bytes instead of m + 2 d_v.
//
// Work: the flat sequence (unit, block of 4096 tokens; 2048 where m + m_v > 16), unit = (batch row, KV head, group
// of HG <= 4 query heads), cut into equal contiguous ranges, one per CTA (persistent, one CTA per SM).  Per unit a
// CTA keeps in shared memory the unit's key tables and one histogram per (value subspace, head), both laid out
// [code][subspace][head] with the head fastest.
//
// A warp step covers 32 / LT tokens (LT = lanes per token: 2 for HG = 4, else 1); a lane carries two heads of its
// token (one for HG = 1) and walks the subspaces starting at subspace `slot mod m`, so that the lanes of a table
// read (8 bytes: both heads) and of a histogram update fall into different banks, never onto one address.  The
// codes reach the lanes by coalesced loads (one token per lane, a block ahead) and a shuffle per step.
//
// Per block: pass 1 sums the table entries into scores (kept in registers: 16 or 32 per lane) and forms the
// weights against the warp's own maximum; one barrier later every warp derives the block's maximum and weight sum
// from the warps' pairs, and pass 2 adds the weights, scaled, to the histograms.
//
// The histograms are 32-bit fixed point: a weight p <= 1 is added as round(p * S), so that integer adds in shared
// memory do the work (a floating-point add there is a compare-and-swap loop; a 64-bit add, measured, is as slow)
// and the result does not depend on the order of the adds.  S is set to 2^30 / l (l = sum of the weights so far)
// and kept while the running maximum stays and l * S <= 2^31; otherwise the histogram is rescaled in place
// (16,384 entries for m_v = 8, HG = 4 with doubled rows: 32 per thread, a few times per unit).  So S >= 2^30 / l:
// rounding a weight costs at most 2^-31 of the denominator, n tokens at most n * 2^-31 relative to the largest
// value centroid (1.5e-5 at 32K tokens), and no bin can reach 2^32.
//
// After a unit's last block the histograms are contracted with the value codebooks into a partial output; the CTA
// that completes a unit merges its partials (arrival counters, as in the streaming decode kernel): one launch.
//
// What bounds it: the table reads and histogram adds, 4 + 4 bytes of shared-memory traffic per (token, head,
// subspace) at 128 bytes per clock and SM, not HBM (m + m_v bytes per token and KV head).
#include "common.cuh"

#include <utility>

namespace lookat {

namespace {

constexpr int kPqThreads = 512;
constexpr int kPqWarps = kPqThreads / 32;
// Coalesced code loads per lane and block: a block is 16 warps x 32 lanes x this many tokens.  Larger blocks spread
// the per-block barriers and reductions over more tokens; the loaded codes and the weights of a block live in
// registers, which bounds it.
template <int M_K, int M_V>
__host__ __device__ constexpr int pqv_loads()
{
    return M_K + M_V <= 16 ? 8 : 4;
}
constexpr int kPqEntries = 256;                       // codes are bytes
constexpr float kPqNegBig = -1.0e30f;

struct PqvArgs {
    const float *lut;        // [B][H_q][m][K]
    const uint8_t *codes;    // [B][H_kv][L_max][m]
    const float *v_books;    // [H_kv][m_v][K_v][d_vsub]
    const uint8_t *v_codes;  // [B][H_kv][L_max][m_v]
    const int32_t *seq_lens;
    float *part_o;           // [CTA + unit][4][d_v]
    float *part_ml;          // [CTA + unit][4][2]: maximum (base-2 units), sum
    unsigned *tickets;       // [unit] arrival counters, zero between launches
    float *out;              // [B][H_q][d_v]
    long long L_max;
    long long blocks_per_unit, blocks_per_cta, n_units;
    int B, H_q, H_kv, g, K, K_v, d_vsub, d_v;
    int vec4;                // the value codebooks can be read four dims at a time
    float scale_log2;
    int *status;             // the context's status word (debug build)
};

// the m code bytes of one token as 32-bit words (m = 2: the low half of one word)
template <int M>
struct CodeWords {
    static constexpr int NW = M >= 4 ? M / 4 : 1;
    uint32_t w[NW];
};

// debug build: every code byte against its limit (clamped and recorded); nothing in the normal build
template <int M>
__device__ __forceinline__ void check_code_words(CodeWords<M> &c, int K, int *status)
{
#ifdef LOOKAT_DEBUG
    constexpr int BYTES = M >= 4 ? M : (M == 2 ? 4 : 4);        // m = 2 keeps its two bytes twice in one word
#pragma unroll
    for (int byte = 0; byte < BYTES; ++byte) {
        const unsigned sh = (unsigned)(byte & 3) * 8u;
        const int code = (int)((c.w[byte >> 2] >> sh) & 0xffu);
        const int ok = checked_code(code, K, status);
        c.w[byte >> 2] = (c.w[byte >> 2] & ~(0xffu << sh)) | ((uint32_t)ok << sh);
    }
#endif
}

template <int M>
__device__ __forceinline__ CodeWords<M> load_code_words(const uint8_t *row)
{
    CodeWords<M> c;
    if constexpr (M == 16) {
        const uint4 x = __ldg(reinterpret_cast<const uint4 *>(row));
        c.w[0] = x.x, c.w[1] = x.y, c.w[2] = x.z, c.w[3] = x.w;
    } else if constexpr (M == 8) {
        const uint2 x = __ldg(reinterpret_cast<const uint2 *>(row));
        c.w[0] = x.x, c.w[1] = x.y;
    } else if constexpr (M == 4) {
        c.w[0] = __ldg(reinterpret_cast<const uint32_t *>(row));
    } else {
        c.w[0] = __ldg(reinterpret_cast<const uint16_t *>(row));
    }
    return c;
}

template <int M>
__device__ __forceinline__ CodeWords<M> shfl_code_words(const CodeWords<M> &c, int src)
{
    CodeWords<M> r;
#pragma unroll
    for (int i = 0; i < CodeWords<M>::NW; ++i) r.w[i] = __shfl_sync(0xffffffffu, c.w[i], src);
    return r;
}

// rotate the m bytes so that byte (s + r) mod m comes to position s (0 <= r < m)
template <int M>
__device__ __forceinline__ void rotate_code_bytes(CodeWords<M> &c, int r)
{
    const int sh = 8 * (r & 3);
    if constexpr (M == 2) {
        c.w[0] = ((c.w[0] & 0xffffu) * 0x10001u) >> sh;
    } else if constexpr (M == 4) {
        c.w[0] = __funnelshift_r(c.w[0], c.w[0], sh);
    } else if constexpr (M == 8) {
        const uint32_t lo = (r & 4) ? c.w[1] : c.w[0], hi = (r & 4) ? c.w[0] : c.w[1];
        c.w[0] = __funnelshift_r(lo, hi, sh);
        c.w[1] = __funnelshift_r(hi, lo, sh);
    } else {
        uint32_t t[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) t[i] = (r & 4) ? c.w[(i + 1) & 3] : c.w[i];
        uint32_t u[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) u[i] = (r & 8) ? t[(i + 2) & 3] : t[i];
#pragma unroll
        for (int i = 0; i < 4; ++i) c.w[i] = __funnelshift_r(u[i], u[(i + 1) & 3], sh);
    }
}

template <int M>
__device__ __forceinline__ unsigned code_byte(const CodeWords<M> &c, int s)     // s is a compile-time constant
{
    return __byte_perm(c.w[s >> 2], 0u, 0x4440u | (unsigned)(s & 3));           // byte s, zero-extended
}

// Shared-memory accesses of the two passes, by 32-bit shared address plus a constant: the address arithmetic of
// a lookup stays at "take the byte, shift, add".
template <int IMM>
__device__ __forceinline__ float lds_f32(unsigned addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(IMM));
    return v;
}

__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int IMM>
__device__ __forceinline__ float2 lds_f32x2(unsigned addr)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2+%3];" : "=f"(v.x), "=f"(v.y) : "r"(addr), "n"(IMM));
    return v;
}

template <int IMM>
__device__ __forceinline__ void red_shared_add_u32(unsigned addr, unsigned val)
{
    asm volatile("red.shared.add.u32 [%0+%1], %2;" ::"r"(addr), "n"(IMM), "r"(val) : "memory");
}

template <int N, class F>
__device__ __forceinline__ void static_for(F &&f)
{
    [&]<int... I>(std::integer_sequence<int, I...>) { (f(std::integral_constant<int, I>{}), ...); }(std::make_integer_sequence<int, N>{});
}

__host__ __device__ constexpr int pqv_log2(int v)
{
    int r = 0;
    while (v > 1) v >>= 1, ++r;
    return r;
}

// Rows of the tables and histograms: per code value, [subspace][head].  Where shared memory allows, a row holds
// its m subspaces twice over, so that "subspace (slot + step) mod m" is the plain sum slot + step and a lane's
// address is one register plus a constant per step; otherwise the sum wraps.
template <int M_K, int M_V, int HG>
__host__ __device__ constexpr bool pqv_doubled()
{
#ifdef LOOKAT_PQV_NODUP
    return false;
#else
    return (size_t)kPqEntries * 2 * (M_K + M_V) * HG * 4 <= 160 * 1024;
#endif
}

template <int M_K, int M_V, int HG>
constexpr size_t pqv_table_bytes()
{
    return (size_t)kPqEntries * (M_K + M_V) * HG * 4 * (pqv_doubled<M_K, M_V, HG>() ? 2 : 1);
}

template <int M_K, int M_V, int HG>
constexpr int pqv_min_ctas()
{
#ifdef LOOKAT_PQV_MIN_CTAS
    return LOOKAT_PQV_MIN_CTAS;
#else
    return pqv_table_bytes<M_K, M_V, HG>() + 16 * 1024 <= 100 * 1024 ? 2 : 1;
#endif
}

template <int M_K, int M_V, int HG>
__global__ void __launch_bounds__(kPqThreads, pqv_min_ctas<M_K, M_V, HG>()) attend_pqv_kernel(PqvArgs a)
{
    extern __shared__ __align__(16) unsigned char pq_smem[];
    constexpr int kPqLoads = pqv_loads<M_K, M_V>();
    constexpr int kPqWarpTokens = 32 * kPqLoads;           // tokens of a block that one warp handles
    constexpr int kPqBlock = kPqWarps * kPqWarpTokens;     // tokens of a block
    constexpr int HL = HG >= 2 ? 2 : 1;                    // heads per lane (one 8-byte table read serves two)
    constexpr int LT = HG / HL;                            // lanes per token
    constexpr int SLOTS = 32 / LT;                         // tokens per warp step
    constexpr int G = kPqLoads * LT;                       // warp steps per block
    constexpr bool DUP = pqv_doubled<M_K, M_V, HG>();
    constexpr int ROW_K = M_K * HG * (DUP ? 2 : 1), ROW_V = M_V * HG * (DUP ? 2 : 1);   // entries per code value
    float *tab = reinterpret_cast<float *>(pq_smem);                                    // [256][M_K (x2)][HG]
    unsigned *hist = reinterpret_cast<unsigned *>(pq_smem + kPqEntries * ROW_K * 4);    // [256][M_V (x2)][HG]
    float *hist_f = reinterpret_cast<float *>(hist);
    float *red = reinterpret_cast<float *>(pq_smem + kPqEntries * (ROW_K + ROW_V) * 4); // [c range][HG][d_v]
    __shared__ float s_max[kPqWarps][HG], s_sum[kPqWarps][HG];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hp = lane % LT, ts = lane / LT;              // this lane: token slot ts, heads hp * HL + {0, HL - 1}
    const int h0 = hp * HL;                                // tid % LT == hp as well: the thread count is a multiple
    const int rk = ts & (M_K - 1), rv = ts & (M_V - 1);    // the subspace this lane starts at
    const int src_rk = (lane % SLOTS) & (M_K - 1);         // ... and that of the lanes which get the codes this lane loads
    const int src_rv = (lane % SLOTS) & (M_V - 1);
    // entry of (code, step) for this lane: code * ROW + pos(step), pos = (start + step [mod m]) * HG + head
    constexpr int SH_K = pqv_log2(ROW_K * 4), SH_V = pqv_log2(ROW_V * 4);      // a row's bytes are a power of two
    const unsigned tab_s = (unsigned)__cvta_generic_to_shared(tab), hist_s = (unsigned)__cvta_generic_to_shared(hist);
    const unsigned kbase = tab_s + 4u * (rk * HG + h0), vbase = hist_s + 4u * (rv * HG + h0);
    const int hgroups = (a.g + HG - 1) / HG;

    const long long cta = blockIdx.x;
    const long long T_lo = cta * a.blocks_per_cta;
    const long long T_hi = min(a.n_units * a.blocks_per_unit, T_lo + a.blocks_per_cta);

    for (long long T = T_lo; T < T_hi;) {
        const long long unit = T / a.blocks_per_unit;
        const long long blk0 = T - unit * a.blocks_per_unit;
        const long long nblk = min(a.blocks_per_unit - blk0, T_hi - T);
        const int hgrp = (int)(unit % hgroups);
        const long long kv_row = unit / hgroups;
        const int b = (int)(kv_row / a.H_kv), kvh = (int)(kv_row - (long long)b * a.H_kv);
        const int heads = min(HG, a.g - hgrp * HG);
        const int hq0 = kvh * a.g + hgrp * HG;
        long long len = a.seq_lens ? (long long)a.seq_lens[b] : a.L_max;
        len = len < 0 ? 0 : (len > a.L_max ? a.L_max : len);

        // ---- the unit's key tables, head fastest; histograms cleared ----
        __syncthreads();                                   // the previous unit's shared memory is no longer read
        // this lane's code rows: token (block * 2048 + warp * 128 + load * 32 + lane)
        const uint8_t *kptr = a.codes + ((size_t)kv_row * a.L_max + (size_t)blk0 * kPqBlock + warp * kPqWarpTokens + lane) * M_K;
        const uint8_t *vptr = a.v_codes + ((size_t)kv_row * a.L_max + (size_t)blk0 * kPqBlock + warp * kPqWarpTokens + lane) * M_V;
        // tokens of this warp's part of a block that exist (at most 128, possibly none or negative)
        auto warp_tokens = [&](long long blk) {
            const long long left = len - blk * kPqBlock - warp * kPqWarpTokens;
            return (int)(left < kPqWarpTokens ? (left < 0 ? 0 : left) : kPqWarpTokens);
        };
        CodeWords<M_K> kc[kPqLoads];
        CodeWords<M_V> vc[kPqLoads];
        auto load_k = [&](int n_tok) {
#pragma unroll
            for (int i = 0; i < kPqLoads; ++i) {
                if (i * 32 + lane < n_tok) {
                    kc[i] = load_code_words<M_K>(kptr + (size_t)i * 32 * M_K);
                    check_code_words<M_K>(kc[i], a.K, a.status);
                } else {
#pragma unroll
                    for (int w = 0; w < CodeWords<M_K>::NW; ++w) kc[i].w[w] = 0u;
                }
            }
            kptr += (size_t)kPqBlock * M_K;
        };
        auto load_v = [&](int n_tok) {
#pragma unroll
            for (int i = 0; i < kPqLoads; ++i) {
                if (i * 32 + lane < n_tok) {
                    vc[i] = load_code_words<M_V>(vptr + (size_t)i * 32 * M_V);
                    check_code_words<M_V>(vc[i], a.K_v, a.status);
                } else {
#pragma unroll
                    for (int w = 0; w < CodeWords<M_V>::NW; ++w) vc[i].w[w] = 0u;
                }
            }
            vptr += (size_t)kPqBlock * M_V;
        };
        load_k(warp_tokens(blk0));                         // in flight while the tables are set up

        // The query-time tables are [head][subspace][code]; rows here are [code][subspace][head].  Read coalesced into
        // the (still unused) histogram region, a row's entries XOR-swizzled by the row number, and transposed from
        // there: neither side has a bank conflict.  (Without room there: strided reads straight from global memory.)
        constexpr bool STAGE = ROW_V >= M_K * HG;
        if constexpr (STAGE) {
            const float *src = a.lut + ((size_t)b * a.H_q + hq0) * M_K * a.K;      // heads * M_K rows of K entries
            const int rows = heads * M_K;
#pragma unroll 8
            for (int i = tid; i < kPqEntries * M_K * HG; i += kPqThreads) {
                const int row = i / kPqEntries, cc = i % kPqEntries;
                hist_f[row * kPqEntries + (cc ^ (row & 31))] = (row < rows && cc < a.K) ? __ldg(src + (size_t)row * a.K + cc) : 0.f;
            }
            __syncthreads();
        }
#pragma unroll 8
        for (int i = tid; i < kPqEntries * M_K * HG; i += kPqThreads) {
            const int hh = i % HG, j = (i / HG) % M_K, cc = i / (M_K * HG);
            float e;
            if constexpr (STAGE) {
                const int row = hh * M_K + j;
                e = hist_f[row * kPqEntries + (cc ^ (row & 31))];
            } else {
                e = (hh < heads && cc < a.K) ? __ldg(a.lut + (((size_t)b * a.H_q + hq0 + hh) * M_K + j) * a.K + cc) : 0.f;
            }
            tab[cc * ROW_K + j * HG + hh] = e;
            if (DUP) tab[cc * ROW_K + (j + M_K) * HG + hh] = e;
        }
        if constexpr (STAGE) __syncthreads();              // the staged tables are read: the region becomes the histograms
        for (int i = tid; i < kPqEntries * ROW_V / 4; i += kPqThreads) reinterpret_cast<uint4 *>(hist)[i] = make_uint4(0u, 0u, 0u, 0u);

        __syncthreads();

        // running maximum, weight sum and histogram scale of this lane's heads (the same in every thread of a head)
        float M_run[HL], l_run[HL], S_run[HL];
#pragma unroll
        for (int e = 0; e < HL; ++e) M_run[e] = kPqNegBig, l_run[e] = 0.f, S_run[e] = 0.f;
        for (long long blk = blk0; blk < blk0 + nblk; ++blk) {
            if (blk * kPqBlock >= len) break;              // the same decision in every thread
            const int n_tok = warp_tokens(blk);
            load_v(n_tok);                                 // lands during pass 1

            // ---- pass 1: scores (base-2 units) into registers, the block's maxima ----
            float x[G][HL];
            float mx[HL];
#pragma unroll
            for (int e = 0; e < HL; ++e) mx[e] = -INFINITY;
#pragma unroll
            for (int i = 0; i < kPqLoads; ++i) {
                CodeWords<M_K> rot = kc[i];
                rotate_code_bytes<M_K>(rot, src_rk);       // step s of the receiving lanes finds its byte at position s
#pragma unroll
                for (int r = 0; r < LT; ++r) {
                    const CodeWords<M_K> cw = shfl_code_words<M_K>(rot, r * SLOTS + ts);
                    float s[HL];
#pragma unroll
                    for (int e = 0; e < HL; ++e) s[e] = 0.f;
                    static_for<M_K>([&](auto st_c) {
                        constexpr int ST = decltype(st_c)::value;
                        const unsigned off = code_byte<M_K>(cw, ST) << SH_K;
                        unsigned addr;
                        if constexpr (DUP) addr = kbase + off;
                        else addr = tab_s + 4u * (((rk + ST) & (M_K - 1)) * HG + h0) + off;
                        if constexpr (HL == 2) {
                            const float2 t = lds_f32x2<DUP ? ST * HG * 4 : 0>(addr);
                            s[0] += t.x, s[1] += t.y;
                        } else {
                            s[0] += lds_f32<DUP ? ST * HG * 4 : 0>(addr);
                        }
                    });
                    const bool tok_ok = i * 32 + r * SLOTS + ts < n_tok;
#pragma unroll
                    for (int e = 0; e < HL; ++e) {
                        const float v = (tok_ok && h0 + e < heads) ? s[e] * a.scale_log2 : -INFINITY;
                        x[i * LT + r][e] = v;
                        mx[e] = fmaxf(mx[e], v);
                    }
                }
            }
            if (blk + 1 < blk0 + nblk) load_k(warp_tokens(blk + 1));   // lands during pass 2

            // ---- weights against this warp's maxima; the warp's (maximum, sum) pairs go to shared memory ----
            float ls[HL];
#pragma unroll
            for (int e = 0; e < HL; ++e) {
#pragma unroll
                for (int o = LT; o < 32; o <<= 1) mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], o));
                mx[e] = fmaxf(mx[e], kPqNegBig);           // a warp without tokens: finite, so that -inf minus it stays -inf
                ls[e] = 0.f;
            }
#pragma unroll
            for (int gi = 0; gi < G; ++gi) {
#pragma unroll
                for (int e = 0; e < HL; ++e) {
                    x[gi][e] = ex2_approx(x[gi][e] - mx[e]);           // a token past the end has -inf: weight 0
                    ls[e] += x[gi][e];
                }
            }
#pragma unroll
            for (int e = 0; e < HL; ++e) {
#pragma unroll
                for (int o = LT; o < 32; o <<= 1) ls[e] += __shfl_xor_sync(0xffffffffu, ls[e], o);
                if (ts == 0) s_max[warp][h0 + e] = mx[e], s_sum[warp][h0 + e] = ls[e];
            }
            __syncthreads();

            // ---- the block's maximum and sum from the warps' pairs (lane = (warp, head pair); butterfly sums are
            //      the same in every lane and warp), then the histogram's scale ----
            float wscale[HL], resc[HL];
            bool any_resc = false;
#pragma unroll
            for (int e = 0; e < HL; ++e) {
                constexpr int PER = (kPqWarps + SLOTS - 1) / SLOTS;    // pairs per lane
                float m_w[PER], l_w[PER];
                float m_blk = kPqNegBig;
#pragma unroll
                for (int k = 0; k < PER; ++k) {
                    const int w = ts + k * SLOTS;
                    m_w[k] = w < kPqWarps ? s_max[w][h0 + e] : kPqNegBig;
                    l_w[k] = w < kPqWarps ? s_sum[w][h0 + e] : 0.f;
                    m_blk = fmaxf(m_blk, m_w[k]);
                }
#pragma unroll
                for (int o = LT; o < 32; o <<= 1) m_blk = fmaxf(m_blk, __shfl_xor_sync(0xffffffffu, m_blk, o));
                const float M_new = fmaxf(M_run[e], m_blk);
                float l_blk = 0.f;
#pragma unroll
                for (int k = 0; k < PER; ++k) l_blk += l_w[k] * ex2_approx(m_w[k] - M_new);
#pragma unroll
                for (int o = LT; o < 32; o <<= 1) l_blk += __shfl_xor_sync(0xffffffffu, l_blk, o);
                const float f = ex2_approx(M_run[e] - M_new);          // what the histogram so far is worth against M_new
                const float l_new = l_run[e] * f + l_blk;
                // The scale stays while the maximum does and the sum of all bins, l * S, stays within 2^31; otherwise
                // it is set to 2^30 / l (room for the sum to double) and the histogram is rescaled.  So S >= 2^30 / l
                // always: rounding one weight costs at most 2^-31 of the denominator.
                float S_new = S_run[e];
                resc[e] = 1.f;
                if (!(f == 1.f && l_new * S_run[e] <= 2147483648.f) || S_run[e] == 0.f) {
                    S_new = l_new > 0.f ? 1073741824.f * rcp_approx(l_new) : 0.f;     // any value near it serves
                    if (S_run[e] > 0.f) resc[e] = f * S_new * rcp_approx(S_run[e]), any_resc = true;
                }
                wscale[e] = S_new * ex2_approx(mx[e] - M_new);         // this warp's weights are against its own maximum
                M_run[e] = M_new, l_run[e] = l_new, S_run[e] = S_new;
            }
            if (any_resc) {
                // entries HL at a time: vector v holds heads (v mod LT) * HL + e, and v = tid (mod LT) here
#pragma unroll 4
                for (int v = tid; v < kPqEntries * ROW_V / HL; v += kPqThreads) {
                    if constexpr (HL == 2) {
                        uint2 n = reinterpret_cast<uint2 *>(hist)[v];
                        n.x = __float2uint_rn(__uint2float_rn(n.x) * resc[0]);
                        n.y = __float2uint_rn(__uint2float_rn(n.y) * resc[1]);
                        reinterpret_cast<uint2 *>(hist)[v] = n;
                    } else {
                        hist[v] = __float2uint_rn(__uint2float_rn(hist[v]) * resc[0]);
                    }
                }
            }
            __syncthreads();

            // ---- pass 2: the weights into the histograms ----
            // With two heads per lane the slots ts and ts + 8 would meet in one bank: the upper half of the slots
            // adds its heads in the other order, so that each of the two adds spreads over all 32 banks.
            const int sw = HL == 2 ? (ts >> 3) & 1 : 0;
            const unsigned vbase_a = vbase + 4u * sw, vbase_b = vbase + 4u * (1 - sw);
#pragma unroll
            for (int i = 0; i < kPqLoads; ++i) {
                CodeWords<M_V> rot = vc[i];
                rotate_code_bytes<M_V>(rot, src_rv);
#pragma unroll
                for (int r = 0; r < LT; ++r) {
                    const CodeWords<M_V> vw = shfl_code_words<M_V>(rot, r * SLOTS + ts);
                    unsigned wq[HL];
#pragma unroll
                    for (int e = 0; e < HL; ++e) wq[e] = __float2uint_rn(x[i * LT + r][e] * wscale[e]);
                    const unsigned wa = sw ? wq[HL - 1] : wq[0], wb = sw ? wq[0] : wq[HL - 1];
                    static_for<M_V>([&](auto st_c) {
                        constexpr int ST = decltype(st_c)::value;
                        constexpr int IMM = DUP ? ST * HG * 4 : 0;
                        const unsigned off = (code_byte<M_V>(vw, ST) << SH_V) + (DUP ? 0u : 4u * (((rv + ST) & (M_V - 1)) * HG) - 4u * (rv * HG));
                        red_shared_add_u32<IMM>(vbase_a + off, wa);
                        if constexpr (HL == 2) red_shared_add_u32<IMM>(vbase_b + off, wb);
                    });
                }
            }
        }
        __syncthreads();                                   // every add has landed

        // ---- partial output of the range: o[h][j * d_vsub + i] = sum_c w[h][j][c] * C^V_j[c][i] ----
        {
            float inv_S[HL];
#pragma unroll
            for (int e = 0; e < HL; ++e) inv_S[e] = S_run[e] > 0.f ? 1.f / S_run[e] : 0.f;
            for (int v = tid; v < kPqEntries * M_V * HG / HL; v += kPqThreads) {    // v = tid (mod LT) here too
                const int row = v / (M_V * HG / HL), col = v - row * (M_V * HG / HL);
                const int e0 = row * ROW_V + col * HL;
#pragma unroll
                for (int e = 0; e < HL; ++e) {
                    const unsigned n = DUP ? hist[e0 + e] + hist[e0 + e + M_V * HG] : hist[e0 + e];   // both halves of a doubled row
                    hist_f[e0 + e] = __uint2float_rn(n) * inv_S[e];
                }
            }
        }
        __syncthreads();
        const float *vb = a.v_books + (size_t)kvh * M_V * a.K_v * a.d_vsub;
        int nq;                                            // ranges of c summed side by side
        float *pbuf = red;                                 // their partial sums [range][head][d_v]
        if (a.vec4) {
            // four dims per thread, up to 16 ranges, every load of a range in flight at once; the partial sums go
            // where the key tables were (no longer read)
            const int Q = a.d_v >> 2;
            nq = kPqThreads / Q < 16 ? kPqThreads / Q : 16;
            while (nq > 1 && (size_t)nq * HG * a.d_v > (size_t)kPqEntries * ROW_K) nq >>= 1;
            if ((size_t)nq * HG * a.d_v <= (size_t)kPqEntries * ROW_K) pbuf = tab;      // else one range, in `red`
            const int cspan = (a.K_v + nq - 1) / nq;
            for (int idx = tid; idx < nq * Q; idx += kPqThreads) {
                const int cq = idx / Q, dim = (idx - cq * Q) * 4, j = dim / a.d_vsub, i = dim - j * a.d_vsub;
                const int c0 = cq * cspan, c1 = min(a.K_v, c0 + cspan);
                const float *w = hist_f + j * HG;
                const float *cv = vb + (size_t)j * a.K_v * a.d_vsub + i;
                float4 acc[HG];
#pragma unroll
                for (int hh = 0; hh < HG; ++hh) acc[hh] = make_float4(0.f, 0.f, 0.f, 0.f);
                int c = c0;
                for (; c + 16 <= c1; c += 16) {
                    float4 v[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u) v[u] = __ldg(reinterpret_cast<const float4 *>(cv + (size_t)(c + u) * a.d_vsub));
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
#pragma unroll
                        for (int hh = 0; hh < HG; ++hh) {
                            const float ww = w[(c + u) * ROW_V + hh];
                            acc[hh].x = fmaf(ww, v[u].x, acc[hh].x), acc[hh].y = fmaf(ww, v[u].y, acc[hh].y);
                            acc[hh].z = fmaf(ww, v[u].z, acc[hh].z), acc[hh].w = fmaf(ww, v[u].w, acc[hh].w);
                        }
                    }
                }
                for (; c < c1; ++c) {
                    const float4 v = __ldg(reinterpret_cast<const float4 *>(cv + (size_t)c * a.d_vsub));
#pragma unroll
                    for (int hh = 0; hh < HG; ++hh) {
                        const float ww = w[c * ROW_V + hh];
                        acc[hh].x = fmaf(ww, v.x, acc[hh].x), acc[hh].y = fmaf(ww, v.y, acc[hh].y);
                        acc[hh].z = fmaf(ww, v.z, acc[hh].z), acc[hh].w = fmaf(ww, v.w, acc[hh].w);
                    }
                }
#pragma unroll
                for (int hh = 0; hh < HG; ++hh) *reinterpret_cast<float4 *>(pbuf + (size_t)(cq * HG + hh) * a.d_v + dim) = acc[hh];
            }
        } else {
        nq = a.d_v >= kPqThreads ? 1 : kPqThreads / a.d_v;
        const int cspan = (a.K_v + nq - 1) / nq;
        for (int idx = tid; idx < nq * a.d_v; idx += kPqThreads) {
            const int cq = idx / a.d_v, dim = idx - cq * a.d_v, j = dim / a.d_vsub, i = dim - j * a.d_vsub;
            const int c0 = cq * cspan, c1 = min(a.K_v, c0 + cspan);
            const float *w = hist_f + j * HG;
            const float *cv = vb + (size_t)j * a.K_v * a.d_vsub + i;
            float acc[HG];
#pragma unroll
            for (int hh = 0; hh < HG; ++hh) acc[hh] = 0.f;
            int c = c0;
            for (; c + 8 <= c1; c += 8) {                  // eight loads in flight
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = __ldg(cv + (size_t)(c + u) * a.d_vsub);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
#pragma unroll
                    for (int hh = 0; hh < HG; ++hh) acc[hh] = fmaf(w[(c + u) * ROW_V + hh], v[u], acc[hh]);
                }
            }
            for (; c < c1; ++c) {
                const float v = __ldg(cv + (size_t)c * a.d_vsub);
#pragma unroll
                for (int hh = 0; hh < HG; ++hh) acc[hh] = fmaf(w[c * ROW_V + hh], v, acc[hh]);
            }
#pragma unroll
            for (int hh = 0; hh < HG; ++hh) red[(cq * HG + hh) * a.d_v + dim] = acc[hh];
        }
        }
        __syncthreads();
        const size_t pslot = (size_t)(cta + unit) * 4;     // + head
        for (int o = tid; o < heads * a.d_v; o += kPqThreads) {
            const int hh = o / a.d_v, dim = o - hh * a.d_v;
            float sum = 0.f;
            for (int cq = 0; cq < nq; ++cq) sum += pbuf[(cq * HG + hh) * a.d_v + dim];
            a.part_o[(pslot + hh) * a.d_v + dim] = sum;
        }
        if (tid < LT) {                                    // thread tid < LT carries heads tid * HL + e
#pragma unroll
            for (int e = 0; e < HL; ++e) {
                if (h0 + e < heads) {
                    a.part_ml[(pslot + h0 + e) * 2] = M_run[e];
                    a.part_ml[(pslot + h0 + e) * 2 + 1] = l_run[e];
                }
            }
        }

        // ---- the CTA that completes a unit merges the unit's partials into the output ----
        const long long c_lo = unit * a.blocks_per_unit / a.blocks_per_cta;
        const long long c_hi = ((unit + 1) * a.blocks_per_unit - 1) / a.blocks_per_cta;
        // the CTA's partial is written (barrier), thread 0's fence makes it visible before the ticket (fences are
        // cumulative over what the barrier ordered); the same on the reading side
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            const unsigned arrived = atomicAdd(a.tickets + unit, 1u);
            s_last = arrived == (unsigned)(c_hi - c_lo);
            if (s_last) {
                a.tickets[unit] = 0u;                      // ready for the next launch
                __threadfence();
            }
        }
        __syncthreads();
        if (s_last) {
            for (int o = tid; o < heads * a.d_v; o += kPqThreads) {
                const int hh = o / a.d_v, dim = o - hh * a.d_v;
                float Mx = kPqNegBig;
                for (long long c2 = c_lo; c2 <= c_hi; ++c2)
                    Mx = fmaxf(Mx, __ldcg(a.part_ml + ((size_t)(c2 + unit) * 4 + hh) * 2));
                float acc = 0.f, l = 0.f;
                for (long long c2 = c_lo; c2 <= c_hi; ++c2) {
                    const size_t pp = (size_t)(c2 + unit) * 4 + hh;
                    const float lp = __ldcg(a.part_ml + pp * 2 + 1);
                    if (lp > 0.f) {
                        const float fp = ex2_approx(__ldcg(a.part_ml + pp * 2) - Mx);
                        l += fp * lp;
                        acc += fp * __ldcg(a.part_o + pp * a.d_v + dim);
                    }
                }
                a.out[((size_t)b * a.H_q + hq0 + hh) * a.d_v + dim] = l > 0.f ? acc / l : 0.f;
            }
        }
        T += nblk;
    }
}

template <int M_K, int M_V, int HG>
lookat_status launch_pqv(Ctx *ctx, PqvArgs &a)
{
    const int red_floats = HG * (a.d_v > kPqThreads ? a.d_v : kPqThreads);
    const size_t smem = pqv_table_bytes<M_K, M_V, HG>() + (size_t)red_floats * sizeof(float);
    if (smem > (size_t)ctx->max_smem_optin)
        return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: tables and histograms need %zu bytes of shared memory", smem);
    auto kern = attend_pqv_kernel<M_K, M_V, HG>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return check_launch(ctx, "attend_pqv: shared-memory opt-in");
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kPqThreads, smem) != cudaSuccess || per_sm < 1)
        return check_launch(ctx, "attend_pqv: occupancy query");
    const long long hgroups = (a.g + HG - 1) / HG;
    a.n_units = (long long)a.B * a.H_kv * hgroups;
    constexpr int kPqBlock = kPqWarps * 32 * pqv_loads<M_K, M_V>();
    a.blocks_per_unit = (a.L_max + kPqBlock - 1) / kPqBlock;
    const long long total = a.n_units * a.blocks_per_unit;
    if (a.n_units > (1ll << 30) || total > (1ll << 40)) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: problem too large");
    long long ctas = (long long)per_sm * ctx->sm_count;
    if (ctas > total) ctas = total;
    a.blocks_per_cta = (total + ctas - 1) / ctas;
    const long long n_ctas = (total + a.blocks_per_cta - 1) / a.blocks_per_cta;

    const size_t slots = (size_t)(n_ctas + a.n_units) * 4;                 // slot of (CTA c, unit u) = c + u
    lookat_status st = ensure(ctx, (void **)&ctx->part_o, &ctx->part_o_cap, slots * a.d_v * sizeof(float), "partials");
    if (st == LOOKAT_OK) st = ensure(ctx, (void **)&ctx->part_ml, &ctx->part_ml_cap, slots * 2 * sizeof(float), "partials");
    if (st != LOOKAT_OK) return st;
    const size_t need = (size_t)a.n_units * sizeof(unsigned);             // all zero between launches
    if (need > ctx->tickets_cap) {
        st = ensure(ctx, (void **)&ctx->tickets, &ctx->tickets_cap, need, "unit counters");
        if (st != LOOKAT_OK) return st;
        if (cudaMemsetAsync(ctx->tickets, 0, ctx->tickets_cap, ctx->stream) != cudaSuccess)
            return set_error(ctx, LOOKAT_ERR_CUDA, "memset failed");
    }
    a.part_o = ctx->part_o;
    a.part_ml = ctx->part_ml;
    a.tickets = ctx->tickets;
    kern<<<(unsigned)n_ctas, kPqThreads, smem, ctx->stream>>>(a);
    return check_launch(ctx, "attend_pqv_kernel");
}

template <int M_K, int M_V>
lookat_status launch_pqv_hg(Ctx *ctx, PqvArgs &a)
{
    if (a.g >= 3) return launch_pqv<M_K, M_V, 4>(ctx, a);
    if (a.g == 2) return launch_pqv<M_K, M_V, 2>(ctx, a);
    return launch_pqv<M_K, M_V, 1>(ctx, a);
}

template <int M_K>
lookat_status launch_pqv_mv(Ctx *ctx, PqvArgs &a, int m_v)
{
    switch (m_v) {
        case 2: return launch_pqv_hg<M_K, 2>(ctx, a);
        case 4: return launch_pqv_hg<M_K, 4>(ctx, a);
        case 8: return launch_pqv_hg<M_K, 8>(ctx, a);
        case 16: return launch_pqv_hg<M_K, 16>(ctx, a);
        default: return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: m_v must be 2, 4, 8 or 16");
    }
}

}  // namespace

lookat_status attend_pqv_impl(Ctx *ctx, const float *lut, const uint8_t *codes, const float *v_books, const uint8_t *v_codes,
                              int m_v, int K_v, int B, long long L_max, const int32_t *seq_lens, float *out)
{
    const lookat_config &c = ctx->cfg;
    if (m_v < 1 || c.d_v % m_v != 0 || K_v < 1 || K_v > 256)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "attend_pqv: need m_v | d_v and 1 <= K_v <= 256 (m_v=%d K_v=%d)", m_v, K_v);
    if (c.K > 256) return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: K must be at most 256");
    // code rows are read with one aligned load of m (m_v) bytes
    if (((uintptr_t)codes % (c.m >= 16 ? 16 : c.m)) != 0 || ((uintptr_t)v_codes % (m_v >= 16 ? 16 : m_v)) != 0)
        return set_error(ctx, LOOKAT_ERR_INVALID_ARG, "attend_pqv: code arrays must be aligned to their row size");
    PqvArgs a;
    memset(&a, 0, sizeof(a));
    a.lut = lut;
    a.codes = codes;
    a.v_books = v_books;
    a.v_codes = v_codes;
    a.seq_lens = seq_lens;
    a.out = out;
    a.L_max = L_max;
    a.B = B;
    a.H_q = c.n_q_heads;
    a.H_kv = c.n_kv_heads;
    a.g = c.n_q_heads / c.n_kv_heads;
    a.K = c.K;
    a.K_v = K_v;
    a.d_v = c.d_v;
    a.d_vsub = c.d_v / m_v;
    a.scale_log2 = ctx->scale * 1.4426950408889634f;
    a.status = ctx->status_word;
    a.vec4 = (a.d_vsub % 4 == 0 && ((uintptr_t)v_books & 15u) == 0 && a.d_v / 4 <= kPqThreads) ? 1 : 0;
    switch (c.m) {
        case 2: return launch_pqv_mv<2>(ctx, a, m_v);
        case 4: return launch_pqv_mv<4>(ctx, a, m_v);
        case 8: return launch_pqv_mv<8>(ctx, a, m_v);
        case 16: return launch_pqv_mv<16>(ctx, a, m_v);
        default: return set_error(ctx, LOOKAT_ERR_UNSUPPORTED, "attend_pqv: m must be 2, 4, 8 or 16");
    }
}

}  // namespace lookat
