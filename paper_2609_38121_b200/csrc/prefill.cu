// Chunk (prefill) attention over the mixed cache: Algorithm 2 line 3 (query / key transforms) and line 5 for a
// chunk of S' > 1 new positions, after the chunk has been appended (line 4); Sections 4.4 and 5.3.
//
// Chunk position i of a sequence attends to every cached position up to itself.  Positions of the chunk are read
// in full precision (k' = bf16(T_K k), v as given: the method appends a new chunk in full precision and computes the
// chunk's attention output from those copies), older positions follow the window rule: the sink and the recent window from
// their bf16 copies, the quantized middle from the packed pages (x_hat = x_min + Delta * code, Eq. 6 / Eq. 5).
//
// Two launches:
//   1. transforms              q' = T_K^{-T} q and k' = T_K k of the chunk on tensor cores (bf16 products, fp32
//                              accumulation), written as fp16 operands of the attention kernel (k' through its bf16
//                              rounding, the value the cache's window copies hold; q' as value + rounding
//                              remainder), the chunk's values as fp16, and sum_c q'_c per query row.
//                              prefill_prep_tc_kernel (tcgen05, section 1b); prefill_prep_kernel (mma.sync, section 1)
//                              without bulk tensor copies and as a testing aid.  Projected rows are normalised and
//                              rotated in shared memory first (Algorithm 2 lines 1-2) by either.
//   2. attention               prefill_attn_ws_kernel (default, section 2c): one CTA per (sequence, KV head, pair of
//                              128-row tiles that pack the G query heads), warp-specialised, both contractions as
//                              tcgen05.mma with accumulators in tensor memory.
//                              prefill_attn_tc_kernel (testing aid "prefill_one_tile", section 2b): the same contractions,
//                              one tile per CTA, no role split.
//                              prefill_attn_kernel (testing aid "prefill_legacy", section 2): one CTA per (sequence, query
//                              head, 64 query rows) on mma.sync.m16n8k16; the first version.
//                              The last two are kept as further implementations to test against.
//   All stream 64-key tiles of the three sources through shared memory and keep an online softmax
//   (flash-attention recurrence) per row.  The affine part of the quantizer is factored out of the contractions,
//   per key j of a tile:
//                                score_ij = Delta_k,j (q'_i . c_k,j) + x_min_k,j sum(q'_i)
//                                o_i     += (p_ij Delta_v,j) c_v,j + (p_ij x_min_v,j) 1
//   so packed pages are staged as their integer codes (exact in fp16) and full-precision rows with Delta = 1,
//   x_min = 0.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <type_traits>

#include "host_common.h"
#include "layout.cuh"
#include "prologue.cuh"

namespace wushkv {

namespace {

constexpr unsigned FULLM = 0xffffffffu;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr int BM = 64;                    // query rows per CTA
constexpr int BN = 64;                    // keys per tile (= one packed page)
constexpr int TILE_PITCH = D + 8;         // halves per staged row: 272 bytes, conflict-free for ldmatrix
constexpr int PF_THREADS = 128;

struct PrefillParams {
    CacheView c;
    int batch, total_new;
    const int* slot;
    const int* seq_len;                   // lengths after the chunk was appended
    const int* cu_new;
    const unsigned short* K_new;          // bf16 [total_new][n_kv][D] post-RoPE
    const unsigned short* V_new;          // bf16 [total_new][n_kv][D]
    const unsigned short* Q_new;          // bf16 [total_new][n_q][D] post-RoPE
    float* O;                             // [total_new][n_q][D]
    __half* KP;                           // [total_new][n_kv][D]  fp16(bf16(T_K k))
    __half* VP;                           // [total_new][n_kv][D]  fp16(v)
    __half* QP;                           // [2][total_new][n_q][D]  q' = T_K^{-T} q as fp16 value, then fp16 rounding remainder
    float* qsum;                          // [total_new][n_q]      sum over channels of q' (value + remainder)
    int tiles_per_seq;                    // ceil(max_new / BM)
    int use_tma;                          // 1: the tcgen05 kernel stages the chunk's own tiles with bulk tensor copies
    Prologue pro;                         // pro.rope != nullptr: K_new / Q_new are projected; Norm and RoPE are applied by the
    const float* q_weight;                // transform kernel (pro.weight: key weights, q_weight: query weights)
    int n_split;                          // warp-specialised kernel: CTAs per tile pair, each over a share of the key tiles (1: none)
    float* part;                          // n_split > 1: [n_split][total_new][n_q][PART_W] partial outputs
    int wait_limit;                       // poll limit of the barrier waits (0: default, a second or more)
    int drop;                             // testing aid: 1 the first tile's score MMAs are never committed, 2 the first bulk copy of a
                                          // CTA's first chunk tile is announced but never issued, 3 the same in the transform kernel
                                          // (the wait then runs into its limit)
};

__device__ __forceinline__ unsigned smem_addr(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void ldsm_x4(unsigned addr, unsigned& a, unsigned& b, unsigned& c, unsigned& d) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(unsigned addr, unsigned& a, unsigned& b, unsigned& c, unsigned& d) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}
__device__ __forceinline__ void hmma(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
// three-input maximum
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ unsigned pack_half2(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// ------------------------------------------------------------------------------------------------
// 1. transforms of the chunk (Algorithm 2 line 3)
// ------------------------------------------------------------------------------------------------
// One CTA of 8 warps per (tile of 128 tokens, head slot); head slots 0 .. n_kv-1 are the key heads, the rest the
// query heads.  out[token][i] = sum_j x[token][j] T[i][j] on tensor cores (mma.sync bf16, fp32 accumulation): the
// token tile is the A operand as it comes (bf16), the transform the B operand.  T_K is bf16-valued (one term);
// T_K^{-T} is fp32 and is fed as three bf16 terms (value, remainder, remainder of the remainder: 24 mantissa bits),
// so the products are exact and the result is the fp32 dot product up to summation order.
constexpr int PREP_TOK = 128;
constexpr int PREP_PITCH = D + 8;             // bf16 per staged row (272 bytes: conflict-free ldmatrix)
__device__ __forceinline__ void mma_bf16_prep(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__global__ void __launch_bounds__(256) prefill_prep_kernel(PrefillParams P) {
    extern __shared__ __align__(16) unsigned short sm16[];
    unsigned short* Xs = sm16;                            // [PREP_TOK][PREP_PITCH]
    unsigned short* Ts = sm16 + PREP_TOK * PREP_PITCH;    // [terms][D][PREP_PITCH]: Ts[term][i][j] = term of T[i][j]
    const int hs = blockIdx.y;
    const bool is_key = hs < P.c.n_kv;
    const int head = is_key ? hs : hs - P.c.n_kv;
    const int kvh = is_key ? head : head / P.c.G;
    const int n_terms = is_key ? 1 : 3;
    const float* T = (is_key ? P.c.T_K : P.c.T_K_invT) + static_cast<long long>(kvh) * D * D;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    for (int idx = tid; idx < D * D; idx += 256) {
        const int i = idx >> 7, j = idx & 127;
        float x = __ldg(T + idx);
#pragma unroll
        for (int term = 0; term < 3; ++term) {
            if (term < n_terms) {
                const unsigned short hb = float_to_bf16_bits(x);
                Ts[(term * D + i) * PREP_PITCH + j] = hb;
                x -= bf16_bits_to_float(hb);
            }
        }
    }
    const int n_heads = is_key ? P.c.n_kv : P.c.n_q;
    const unsigned short* src = is_key ? P.K_new : P.Q_new;
    // the transform stays in shared memory while the CTA walks over its token tiles
    for (int tok0 = blockIdx.x * PREP_TOK; tok0 < P.total_new; tok0 += gridDim.x * PREP_TOK) {
    __syncthreads();                                      // the previous tile's rows have been consumed
    for (int item = tid; item < PREP_TOK * 16; item += 256) {
        const int r = item >> 4, piece = item & 15, tok = tok0 + r;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (tok < P.total_new) v = __ldg(reinterpret_cast<const uint4*>(src + (static_cast<long long>(tok) * n_heads + head) * D + 8 * piece));
        *reinterpret_cast<uint4*>(Xs + r * PREP_PITCH + 8 * piece) = v;
    }
    if (is_key) {                                         // the chunk's values as fp16 (no transform)
        for (int item = tid; item < PREP_TOK * 16; item += 256) {
            const int r = item >> 4, piece = item & 15, tok = tok0 + r;
            if (tok < P.total_new) {
                const long long off = (static_cast<long long>(tok) * P.c.n_kv + head) * D + 8 * piece;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(P.V_new + off));
                const unsigned w[4] = {v.x, v.y, v.z, v.w};
                unsigned o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) o[e] = pack_half2(bf16_bits_to_float(w[e] & 0xffff), bf16_bits_to_float(w[e] >> 16));
                *reinterpret_cast<uint4*>(P.VP + off) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
    __syncthreads();
    if (P.pro.rope) {
        // Projected keys / queries: normalise and rotate the staged rows in place (Algorithm 2 lines 1-2, fp32, one rounding
        // to bf16).  Two threads share a row: thread u of the pair owns channels 32u .. 32u+31 and their rotation
        // partners 64+32u .. 64+32u+31.
        const int row = tid >> 1, u = tid & 1, tok = tok0 + row;
        unsigned short* xa = Xs + row * PREP_PITCH + 32 * u;
        unsigned short* xb = xa + 64;
        float a[32], b[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) { a[k] = bf16_bits_to_float(xa[k]); b[k] = bf16_bits_to_float(xb[k]); }
        if (P.pro.normalise) {
            float ss = 0.f;
#pragma unroll
            for (int k = 0; k < 32; ++k) ss = fmaf(a[k], a[k], fmaf(b[k], b[k], ss));
            ss += __shfl_xor_sync(FULLM, ss, 1);
            const float rn = ss > 0.f ? 1.f / sqrtf(ss * (1.f / D) + P.pro.eps) : 0.f;
            const float* w = is_key ? P.pro.weight : P.q_weight;
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                const float wa = w ? __ldg(w + static_cast<long long>(head) * D + 32 * u + k) : 1.f;
                const float wb = w ? __ldg(w + static_cast<long long>(head) * D + 64 + 32 * u + k) : 1.f;
                a[k] *= rn * wa; b[k] *= rn * wb;
            }
        }
        int pos = 0;
        if (tok < P.total_new) {                           // position of the token: its sequence's length before the chunk + its index
            int lo = 0, hi = P.batch;
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (__ldg(P.cu_new + mid) <= tok) lo = mid; else hi = mid; }
            const int f0 = __ldg(P.cu_new + lo), n_b = __ldg(P.cu_new + lo + 1) - f0;
            pos = __ldg(P.seq_len + lo) - n_b + (tok - f0);
        }
        pos = prologue_position(P.pro, pos, P.c.dev_status, u == 0 && tok < P.total_new);
        const float2* tab = P.pro.rope + static_cast<long long>(pos) * (D / 2) + 32 * u;
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const float2 cs = __ldg(tab + k);
            xa[k] = float_to_bf16_bits(fmaf(a[k], cs.x, -b[k] * cs.y));
            xb[k] = float_to_bf16_bits(fmaf(a[k], cs.y, b[k] * cs.x));
        }
        __syncthreads();
    }
    // warp w: token rows 16w .. 16w+15, all 128 output channels
    float acc[16][4];
#pragma unroll
    for (int nb = 0; nb < 16; ++nb) acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        unsigned a0, a1, a2, a3;
        ldsm_x4(smem_addr(Xs + (16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * PREP_PITCH + 16 * ks + 8 * (lane >> 4)), a0, a1, a2, a3);
        for (int term = 0; term < n_terms; ++term) {
            const unsigned short* Tt = Ts + term * D * PREP_PITCH;
#pragma unroll
            for (int nb2 = 0; nb2 < 8; ++nb2) {           // two output-channel blocks of 8 per ldmatrix.x4
                unsigned b0, b1, b2, b3;
                ldsm_x4(smem_addr(Tt + (16 * nb2 + 8 * (lane >> 4) + (lane & 7)) * PREP_PITCH + 16 * ks + 8 * ((lane >> 3) & 1)), b0, b1, b2, b3);
                mma_bf16_prep(acc[2 * nb2], a0, a1, a2, a3, b0, b1);
                mma_bf16_prep(acc[2 * nb2 + 1], a0, a1, a2, a3, b2, b3);
            }
        }
    }
    // fragment: acc[nb][0..1] = row g, channels 8nb + 2t, +1; acc[nb][2..3] = row g + 8
    const int tok_a = tok0 + 16 * warp + g, tok_b = tok_a + 8;
    float sum_a = 0.f, sum_b = 0.f;
#pragma unroll
    for (int nb = 0; nb < 16; ++nb) {
        const int ch = 8 * nb + 2 * t;
        if (is_key) {                                     // the cache holds bf16(k')
            const unsigned wa = pack_half2(bf16_bits_to_float(float_to_bf16_bits(acc[nb][0])), bf16_bits_to_float(float_to_bf16_bits(acc[nb][1])));
            const unsigned wb = pack_half2(bf16_bits_to_float(float_to_bf16_bits(acc[nb][2])), bf16_bits_to_float(float_to_bf16_bits(acc[nb][3])));
            if (tok_a < P.total_new) *reinterpret_cast<unsigned*>(P.KP + (static_cast<long long>(tok_a) * n_heads + head) * D + ch) = wa;
            if (tok_b < P.total_new) *reinterpret_cast<unsigned*>(P.KP + (static_cast<long long>(tok_b) * n_heads + head) * D + ch) = wb;
        } else {                                          // q' as fp16 value + fp16 rounding remainder
            float hv[4], lv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                hv[e] = __half2float(__float2half_rn(acc[nb][e]));
                lv[e] = __half2float(__float2half_rn(acc[nb][e] - hv[e]));
            }
            sum_a += (hv[0] + lv[0]) + (hv[1] + lv[1]);
            sum_b += (hv[2] + lv[2]) + (hv[3] + lv[3]);
            const long long lo_off = static_cast<long long>(P.total_new) * n_heads * D;
            if (tok_a < P.total_new) {
                const long long off = (static_cast<long long>(tok_a) * n_heads + head) * D + ch;
                *reinterpret_cast<unsigned*>(P.QP + off) = pack_half2(hv[0], hv[1]);
                *reinterpret_cast<unsigned*>(P.QP + lo_off + off) = pack_half2(lv[0], lv[1]);
            }
            if (tok_b < P.total_new) {
                const long long off = (static_cast<long long>(tok_b) * n_heads + head) * D + ch;
                *reinterpret_cast<unsigned*>(P.QP + off) = pack_half2(hv[2], hv[3]);
                *reinterpret_cast<unsigned*>(P.QP + lo_off + off) = pack_half2(lv[2], lv[3]);
            }
        }
    }
    if (!is_key) {                                        // sum of the two-term q' over the 128 channels
        sum_a += __shfl_xor_sync(FULLM, sum_a, 1); sum_a += __shfl_xor_sync(FULLM, sum_a, 2);
        sum_b += __shfl_xor_sync(FULLM, sum_b, 1); sum_b += __shfl_xor_sync(FULLM, sum_b, 2);
        if (t == 0) {
            if (tok_a < P.total_new) P.qsum[static_cast<long long>(tok_a) * P.c.n_q + head] = sum_a;
            if (tok_b < P.total_new) P.qsum[static_cast<long long>(tok_b) * P.c.n_q + head] = sum_b;
        }
    }
    }
}

// ------------------------------------------------------------------------------------------------
// 2. attention
// ------------------------------------------------------------------------------------------------
struct TileSmem {
    __half Q[2][BM][TILE_PITCH];   // the CTA's query rows: fp16 value and rounding remainder of q'
    __half K[BN][TILE_PITCH];
    __half V[BN][TILE_PITCH];
    float4 meta[BN];          // per key: Delta_k, x_min_k, Delta_v, x_min_v (1, 0, 1, 0 for a full-precision row)
    int pos[BN];              // cached position of the key, -1: not a key of this tile
    unsigned char raw[8704];  // one packed record
};

template <int BITS>
__global__ void __launch_bounds__(PF_THREADS) prefill_attn_kernel(PrefillParams P) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    TileSmem& ts = *reinterpret_cast<TileSmem*>(smem_raw);
    const CacheView& c = P.c;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int qt = blockIdx.x % P.tiles_per_seq, b = blockIdx.x / P.tiles_per_seq;
    const int jq = blockIdx.y, h = jq / c.G;
    const int first = __ldg(P.cu_new + b), n_new = __ldg(P.cu_new + b + 1) - first;
    if (qt * BM >= n_new) return;
    const int S = __ldg(P.seq_len + b), sl = __ldg(P.slot + b);
    if (sl < 0 || sl >= c.n_slots || S < n_new) {
        if (tid == 0) atomicOr(c.dev_status, WUSHKV_DEV_BAD_SLOT);
        return;
    }
    const int S0 = S - n_new;                                   // first position of the chunk
    // ---- where older positions are read from (window rule at length S - lag, Section 4.4)
    const int nq = n_quantized(S - c.lag, c.s_sink, c.s_keep, c.s_flush);
    const int q_lo = c.s_sink, q_hi = min(c.s_sink + nq, S0);   // quantized positions below the chunk
    const int a_hi = min(c.s_sink, S0);                         // sink positions below the chunk: [0, a_hi)
    const int c_lo = max(q_hi, a_hi);                           // recent-window positions below the chunk: [c_lo, S0)
    const int n_old_fp = a_hi + max(S0 - c_lo, 0);              // full-precision old positions, as one index space
    const float k2 = c.sm_scale * LOG2E_F;

    // ---- this warp's 16 query rows as A fragments (kept in registers), and their channel sums
    const int row0 = qt * BM + warp * 16;                       // chunk-relative row of fragment row 0
    const int ra = min(row0 + g, n_new - 1), rb = min(row0 + g + 8, n_new - 1);
    for (int item = tid; item < 2 * BM * 16; item += PF_THREADS) {       // 16-byte pieces of the query rows (rows past the chunk: the last row again)
        const int part = item / (BM * 16), r = (item >> 4) % BM, piece = item & 15;
        const int row = min(qt * BM + r, n_new - 1);
        const __half* src = P.QP + static_cast<long long>(part) * P.total_new * c.n_q * D + (static_cast<long long>(first + row) * c.n_q + jq) * D + 8 * piece;
        *reinterpret_cast<uint4*>(&ts.Q[part][r][8 * piece]) = __ldcg(reinterpret_cast<const uint4*>(src));
    }
    const float qs_a = __ldcg(P.qsum + static_cast<long long>(first + ra) * c.n_q + jq);
    const float qs_b = __ldcg(P.qsum + static_cast<long long>(first + rb) * c.n_q + jq);
    const int pos_a = S0 + row0 + g, pos_b = pos_a + 8;         // cached positions of the two rows (causal limit)

    float o[16][4];
#pragma unroll
    for (int nb = 0; nb < 16; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f, z_a = 0.f, z_b = 0.f;

    // One staged tile: scores, online softmax, value reduction.
    auto consume = [&]() {
        float s[8][4];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            unsigned ah[4], al[4];                              // this warp's 16 rows x 16 channels: value, remainder
            const int qrow = 16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1), qcol = 16 * ks + 8 * (lane >> 4);
            ldsm_x4(smem_addr(&ts.Q[0][qrow][qcol]), ah[0], ah[1], ah[2], ah[3]);
            ldsm_x4(smem_addr(&ts.Q[1][qrow][qcol]), al[0], al[1], al[2], al[3]);
#pragma unroll
            for (int nb2 = 0; nb2 < 4; ++nb2) {                 // two key blocks of 8 per ldmatrix.x4
                unsigned b0, b1, b2, b3;
                ldsm_x4(smem_addr(&ts.K[16 * nb2 + 8 * (lane >> 4) + (lane & 7)][16 * ks + 8 * ((lane >> 3) & 1)]), b0, b1, b2, b3);
                hmma(s[2 * nb2], ah[0], ah[1], ah[2], ah[3], b0, b1);
                hmma(s[2 * nb2 + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
                hmma(s[2 * nb2], al[0], al[1], al[2], al[3], b0, b1);
                hmma(s[2 * nb2 + 1], al[0], al[1], al[2], al[3], b2, b3);
            }
        }
        // affine part, masks, row maxima (log2 domain)
        float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int col = 8 * nb + 2 * t + e;
                const float4 mt = ts.meta[col];
                const int kp = ts.pos[col];
                const float va = (kp >= 0 && kp <= pos_a) ? k2 * fmaf(mt.y, qs_a, mt.x * s[nb][e]) : -INFINITY;
                const float vb = (kp >= 0 && kp <= pos_b) ? k2 * fmaf(mt.y, qs_b, mt.x * s[nb][2 + e]) : -INFINITY;
                s[nb][e] = va; s[nb][2 + e] = vb;
                mx_a = fmaxf(mx_a, va); mx_b = fmaxf(mx_b, vb);
            }
        }
        mx_a = fmaxf(mx_a, __shfl_xor_sync(FULLM, mx_a, 1)); mx_a = fmaxf(mx_a, __shfl_xor_sync(FULLM, mx_a, 2));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(FULLM, mx_b, 1)); mx_b = fmaxf(mx_b, __shfl_xor_sync(FULLM, mx_b, 2));
        const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
        const float ref_a = mn_a == -INFINITY ? 0.f : mn_a, ref_b = mn_b == -INFINITY ? 0.f : mn_b;
        const float al_a = fast_ex2(m_a - ref_a), al_b = fast_ex2(m_b - ref_b);     // old reference -inf: state is zero, factor 0
        m_a = mn_a; m_b = mn_b;
        l_a *= al_a; z_a *= al_a; l_b *= al_b; z_b *= al_b;
#pragma unroll
        for (int nb = 0; nb < 16; ++nb) { o[nb][0] *= al_a; o[nb][1] *= al_a; o[nb][2] *= al_b; o[nb][3] *= al_b; }
        unsigned pa[4][4];                                      // A fragments of (p Delta_v) for the four 16-key steps
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            float w[4];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float4 mt = ts.meta[8 * nb + 2 * t + e];
                const float p0 = fast_ex2(s[nb][e] - ref_a), p1 = fast_ex2(s[nb][2 + e] - ref_b);
                l_a += p0; l_b += p1;
                z_a = fmaf(p0, mt.w, z_a); z_b = fmaf(p1, mt.w, z_b);
                w[e] = p0 * mt.z; w[2 + e] = p1 * mt.z;
            }
            pa[nb >> 1][(nb & 1) * 2 + 0] = pack_half2(w[0], w[1]);
            pa[nb >> 1][(nb & 1) * 2 + 1] = pack_half2(w[2], w[3]);
        }
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
#pragma unroll
            for (int nb2 = 0; nb2 < 8; ++nb2) {                 // two channel blocks of 8 per ldmatrix.x4.trans
                unsigned b0, b1, b2, b3;
                ldsm_x4_t(smem_addr(&ts.V[16 * kb + 8 * ((lane >> 3) & 1) + (lane & 7)][16 * nb2 + 8 * (lane >> 4)]), b0, b1, b2, b3);
                hmma(o[2 * nb2], pa[kb][0], pa[kb][1], pa[kb][2], pa[kb][3], b0, b1);
                hmma(o[2 * nb2 + 1], pa[kb][0], pa[kb][1], pa[kb][2], pa[kb][3], b2, b3);
            }
        }
    };

    // ---- (1) full-precision old positions: sink [0, a_hi) and recent window [c_lo, S0), bf16 rows
    for (int base = 0; base < n_old_fp; base += BN) {
        __syncthreads();
        for (int item = tid; item < BN * 16; item += PF_THREADS) {          // 16-byte pieces: 8 channels of one row
            const int r = item >> 4, piece = item & 15, idx = base + r;
            uint4 kh = make_uint4(0, 0, 0, 0), vh = kh;
            if (idx < n_old_fp) {
                const long long plane = (static_cast<long long>(sl) * c.n_kv + h) * 2;
                const unsigned short *ksrc, *vsrc;
                if (idx < a_hi) {
                    ksrc = c.sink_kv + (plane * c.s_sink + idx) * D;
                    vsrc = c.sink_kv + ((plane + 1) * c.s_sink + idx) * D;
                } else {
                    const int p = c_lo + (idx - a_hi);
                    ksrc = c.ring_kv + (plane * c.ring_cap + p % c.ring_cap) * D;
                    vsrc = c.ring_kv + ((plane + 1) * c.ring_cap + p % c.ring_cap) * D;
                }
                const uint4 kb16 = *reinterpret_cast<const uint4*>(ksrc + 8 * piece), vb16 = *reinterpret_cast<const uint4*>(vsrc + 8 * piece);
                const unsigned kw[4] = {kb16.x, kb16.y, kb16.z, kb16.w}, vw[4] = {vb16.x, vb16.y, vb16.z, vb16.w};
                unsigned ko[4], vo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    ko[e] = pack_half2(bf16_bits_to_float(kw[e] & 0xffff), bf16_bits_to_float(kw[e] >> 16));
                    vo[e] = pack_half2(bf16_bits_to_float(vw[e] & 0xffff), bf16_bits_to_float(vw[e] >> 16));
                }
                kh = make_uint4(ko[0], ko[1], ko[2], ko[3]); vh = make_uint4(vo[0], vo[1], vo[2], vo[3]);
            }
            *reinterpret_cast<uint4*>(&ts.K[r][8 * piece]) = kh;
            *reinterpret_cast<uint4*>(&ts.V[r][8 * piece]) = vh;
            if (piece == 0) {
                ts.meta[r] = make_float4(1.f, 0.f, 1.f, 0.f);
                ts.pos[r] = idx < n_old_fp ? (idx < a_hi ? idx : c_lo + (idx - a_hi)) : -1;
            }
        }
        __syncthreads();
        consume();
    }

    // ---- (2) quantized positions below the chunk: one packed page per tile, staged as integer codes
    if (q_hi > q_lo) {
        constexpr int REC = record_bytes(BITS);
        const int page_first = q_lo / PAGE_TOKENS, page_last = (q_hi - 1) / PAGE_TOKENS;
        for (int pg = page_first; pg <= page_last; ++pg) {
            __syncthreads();
            int page = -1;
            if (pg < c.max_pages) page = __ldg(c.page_table + static_cast<long long>(sl) * c.max_pages + pg);
            const bool page_ok = page >= 0 && page < c.n_pages;
            if (!page_ok && tid == 0) atomicOr(c.dev_status, pg < c.max_pages ? WUSHKV_DEV_BAD_PAGE_ID : WUSHKV_DEV_PAGE_TABLE_FULL);
            if (page_ok) {
                const uint4* src = reinterpret_cast<const uint4*>(c.pages + (static_cast<long long>(page) * c.n_kv + h) * REC);
                for (int k = tid; k < REC / 16; k += PF_THREADS) reinterpret_cast<uint4*>(ts.raw)[k] = __ldg(src + k);
            }
            __syncthreads();
            // thread -> token r = tid & 63, channels (tid >> 6) * 64 .. + 63, two at a time
            {
                const int r = tid & 63, ch0 = (tid >> 6) * 64;
                const int pos = pg * PAGE_TOKENS + r;
                const bool live = page_ok && pos >= q_lo && pos < q_hi;
                constexpr unsigned MASK = (1u << (BITS == 3 ? 2 : BITS)) - 1u;       // 3 bits: low two here, third bit below
                auto field_at = [&](int off, int bit, unsigned mask) { return (static_cast<unsigned>(ts.raw[off + (bit >> 3)]) >> (bit & 7)) & mask; };
                for (int ch = ch0; ch < ch0 + 64; ch += 2) {
                    float k0 = 0.f, k1 = 0.f, v0 = 0.f, v1 = 0.f;
                    if (live) {
                        int off, bit;
                        unsigned ck[2], cv[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            k_code_location(BITS, r, ch + e, off, bit); ck[e] = field_at(off, bit, MASK);
                            v_code_location(BITS, r, ch + e, off, bit); cv[e] = field_at(off, bit, MASK);
                            if (BITS == 3) {
                                k_hi_location(r, ch + e, off, bit); ck[e] |= field_at(off, bit, 1u) << 2;
                                v_hi_location(r, ch + e, off, bit); cv[e] |= field_at(off, bit, 1u) << 2;
                            }
                        }
                        k0 = static_cast<float>(ck[0]); k1 = static_cast<float>(ck[1]);
                        v0 = static_cast<float>(cv[0]); v1 = static_cast<float>(cv[1]);
                    }
                    *reinterpret_cast<unsigned*>(&ts.K[r][ch]) = pack_half2(k0, k1);
                    *reinterpret_cast<unsigned*>(&ts.V[r][ch]) = pack_half2(v0, v1);
                }
                if (ch0 == 0) {
                    float4 mt = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (live) {
                        const __half* mh = reinterpret_cast<const __half*>(ts.raw + meta_location(BITS, r));
                        mt = make_float4(__half2float(mh[0]), __half2float(mh[1]), __half2float(mh[2]), __half2float(mh[3]));
                    }
                    ts.meta[r] = mt;
                    ts.pos[r] = live ? pos : -1;
                }
            }
            __syncthreads();
            consume();
        }
    }

    // ---- (3) the chunk itself, causal: tiles 0 .. qt of its own rows (fp16 copies made by the preparation kernel)
    for (int kt = 0; kt <= qt; ++kt) {
        __syncthreads();
        for (int item = tid; item < BN * 16; item += PF_THREADS) {
            const int r = item >> 4, piece = item & 15, row = kt * BN + r;
            uint4 kh = make_uint4(0, 0, 0, 0), vh = kh;
            if (row < n_new) {
                const long long off = (static_cast<long long>(first + row) * c.n_kv + h) * D + 8 * piece;
                kh = __ldcg(reinterpret_cast<const uint4*>(P.KP + off));
                vh = __ldcg(reinterpret_cast<const uint4*>(P.VP + off));
            }
            *reinterpret_cast<uint4*>(&ts.K[r][8 * piece]) = kh;
            *reinterpret_cast<uint4*>(&ts.V[r][8 * piece]) = vh;
            if (piece == 0) {
                ts.meta[r] = make_float4(1.f, 0.f, 1.f, 0.f);
                ts.pos[r] = row < n_new ? S0 + row : -1;
            }
        }
        __syncthreads();
        consume();
    }

    // ---- output: o_i = (sum_j p_ij v_hat_j) / sum_j p_ij
    l_a += __shfl_xor_sync(FULLM, l_a, 1); l_a += __shfl_xor_sync(FULLM, l_a, 2);
    l_b += __shfl_xor_sync(FULLM, l_b, 1); l_b += __shfl_xor_sync(FULLM, l_b, 2);
    z_a += __shfl_xor_sync(FULLM, z_a, 1); z_a += __shfl_xor_sync(FULLM, z_a, 2);
    z_b += __shfl_xor_sync(FULLM, z_b, 1); z_b += __shfl_xor_sync(FULLM, z_b, 2);
    const float inv_a = l_a > 0.f ? 1.f / l_a : 0.f, inv_b = l_b > 0.f ? 1.f / l_b : 0.f;
    if (row0 + g < n_new) {
        float* dst = P.O + (static_cast<long long>(first + row0 + g) * c.n_q + jq) * D;
#pragma unroll
        for (int nb = 0; nb < 16; ++nb)
            *reinterpret_cast<float2*>(dst + 8 * nb + 2 * t) = make_float2((o[nb][0] + z_a) * inv_a, (o[nb][1] + z_a) * inv_a);
    }
    if (row0 + g + 8 < n_new) {
        float* dst = P.O + (static_cast<long long>(first + row0 + g + 8) * c.n_q + jq) * D;
#pragma unroll
        for (int nb = 0; nb < 16; ++nb)
            *reinterpret_cast<float2*>(dst + 8 * nb + 2 * t) = make_float2((o[nb][2] + z_b) * inv_b, (o[nb][3] + z_b) * inv_b);
    }
}

// ------------------------------------------------------------------------------------------------
// 2b. attention on tcgen05, one tile per CTA (testing aid "prefill_one_tile"; the default before section 2c)
// ------------------------------------------------------------------------------------------------
// One CTA of 128 threads per (sequence, KV head, tile of R = 128 / G chunk positions): the G query heads that
// read the KV head are packed into the M = 128 rows of the tile (row r = position r / G, head r % G), so a staged
// key / value tile serves all of them.  Per 64-key tile:
//   S = Q' K^T     16 x tcgen05.mma.kind::f16, M 128, N 64, K 16 (fp16 value and remainder of q' against the same
//                  keys), fp32 accumulator in tensor memory (64 columns);
//   softmax        thread r reads row r with tcgen05.ld, applies the affine factors and the causal mask, keeps a
//                  lazily raised reference (the accumulator row in tensor memory is rescaled only when the row
//                  maximum grows by more than 2^6) and writes (p Delta_v) as fp16 into the A-operand layout;
//   O += P V       4 x tcgen05.mma, M 128, N 128, K 16, the value tile as an MN-major B operand, accumulator in
//                  tensor memory (128 columns).
// Operands use the no-swizzle canonical layouts: K-major tiles (Q', K, P) as 8-row x 16-byte core matrices at
// (row / 8) * SBO + (k / 8) * 128 + (row % 8) * 16; the MN-major value tile as 8-key x 16-byte core matrices at
// (channel / 8) * SBO + (key / 8) * 128 + (key % 8) * 16.  Every wait on the MMA barrier is bounded.
constexpr int TM = 128;                       // rows of the packed query tile
constexpr int TN = 64;                        // keys per tile (= one packed page)
constexpr int TC_Q_BYTES = TM * D * 2;        // one fp16 query operand
constexpr int TC_K_BYTES = TN * D * 2;        // key tile; reused for P (TM x TN fp16 is the same size)
constexpr int TC_OFF_Q = 0;
constexpr int TC_OFF_K = 2 * TC_Q_BYTES;
constexpr int TC_OFF_V = TC_OFF_K + TC_K_BYTES;                // two value tiles (the next one is staged while the current one is read)
constexpr int TC_OFF_META = TC_OFF_V + 2 * TC_K_BYTES;         // uint2[TN]: four fp16 per key
constexpr int TC_OFF_POS = TC_OFF_META + TN * 8;               // int[TN]
constexpr int TC_OFF_BAR = TC_OFF_POS + TN * 4;                // barriers, tensor-memory slot
constexpr int TC_SMEM = TC_OFF_BAR + 64;                      // [0] score-MMA barrier, [8] tensor-copy barrier, [16] tensor-memory slot, [24] P V barrier
static_assert(2 * (TC_SMEM + 1024) <= 233472, "two CTAs per SM");
static_assert(8704 <= TC_K_BYTES, "a packed record is staged in the idle value buffer");
static_assert(TC_OFF_K % 1024 == 0 && TC_OFF_V % 1024 == 0, "swizzled tiles need 1024-byte alignment");
constexpr float REF_SLACK = 6.f;              // log2 headroom of the lazily raised softmax reference
constexpr unsigned TC_TMEM_COLS = 256;        // O: columns 0..127, S: columns 128..191, P (fp16 pairs): columns 192..223
constexpr unsigned TC_IDESC_S = (1u << 4) | ((TN >> 3) << 17) | ((TM >> 4) << 24);                  // fp32 <- fp16 x fp16, both K-major
constexpr unsigned TC_IDESC_O = (1u << 4) | (1u << 16) | ((D >> 3) << 17) | ((TM >> 4) << 24);      // B (values) MN-major

__device__ __forceinline__ unsigned long long tc_desc(unsigned addr, unsigned lbo, unsigned sbo) {
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((addr >> 4) & 0x3FFFu);
    d |= static_cast<unsigned long long>((lbo >> 4) & 0x3FFFu) << 16;
    d |= static_cast<unsigned long long>((sbo >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    return d;
}
// the same for a tile in the 128-byte-swizzled canonical layout (rows of 128 bytes, as a bulk tensor copy writes them)
__device__ __forceinline__ unsigned long long tc_desc_sw128(unsigned addr, unsigned lbo, unsigned sbo) { return tc_desc(addr, lbo, sbo) | (2ull << 61); }
__device__ __forceinline__ void tma_load_3d(unsigned dst, const CUtensorMap* map, int c0, int c1, int c2, unsigned bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(unsigned tmem, unsigned long long adesc, unsigned long long bdesc, unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same with the A operand in tensor memory (lane = row, a 32-bit column = two consecutive K elements)
__device__ __forceinline__ void tc_mma_ts(unsigned tmem_d, unsigned tmem_a, unsigned long long bdesc, unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_st32u(unsigned taddr, const unsigned (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
          "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]),
          "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tc_st16u(unsigned taddr, const unsigned (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
          "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tc_ld32(unsigned taddr, float (&v)[32]) {
    unsigned r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// two 32-column loads in flight before the one wait
__device__ __forceinline__ void tc_ld64(unsigned taddr, float (&v)[64]) {
    unsigned r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]),
          "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]),
          "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]),
          "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr + 32u) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st32(unsigned taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
          "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
          "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
          "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
          "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
          "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
          "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
__device__ __forceinline__ void cp16(unsigned dst, const void* src, unsigned bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

// Eight consecutive channels 8 kc .. 8 kc + 7 of token r of a packed record as fp16 integers (keys and values), read
// with 16-bit loads straight from the fragment-ordered layout (csrc/layout.cuh): a key half-word holds the two
// channels 8 kc + 2 t, + 1 of fragment lane t; a value half-word holds the code fields of one channel for all channel
// blocks.  Two codes c0, c1 become an fp16 pair by (c0 | c1 << 16 | 0x64006400) - (1024, 1024).
__device__ __forceinline__ float2 h2f2u(unsigned u) { return __half22float2(*reinterpret_cast<const __half2*>(&u)); }

template <int BITS>
__device__ __forceinline__ void unpack_chunk8(const unsigned char* raw, int r, int kc, uint4& kout, uint4& vout) {
    constexpr bool TWO = BITS != 4;                       // 2-bit fields (also the low plane of 3-bit records)
    constexpr unsigned MASK = TWO ? 3u : 15u;
    const int bi = r >> 4, rr = r & 15;
    const __half2 bias = __halves2half2(__ushort_as_half(0x6400), __ushort_as_half(0x6400));
    auto to_h2 = [&](unsigned c0, unsigned c1) {
        const unsigned w = c0 | (c1 << 16) | 0x64006400u;
        const __half2 h = __hsub2(*reinterpret_cast<const __half2*>(&w), bias);
        return *reinterpret_cast<const unsigned*>(&h);
    };
    unsigned ko[4], vo[4];
    {   // keys: token row -> (g, rs); chunk -> k-step s, channel half hh, byte pair bh
        const int g = rr & 7, rs = rr >> 3, s4 = kc >> 2, hh = (kc >> 1) & 1, bh = kc & 1, j = rs + 2 * hh;
        const int base = bi * code_block_bytes(BITS) + (TWO ? 0 : 512 * (s4 >> 1)) + 64 * g + 4 * j + 2 * bh;
        const int sh = TWO ? 2 * s4 : 4 * (s4 & 1);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const unsigned x = *reinterpret_cast<const unsigned short*>(raw + base + 16 * t);
            unsigned c0 = (x >> sh) & MASK, c1 = (x >> (8 + sh)) & MASK;
            if (BITS == 3) {
                const unsigned y = *reinterpret_cast<const unsigned short*>(raw + k_hi_offset(3) + bi * 256 + 8 * (4 * g + t) + 4 * rs + 2 * bh);
                c0 |= ((y >> (2 * s4 + hh)) & 1u) << 2;
                c1 |= ((y >> (8 + 2 * s4 + hh)) & 1u) << 2;
            }
            ko[t] = to_h2(c0, c1);
        }
    }
    {   // values: token -> (ps, t, hi); chunk -> channel block i, row half rsel; channel e of the chunk is fragment row g = e
        const int ps = rr >> 3, tt = (rr & 7) >> 1, hi = rr & 1, i = kc >> 1, rsel = kc & 1;
        const int base = v_codes_offset(BITS) + bi * code_block_bytes(BITS) + (TWO ? 4 * (2 * ps + rsel) : 512 * ps + 4 * (2 * rsel + (i >> 2))) + 16 * tt + 2 * hi;
        const int sh = TWO ? 2 * i : 4 * (i & 3);
        unsigned cv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const unsigned x = *reinterpret_cast<const unsigned short*>(raw + base + 64 * e);
            cv[e] = (x >> sh) & MASK;
            if (BITS == 3) {
                const unsigned y = *reinterpret_cast<const unsigned short*>(raw + v_hi_offset(3) + bi * 256 + 8 * (4 * e + tt) + 4 * ps + 2 * hi);
                cv[e] |= ((y >> v1_bit(rsel, i)) & 1u) << 2;
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) vo[e] = to_h2(cv[2 * e], cv[2 * e + 1]);
    }
    kout = make_uint4(ko[0], ko[1], ko[2], ko[3]);
    vout = make_uint4(vo[0], vo[1], vo[2], vo[3]);
}

// A whole page (all 64 tokens live) as fp16 key codes and fp16 values, by 128 threads: instead of gathering eight channels of a token
// from 16-bit loads (unpack_chunk8), a thread reads the record the way it is laid out and scatters 16-byte chunks.
//   keys:   thread (block bi, k-step s, fragment row g) loads the four 16-byte pieces of row g (fragment lanes t = 0..3: words
//           j = rs + 2 hh, bytes b = 2 b1 + b0; the field of k-step s in a byte = channel 32 s + 16 hh + 8 b1 + 2 t + b0 of
//           token g + 8 rs) and writes, for (rs, hh, b1), the chunk of channels 8 (4 s + 2 hh + b1) .. + 7 of that token:
//           pair t = (b0 0, 1).  At 4 bits the k-steps 0-1 / 2-3 sit in two 512-byte halves, a nibble each.
//   values: thread (block bi, token half ps, row half rsel, half ih of the channel blocks, token pair tt) loads one word of the
//           eight pieces (e, tt) (half-word hi = token 8 ps + 2 tt + hi, field i = channel 16 i + 8 rsel + e) and writes, for
//           (hi, i in 4 ih .. 4 ih + 3), the chunk of channels 8 (2 i + rsel) .. + 7 of that token: element e.
//   3 bits: the 2-bit plane as above plus the high bit of every code from the 1-bit planes (csrc/layout.cuh).
// Keys are left as integer codes (exact in fp16; their factors are applied to the scores in fp32).  Values are written
// dequantized, step * code + offset in one fp16 rounding: the probabilities that multiply them are fp16 already, and the
// softmax then treats a packed page's values like any other's.
template <int BITS>
__device__ __forceinline__ void unpack_page(const unsigned char* raw, unsigned char* sK, unsigned char* sV, const int p) {
    constexpr bool TWO = BITS != 4;                         // 2-bit fields (also the low plane of 3-bit records)
    constexpr unsigned MASK = TWO ? 3u : 15u, MASK2 = MASK * 0x00010001u;
    constexpr int CB = code_block_bytes(BITS);
    // Two codes that sit at bit f of bytes 0 and 2 of `bytes` -> fp16 pair: (1024 + c 2^f) 2^-f - 1024 2^-f = c, one
    // fused multiply-add (exact: c 2^f < 1024); mul = 2^-f and add = -2^(10 - f) in both halves.  3 bits: `high` holds the
    // codes' third bits, already at bit f + 2 of each half.
    auto field_h2 = [](const unsigned bytes, const unsigned mask, const unsigned high, const unsigned mul, const unsigned add) {
        const unsigned w = (bytes & mask) | 0x64006400u | high;
        const __half2 hv = __hfma2(*reinterpret_cast<const __half2*>(&w), *reinterpret_cast<const __half2*>(&mul),
                                   *reinterpret_cast<const __half2*>(&add));
        return *reinterpret_cast<const unsigned*>(&hv);
    };
    auto pow2_neg = [](const int f) { return (0x3C00u - (static_cast<unsigned>(f) << 10)) * 0x00010001u; };            // 2^-f
    auto bias_neg = [](const int f) { return (0x8000u | (static_cast<unsigned>(25 - f) << 10)) * 0x00010001u; };      // -2^(10 - f)
    {
        const int g = p & 7, s = (p >> 3) & 3, bi = p >> 5;
        const unsigned char* src = raw + bi * CB + (TWO ? 0 : 512 * (s >> 1)) + 64 * g;
        const int sh0 = TWO ? 2 * s : 4 * (s & 1);
        const unsigned kmask = MASK2 << sh0, kmul = pow2_neg(sh0), kadd = bias_neg(sh0), khigh = 0x00010001u << (sh0 + 2);
        unsigned w[4][4];                                   // [t][j]
        unsigned wh[4][2];                                  // 3 bits: [t][rs], bit 2 s + hh of byte b
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint4 v = *reinterpret_cast<const uint4*>(src + 16 * t);
            w[t][0] = v.x; w[t][1] = v.y; w[t][2] = v.z; w[t][3] = v.w;
            if (BITS == 3) {
                const uint2 y = *reinterpret_cast<const uint2*>(raw + k_hi_offset(3) + bi * 256 + 8 * (4 * g + t));
                wh[t][0] = y.x; wh[t][1] = y.y;
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {                       // j = rs + 2 hh
#pragma unroll
            for (int b1 = 0; b1 < 2; ++b1) {
                unsigned out[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    // bytes 2 b1 and 2 b1 + 1 of the word to bytes 0 and 2, then the thread's field of each
                    unsigned high = 0u;
                    if constexpr (BITS == 3)            // the same bytes of the 1-bit plane: bit 2 s + hh of each goes to bit 2 s + 2
                        high = (__byte_perm(wh[t][j & 1], 0u, b1 ? 0x4342u : 0x4140u) << (2 - (j >> 1))) & khigh;
                    out[t] = field_h2(__byte_perm(w[t][j], 0u, b1 ? 0x4342u : 0x4140u), kmask, high, kmul, kadd);
                }
                *reinterpret_cast<uint4*>(sK + (2 * bi + (j & 1)) * 2048 + (4 * s + 2 * (j >> 1) + b1) * 128 + g * 16) =
                    make_uint4(out[0], out[1], out[2], out[3]);
            }
        }
    }
    {
        // (the half-word hi is a lane bit: the eight lanes of a quarter warp then write the eight 16-byte pieces of one 128-byte row)
        const int tt = p & 3, hi = (p >> 2) & 1, m = (p >> 3) & 3, bi = p >> 5, ps = m >> 1, rsel = m & 1;
        const unsigned char* src = raw + v_codes_offset(BITS) + bi * CB + (TWO ? 4 * m : 512 * ps + 8 * rsel) + 16 * tt;
        // the values are staged dequantized: step and offset of this thread's token, in both halves of a pair
        const unsigned mv = *reinterpret_cast<const unsigned*>(raw + meta_location(BITS, 16 * bi + 8 * ps + 2 * tt + hi) + 4);
        const unsigned step2 = __byte_perm(mv, mv, 0x1010u), offs2 = __byte_perm(mv, mv, 0x3232u);
        auto dequant = [&](const unsigned codes) {
            const __half2 hv = __hfma2(*reinterpret_cast<const __half2*>(&codes), *reinterpret_cast<const __half2*>(&step2),
                                       *reinterpret_cast<const __half2*>(&offs2));
            return *reinterpret_cast<const unsigned*>(&hv);
        };
        unsigned wa[TWO ? 1 : 2][8], wh[8];                 // [ih][e] (2-bit fields: one word holds both); 3 bits: the word of token half ps
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            wa[0][e] = *reinterpret_cast<const unsigned*>(src + 64 * e);
            if (!TWO) wa[TWO ? 0 : 1][e] = *reinterpret_cast<const unsigned*>(src + 64 * e + 4);
            if (BITS == 3) wh[e] = *reinterpret_cast<const unsigned*>(raw + v_hi_offset(3) + bi * 256 + 8 * (4 * e + tt) + 4 * ps);
        }
        unsigned hw[4];                                     // 3 bits: this thread's half-word of the 1-bit plane, of the words 2 e2 and 2 e2 + 1
        if constexpr (BITS == 3) {
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2) hw[e2] = __byte_perm(wh[2 * e2], wh[2 * e2 + 1], hi ? 0x7632u : 0x5410u);
        }
#pragma unroll
        for (int ih = 0; ih < 2; ++ih) {                    // half of the channel blocks
            const unsigned (&w)[8] = wa[TWO ? 0 : ih];
#pragma unroll
            for (int ii = 0; ii < 4; ++ii) {
                const int i = 4 * ih + ii;
                // the field's byte (of both words, to bytes 0 and 2: the same for the fields of one byte) and its bit inside it
                const int byte = TWO ? 2 * hi + ih : 2 * hi + (ii >> 1), f = TWO ? 2 * ii : 4 * (ii & 1);
                // bit of the 1-bit plane for (rsel, i): rsel 0: 2 i + 2 (i < 5), 2 i + 1 (else); rsel 1: 2 i + 1 (i < 5), 2 i + 2 (i < 7), 0 (i = 7);
                // a rotation takes it to bit f + 2 of each half
                const int hb = rsel == 0 ? (i < 5 ? 2 * i + 2 : 2 * i + 1) : (i < 5 ? 2 * i + 1 : (i < 7 ? 2 * i + 2 : 0));
                unsigned out[4];
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    unsigned high = 0u;
                    if constexpr (BITS == 3) high = __funnelshift_r(hw[e2], hw[e2], (hb - (f + 2)) & 31) & (0x00010001u << (f + 2));
                    const unsigned both = __byte_perm(w[2 * e2], w[2 * e2 + 1], 0x0400u + 0x0101u * static_cast<unsigned>(byte));
                    out[e2] = dequant(field_h2(both, MASK2 << f, high, pow2_neg(f), bias_neg(f)));
                }
                *reinterpret_cast<uint4*>(sV + (2 * i + rsel) * 1024 + (2 * bi + ps) * 128 + (2 * tt + hi) * 16) =
                    make_uint4(out[0], out[1], out[2], out[3]);
            }
        }
    }
}

template <int BITS>
__global__ void __launch_bounds__(TM, 2) prefill_attn_tc_kernel(PrefillParams P, const __grid_constant__ CUtensorMap map_k,
                                                                 const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ __align__(1024) unsigned char sm_tc[];
    const CacheView& c = P.c;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int G = c.G, R = TM / G;                              // chunk positions per tile
    const int qt = P.tiles_per_seq - 1 - static_cast<int>(blockIdx.x % P.tiles_per_seq);      // long tiles first
    const int b = blockIdx.x / P.tiles_per_seq, h = blockIdx.y;
    const int first = __ldg(P.cu_new + b), n_new = __ldg(P.cu_new + b + 1) - first;
    if (qt * R >= n_new) return;
    const int S = __ldg(P.seq_len + b), sl = __ldg(P.slot + b);
    if (sl < 0 || sl >= c.n_slots || S < n_new) {
        if (tid == 0) atomicOr(c.dev_status, WUSHKV_DEV_BAD_SLOT);
        return;
    }
    unsigned char* sQ = sm_tc + TC_OFF_Q;
    unsigned char* sK = sm_tc + TC_OFF_K;
    unsigned char* sVb = sm_tc + TC_OFF_V;                      // two value buffers; `vb` selects the one of the tile being staged / consumed
    int vb = 0;
    uint2* meta = reinterpret_cast<uint2*>(sm_tc + TC_OFF_META);
    int* kpos = reinterpret_cast<int*>(sm_tc + TC_OFF_POS);
    unsigned long long* mbar = reinterpret_cast<unsigned long long*>(sm_tc + TC_OFF_BAR);
    const unsigned obar = smem_addr(sm_tc + TC_OFF_BAR + 24);    // completion of O += P V of a tile
    unsigned ophase = 0;
    bool pv_pending = false;
    const uint2 META_PLAIN = make_uint2(0x00003C00u, 0x00003C00u);   // (1, 0, 1, 0) as fp16: a full-precision key
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(sm_tc + TC_OFF_BAR + 16);
    const unsigned tbar = smem_addr(sm_tc + TC_OFF_BAR + 8);     // completion of the bulk tensor copies of a tile
    unsigned tphase = 0;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(mbar)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tbar) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(obar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int S0 = S - n_new;
    const int nq = n_quantized(S - c.lag, c.s_sink, c.s_keep, c.s_flush);
    const int q_lo = c.s_sink, q_hi = min(c.s_sink + nq, S0);
    const int a_hi = min(c.s_sink, S0);
    const int c_lo = max(q_hi, a_hi);
    const int n_old_fp = a_hi + max(S0 - c_lo, 0);
    const float k2 = c.sm_scale * LOG2E_F;

    // ---- the packed query tile: row r = chunk position qt R + r / G (clamped to the chunk), head h G + r % G
    const int n_rows = min(R, n_new - qt * R) * G;              // rows that carry a query
    for (int item = tid; item < 2 * TM * 16; item += TM) {
        const int part = item / (TM * 16), r = (item >> 4) % TM, piece = item & 15;
        const int rr = min(r, n_rows - 1);
        const int tok = first + qt * R + rr / G, jq = h * G + rr % G;
        const __half* src = P.QP + static_cast<long long>(part) * P.total_new * c.n_q * D + (static_cast<long long>(tok) * c.n_q + jq) * D + 8 * piece;
        cp16(smem_addr(sQ + part * TC_Q_BYTES + (r >> 3) * 2048 + piece * 128 + (r & 7) * 16), src, 16u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    const int my_r = min(tid, n_rows - 1);
    const int my_tok = first + qt * R + my_r / G, my_jq = h * G + my_r % G;
    const float my_qsum = __ldcg(P.qsum + static_cast<long long>(my_tok) * c.n_q + my_jq);
    const int my_pos = S0 + qt * R + my_r / G;                  // causal limit of this thread's row
    const int tile_pos_lo = S0 + qt * R;                        // smallest causal limit of the tile

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;
    const unsigned tmem_row = tmem_base + (static_cast<unsigned>(warp * 32) << 16);
    unsigned phase = 0;
    bool failed = false, have_o = false;
    float m_ref = -INFINITY, l = 0.f, z = 0.f;
    const int wait_limit = P.wait_limit > 0 ? P.wait_limit : (1 << 24);      // polls of at least ~60 ns each: a second or more
    bool first_tile = true;

    auto wait_mma = [&]() -> bool {                             // bounded; the decision is uniform for the CTA
        bool done = false;
        for (int it = 0; it < wait_limit && !done; ++it) {       // short suspensions: the MMAs of a tile take about a microsecond
            unsigned ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(smem_addr(mbar)), "r"(phase), "r"(64u) : "memory");
            done = ok != 0;
        }
        if (!__syncthreads_and(done ? 1 : 0)) return false;
        phase ^= 1u;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        return true;
    };

    // O += P V of the previous tile is only awaited where its operands or its accumulator are needed again
    auto drain_pv = [&]() -> bool {
        if (!pv_pending) return true;
        bool done = false;
        for (int it = 0; it < wait_limit && !done; ++it) {
            unsigned ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(obar), "r"(ophase), "r"(64u) : "memory");
            done = ok != 0;
        }
        pv_pending = false;
        ophase ^= 1u;
        if (!__syncthreads_and(done ? 1 : 0)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        return true;
    };

    // One staged tile: S = Q' K^T, softmax of this thread's row, O += P V.  PACKED: the keys carry affine factors
    // (codes of a packed page); MASKED: some key of the tile may be invisible to some row (padding, or a chunk
    // position beyond the row's own).  Full-precision, fully visible tiles (most of a long chunk) take the short form.
    // `swz`: the key / value tile was written by bulk tensor copies (128-byte-swizzled rows, two 64-channel boxes each).
    // `next_row` >= 0: the first token row of the next tile, to be fetched by bulk tensor copies as soon as the scores of
    // this tile are done (the key buffer is free then, the other value buffer has been free since the previous tile).
    auto consume = [&](auto packed_tag, auto masked_tag, const bool swz, const int next_row) {
        constexpr bool PACKED = decltype(packed_tag)::value, MASKED = decltype(masked_tag)::value;
        unsigned char* sV = sVb + vb * TC_K_BYTES;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (swz) {                                             // bounded wait for the tile's bulk copies
            bool done = false;
            for (int it = 0; it < wait_limit && !done; ++it) {
                unsigned ok;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(tbar), "r"(tphase), "r"(64u) : "memory");
                done = ok != 0;
            }
            tphase ^= 1u;
            if (!__syncthreads_and(done ? 1 : 0)) { failed = true; return; }
        } else {
            __syncthreads();
        }
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                // swizzled: channels 0-63 and 64-127 are two boxes of 8 KB; a k-step of 16 channels is 32 bytes inside the 128-byte row
                const unsigned long long bdesc = swz ? tc_desc_sw128(smem_addr(sK) + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024)
                                                     : tc_desc(smem_addr(sK) + ks * 256, 128, 2048);
                tc_mma(tmem_base + 128, tc_desc(smem_addr(sQ) + ks * 256, 128, 2048), bdesc, TC_IDESC_S, ks > 0 ? 1u : 0u);
                tc_mma(tmem_base + 128, tc_desc(smem_addr(sQ + TC_Q_BYTES) + ks * 256, 128, 2048), bdesc, TC_IDESC_S, 1u);
            }
            if (!(P.drop == 1 && first_tile))
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(mbar)) : "memory");
        }
        first_tile = false;
        if (!wait_mma()) { failed = true; return; }
        if (next_row >= 0 && tid == 0) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tbar), "r"(2u * TC_K_BYTES) : "memory");
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                tma_load_3d(smem_addr(sK) + hf * 8192, &map_k, 64 * hf, h, next_row, tbar);
                tma_load_3d(smem_addr(sVb + (vb ^ 1) * TC_K_BYTES) + hf * 8192, &map_v, 64 * hf, h, next_row, tbar);
            }
        }
        // ---- this thread's row of scores (log2 domain after the scaling below)
        float s[TN];
        {
            float lo[32], hi[32];
            tc_ld32(tmem_row + 128, lo);
            tc_ld32(tmem_row + 160, hi);
#pragma unroll
            for (int i = 0; i < 32; ++i) { s[i] = lo[i]; s[32 + i] = hi[i]; }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            float v;
            if (PACKED) { const float2 mk = h2f2u(meta[j].x); v = k2 * fmaf(mk.y, my_qsum, mk.x * s[j]); }
            else v = k2 * s[j];
            if (MASKED) { const int kp = kpos[j]; if (kp < 0 || kp > my_pos) v = -INFINITY; }
            s[j] = v;
            mx = fmaxf(mx, v);
        }
        const bool raise = mx > m_ref + REF_SLACK;                 // also the first finite maximum (m_ref = -inf)
        const float new_ref = raise ? mx : m_ref;
        const float factor = raise ? fast_ex2(m_ref - new_ref) : 1.f;      // old reference -inf: factor 0, state is zero anyway
        if (!drain_pv()) { failed = true; return; }                // the accumulator and the probability columns are free again
        if (__any_sync(FULLM, raise) && have_o) {                  // rescale this warp's accumulator rows in tensor memory
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                float o[32];
                tc_ld32(tmem_row + 32 * q4, o);
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] *= factor;
                tc_st32(tmem_row + 32 * q4, o);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        l *= factor; z *= factor;
        m_ref = new_ref;
        const float ref = m_ref == -INFINITY ? 0.f : m_ref;
        // ---- probabilities: (p Delta_v) as fp16 pairs into tensor memory (columns 192..223), the A operand of O += P V
        unsigned pk[32];
#pragma unroll
        for (int kc = 0; kc < TN / 8; ++kc) {
            float w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float p = fast_ex2(s[8 * kc + e] - ref);
                l += p;
                if (PACKED) { const float2 mv = h2f2u(meta[8 * kc + e].y); z = fmaf(p, mv.y, z); w[e] = p * mv.x; }
                else w[e] = p;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) pk[4 * kc + e] = pack_half2(w[2 * e], w[2 * e + 1]);
        }
        tc_st32u(tmem_row + 192, pk);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int ks = 0; ks < TN / 16; ++ks)     // swizzled values: rows (keys) of 128 bytes, 8-key groups 1024 bytes apart, channel halves 8192 bytes apart
                tc_mma_ts(tmem_base, tmem_base + 192 + 8 * ks,
                          swz ? tc_desc_sw128(smem_addr(sV) + ks * 2048, 8192, 1024) : tc_desc(smem_addr(sV) + ks * 256, 128, 1024), TC_IDESC_O,
                          (have_o || ks > 0) ? 1u : 0u);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(obar) : "memory");
        }
        have_o = true;
        pv_pending = true;                                       // awaited by the next tile (or the epilogue)
        vb ^= 1;
    };

    // ---- (1) full-precision old positions: sink [0, a_hi) and recent window [c_lo, S0), bf16 rows
    for (int base = 0; base < n_old_fp && !failed; base += TN) {
        unsigned char* sV = sVb + vb * TC_K_BYTES;
        for (int item = tid; item < TN * 16; item += TM) {
            const int r = item >> 4, piece = item & 15, idx = base + r;
            uint4 kh = make_uint4(0, 0, 0, 0), vh = kh;
            if (idx < n_old_fp) {
                const long long plane = (static_cast<long long>(sl) * c.n_kv + h) * 2;
                const unsigned short *ksrc, *vsrc;
                if (idx < a_hi) {
                    ksrc = c.sink_kv + (plane * c.s_sink + idx) * D;
                    vsrc = c.sink_kv + ((plane + 1) * c.s_sink + idx) * D;
                } else {
                    const int p = c_lo + (idx - a_hi);
                    ksrc = c.ring_kv + (plane * c.ring_cap + p % c.ring_cap) * D;
                    vsrc = c.ring_kv + ((plane + 1) * c.ring_cap + p % c.ring_cap) * D;
                }
                const uint4 kb16 = *reinterpret_cast<const uint4*>(ksrc + 8 * piece), vb16 = *reinterpret_cast<const uint4*>(vsrc + 8 * piece);
                const unsigned kw[4] = {kb16.x, kb16.y, kb16.z, kb16.w}, vw[4] = {vb16.x, vb16.y, vb16.z, vb16.w};
                unsigned ko[4], vo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    ko[e] = pack_half2(bf16_bits_to_float(kw[e] & 0xffff), bf16_bits_to_float(kw[e] >> 16));
                    vo[e] = pack_half2(bf16_bits_to_float(vw[e] & 0xffff), bf16_bits_to_float(vw[e] >> 16));
                }
                kh = make_uint4(ko[0], ko[1], ko[2], ko[3]); vh = make_uint4(vo[0], vo[1], vo[2], vo[3]);
            }
            *reinterpret_cast<uint4*>(sK + (r >> 3) * 2048 + piece * 128 + (r & 7) * 16) = kh;
            *reinterpret_cast<uint4*>(sV + piece * 1024 + (r >> 3) * 128 + (r & 7) * 16) = vh;
            if (piece == 0) {
                meta[r] = META_PLAIN;
                kpos[r] = idx < n_old_fp ? (idx < a_hi ? idx : c_lo + (idx - a_hi)) : -1;
            }
        }
        if (base + TN > n_old_fp) consume(std::false_type{}, std::true_type{}, false, -1); else consume(std::false_type{}, std::false_type{}, false, -1);
    }

    // ---- (2) quantized positions below the chunk: one packed page per tile, staged as integer codes
    if (q_hi > q_lo) {
        constexpr int REC = record_bytes(BITS);
        const int page_first = q_lo / PAGE_TOKENS, page_last = (q_hi - 1) / PAGE_TOKENS;
        for (int pg = page_first; pg <= page_last && !failed; ++pg) {
            int page = -1;
            if (pg < c.max_pages) page = __ldg(c.page_table + static_cast<long long>(sl) * c.max_pages + pg);
            const bool page_ok = page >= 0 && page < c.n_pages;
            if (!page_ok && tid == 0) atomicOr(c.dev_status, pg < c.max_pages ? WUSHKV_DEV_BAD_PAGE_ID : WUSHKV_DEV_PAGE_TABLE_FULL);
            if (!drain_pv()) { failed = true; break; }          // the record is staged in the value buffer of the previous tile
            unsigned char* sV = sVb + vb * TC_K_BYTES;
            unsigned char* raw = sVb + (vb ^ 1) * TC_K_BYTES;
            if (page_ok) {
                const uint4* src = reinterpret_cast<const uint4*>(c.pages + (static_cast<long long>(page) * c.n_kv + h) * REC);
                for (int k = tid; k < REC / 16; k += TM) reinterpret_cast<uint4*>(raw)[k] = __ldg(src + k);
            }
            __syncthreads();
            {   // thread -> token r = tid & 63, channels (tid >> 6) * 64 .. + 63, eight at a time
                const int r = tid & 63, ch0 = (tid >> 6) * 64;
                const int pos = pg * PAGE_TOKENS + r;
                const bool live = page_ok && pos >= q_lo && pos < q_hi;
                const uint4 zero4 = make_uint4(0, 0, 0, 0);
                for (int kc = ch0 / 8; kc < ch0 / 8 + 8; ++kc) {
                    uint4 kq = zero4, vq = zero4;
                    if (live) unpack_chunk8<BITS>(raw, r, kc, kq, vq);
                    *reinterpret_cast<uint4*>(sK + (r >> 3) * 2048 + kc * 128 + (r & 7) * 16) = kq;
                    *reinterpret_cast<uint4*>(sV + kc * 1024 + (r >> 3) * 128 + (r & 7) * 16) = vq;
                }
                if (ch0 == 0) {
                    meta[r] = live ? *reinterpret_cast<const uint2*>(raw + meta_location(BITS, r)) : make_uint2(0u, 0u);
                    kpos[r] = live ? pos : -1;
                }
            }
            consume(std::true_type{}, std::true_type{}, false, -1);
        }
    }

    // ---- (3) the chunk itself, causal: key tiles up to the tile's last position
    const int last_row = min(qt * R + R, n_new) - 1;
    for (int kt = 0; kt * TN <= last_row && !failed; ++kt) {
        unsigned char* sV = sVb + vb * TC_K_BYTES;
        if (P.use_tma) {
            // four bulk tensor copies (keys / values x channel halves) of 64 rows x 128 bytes each; rows past the end of
            // the chunk read zeros, rows of the next sequence are masked below.  Only the first tile is fetched here: every
            // later one was requested while its predecessor's softmax ran (see consume).
            if (kt == 0 && tid == 0) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tbar), "r"(2u * TC_K_BYTES) : "memory");
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (!(P.drop == 2 && hf == 0))
                        tma_load_3d(smem_addr(sK) + hf * 8192, &map_k, 64 * hf, h, first, tbar);
                    tma_load_3d(smem_addr(sV) + hf * 8192, &map_v, 64 * hf, h, first, tbar);
                }
            }
            if (tid < TN) {
                const int row = kt * TN + tid;
                meta[tid] = META_PLAIN;
                kpos[tid] = row < n_new ? S0 + row : -1;
            }
        } else {
            for (int item = tid; item < TN * 16; item += TM) {
                const int r = item >> 4, piece = item & 15, row = kt * TN + r;
                const bool in = row < n_new;
                const long long off = (static_cast<long long>(first + (in ? row : 0)) * c.n_kv + h) * D + 8 * piece;
                cp16(smem_addr(sK + (r >> 3) * 2048 + piece * 128 + (r & 7) * 16), P.KP + off, in ? 16u : 0u);
                cp16(smem_addr(sV + piece * 1024 + (r >> 3) * 128 + (r & 7) * 16), P.VP + off, in ? 16u : 0u);
                if (piece == 0) {
                    meta[r] = META_PLAIN;
                    kpos[r] = in ? S0 + row : -1;
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        const int next_row = (P.use_tma && (kt + 1) * TN <= last_row) ? first + (kt + 1) * TN : -1;
        // no mask needed when every key of the tile exists and lies at or below every row's own position
        if (kt * TN + TN <= n_new && S0 + kt * TN + TN - 1 <= tile_pos_lo) consume(std::false_type{}, std::false_type{}, P.use_tma != 0, next_row);
        else consume(std::false_type{}, std::true_type{}, P.use_tma != 0, next_row);
    }

    // ---- output: o = (O + z) / l for the rows that carry a query
    if (!failed && !drain_pv()) failed = true;
    if (!failed && have_o) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        float* dst = P.O + (static_cast<long long>(my_tok) * c.n_q + my_jq) * D;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            float o[32];
            tc_ld32(tmem_row + 32 * q4, o);
            if (tid < n_rows) {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    *reinterpret_cast<float4*>(dst + 32 * q4 + i) = make_float4((o[i] + z) * inv, (o[i + 1] + z) * inv, (o[i + 2] + z) * inv, (o[i + 3] + z) * inv);
            }
        }
    }
    if (failed) {
        // commit whatever was issued once more and give it a bounded time, so that no MMA is still writing tensor
        // memory when it is released below
        if (tid == 0) {
            atomicOr(c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(mbar)) : "memory");
        }
        for (int it = 0; it < 512; ++it) {
            unsigned ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(smem_addr(mbar)), "r"(phase), "r"(2000u) : "memory");
            if (ok) break;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
}

// ------------------------------------------------------------------------------------------------
// 2c. attention on tcgen05, warp-specialised (the default path)
// ------------------------------------------------------------------------------------------------
// One CTA of 512 threads per (sequence, KV head, PAIR of consecutive 128-row query tiles), one CTA per SM.  The
// roles run on their own and meet only at mbarriers, so that the tensor pipe computes the scores of later key tiles
// while the softmax warps work on the current one:
//   warps 0-3 / 4-7   softmax of query tile 0 / 1: thread r owns row r.  Per key tile: wait for S, read the row with
//                     tcgen05.ld, scale / mask, raise the lazy reference (rescaling the accumulator rows in tensor memory
//                     only then), write (p Delta_v) as fp16 pairs over the first 32 columns of the score buffer just read,
//                     arrive on the tile's "probabilities ready" barrier.
//   warps 8 / 11      issue the tcgen05.mma of query tile 0 / 1 (one lane each): per key tile g, once the probabilities
//                     are ready, O_t += P_t(g) V(g) and then S_t(g+2) = Q'_t K(g+2)^T (into the score buffer P_t(g) sat in);
//                     commits release the key / value stages (two arrivals each) and signal the softmax warps.
//   warps 9 / 10      one lane each requests the chunk's own key / value tiles (and warp 9 the query tiles) as bulk tensor
//                     copies into rings of two / three stages.
//   warps 12-15       write the other key / value tiles into the same rings: bf16 window rows, and packed pages (the raw
//                     record arrives by a bulk copy one tile ahead and is unpacked into fp16 codes).
// Registers are moved from warps 8-15 to the softmax warps (setmaxnreg, per group of four warps).
// When the tile pairs of a call are too few to fill the GPU, n_split CTAs share a pair: each takes a contiguous share of the
// pair's key tiles and writes a partial row (O, reference, sum) per query row; prefill_merge_kernel combines them.
// Tensor memory (512 columns): query tile t owns columns 256 t .. 256 t + 255: O (128), two score buffers (64 each).
// Every wait is bounded; a wait that runs out raises a CTA-wide flag that ends all roles.
constexpr int WS_THREADS = 512;
constexpr int PART_W = 132;                                      // floats of a partial row: O (128), reference, sum, padding
constexpr int WS_KS = 2, WS_VS = 3;                              // ring depths of the key / value stages: a key stage is free again when
                                                                 // its scores are done, a value stage only after O += P V a softmax later
constexpr int WS_OFF_Q = 0;                                      // (tile 0 value, remainder), (tile 1 value, remainder)
constexpr int WS_OFF_K = 4 * TC_Q_BYTES;
constexpr int WS_OFF_V = WS_OFF_K + WS_KS * TC_K_BYTES;
constexpr int WS_OFF_RAW = WS_OFF_V + WS_VS * TC_K_BYTES;        // two raw records
enum { WB_KFULL = 0, WB_KEMPTY = WB_KFULL + WS_KS, WB_VFULL = WB_KEMPTY + WS_KS, WB_VEMPTY = WB_VFULL + WS_VS,
       WB_S = WB_VEMPTY + WS_VS, WB_PV = WB_S + 4, WB_PREADY = WB_PV + 4, WB_RAW = WB_PREADY + 4, WB_Q = WB_RAW + 2,
       WB_STAGED, WB_DRAIN, WB_RAWFREE, WB_COUNT = WB_RAWFREE + 2 };
// The rest of the layout depends on the record size.  Per-key factors of a packed tile, per value stage: (step, offset) of
// the key side for the 64 keys as fp32 pairs (the softmax threads load them ready to use, two keys per 16-byte load).
__host__ __device__ constexpr int ws_meta_stage(int) { return TN * 8; }
__host__ __device__ constexpr int ws_off_meta(int bits) { return WS_OFF_RAW + 2 * record_bytes(bits); }
__host__ __device__ constexpr int ws_off_live(int bits) { return ws_off_meta(bits) + WS_VS * ws_meta_stage(bits); }      // uint2[WS_VS]: which keys of a packed tile exist
__host__ __device__ constexpr int ws_off_bar(int bits) { return ws_off_live(bits) + WS_VS * 8; }
__host__ __device__ constexpr int ws_off_misc(int bits) { return ws_off_bar(bits) + WB_COUNT * 8; }                       // [0] tensor-memory slot, [4] abort flag
__host__ __device__ constexpr int ws_smem(int bits) { return ws_off_misc(bits) + 16; }
static_assert(ws_smem(2) <= 232448 && ws_smem(3) <= 232448 && ws_smem(4) <= 232448, "the dynamic shared memory of one CTA");
static_assert(WS_OFF_K % 1024 == 0 && WS_OFF_V % 1024 == 0 && WS_OFF_RAW % 16 == 0, "alignment of the stages");
static_assert(record_bytes(2) % 16 == 0 && record_bytes(3) % 16 == 0 && record_bytes(4) % 16 == 0, "raw records are copied in 16-byte units");

// Bounded wait for a phase of an mbarrier; gives up early when another role has raised the abort flag and raises it
// itself when the limit runs out.
__device__ __forceinline__ bool ws_wait(unsigned bar, unsigned parity, int limit, volatile int* abort_flag) {
    {   // the common case: the phase is complete already (a test is cheaper than a wait that may suspend the thread)
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
    }
    for (int it = 0; it < limit; ++it) {
        unsigned ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity), "r"(64u) : "memory");
        if (ok) return true;
        if ((it & 7) == 7 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void ws_arrive(unsigned bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ void ws_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void ws_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ws_bulk_g2s(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// AND of a predicate over the 128 staging threads (named barrier 1): keeps their give-up decision uniform
__device__ __forceinline__ bool ws_stagers_and(bool pred) {
    unsigned r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "r"(pred ? 1u : 0u) : "memory");
    return r != 0;
}

#ifndef WUSHKV_WS_TIMING
#define WUSHKV_WS_TIMING 0      // timing experiments only: per-role cycle counters of CTA (0, 0)
#endif
#if WUSHKV_WS_TIMING
__device__ unsigned long long g_ws_t[32];
#define WST_DECL long long wst_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long wst_last = clock64()
#define WST(slot) do { const long long now = clock64(); wst_acc[slot] += now - wst_last; wst_last = now; } while (0)
#define WST_FLUSH do { if (blockIdx.x == 0 && blockIdx.y == 0 && lane == 0 && (warp == 0 || warp == 8 || warp == 9 || warp == 12)) \
    for (int i = 0; i < 8; ++i) g_ws_t[(warp == 8 ? 16 : warp == 9 ? 24 : warp == 12 ? 8 : 0) + i] += wst_acc[i]; } while (0)
#else
#define WST_DECL
#define WST(slot) do { } while (0)
#define WST_FLUSH do { } while (0)
#endif

template <int BITS>
__global__ void __launch_bounds__(WS_THREADS, 1) prefill_attn_ws_kernel(PrefillParams P, const __grid_constant__ CUtensorMap map_k,
                                                                        const __grid_constant__ CUtensorMap map_v,
                                                                        const __grid_constant__ CUtensorMap map_q0,
                                                                        const __grid_constant__ CUtensorMap map_q1) {
    extern __shared__ __align__(1024) unsigned char sm_ws[];
    constexpr int REC = record_bytes(BITS);
    constexpr int META_STAGE = ws_meta_stage(BITS);
    const CacheView& c = P.c;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = c.G, R = TM / G;                              // chunk positions per query tile
    // n_split CTAs share a tile pair: each takes a contiguous share of the pair's key tiles and leaves a partial result
    // (short chunks over long caches would otherwise occupy a few SMs only)
    const int n_split = P.n_split, sp = static_cast<int>(blockIdx.x % n_split), bx = static_cast<int>(blockIdx.x / n_split);
    const int pairs = (P.tiles_per_seq + 1) >> 1;
    const int pr = pairs - 1 - bx % pairs;                      // long pairs first
    const int b = bx / pairs, h = blockIdx.y;
    const int first = __ldg(P.cu_new + b), n_new = __ldg(P.cu_new + b + 1) - first;
    if (2 * pr * R >= n_new) return;
    const int S = __ldg(P.seq_len + b), sl = __ldg(P.slot + b);
    if (sl < 0 || sl >= c.n_slots || S < n_new) {
        if (tid == 0) atomicOr(c.dev_status, WUSHKV_DEV_BAD_SLOT);
        return;
    }
    const unsigned bar0 = smem_addr(sm_ws + ws_off_bar(BITS));
    auto bar = [&](int i) -> unsigned { return bar0 + 8u * static_cast<unsigned>(i); };
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(sm_ws + ws_off_misc(BITS));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm_ws + ws_off_misc(BITS) + 4);
    unsigned char* meta_all = sm_ws + ws_off_meta(BITS);         // [stage][key side, value side][key]: (step, offset)
    uint2* live_all = reinterpret_cast<uint2*>(sm_ws + ws_off_live(BITS));

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < WB_COUNT; ++i) {
            // probabilities: the 128 softmax threads of a tile; stage releases: the two issuing warps; queries: one announcement
            // of bulk tensor copies, or warps 0-8 with their 16-byte copies
            const unsigned count = (i >= WB_PREADY && i < WB_PREADY + 4) ? 128u : i == WB_Q ? (P.use_tma ? 1u : 256u)
                                 : (i >= WB_KEMPTY && i < WB_KEMPTY + WS_KS) || (i >= WB_VEMPTY && i < WB_VEMPTY + WS_VS) ? 2u : 1u;
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(i)), "r"(count) : "memory");
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // ---- geometry of the key side (as in the one-tile kernel) and of the two query tiles
    const int S0 = S - n_new;
    const int nq = n_quantized(S - c.lag, c.s_sink, c.s_keep, c.s_flush);
    const int q_lo = c.s_sink, q_hi = min(c.s_sink + nq, S0);
    const int a_hi = min(c.s_sink, S0);
    const int c_lo = max(q_hi, a_hi);
    const int n_old_fp = a_hi + max(S0 - c_lo, 0);
    const float k2 = c.sm_scale * LOG2E_F;
    const int nA_all = (n_old_fp + TN - 1) / TN;                // tiles of full-precision old positions
    const int page_first = q_lo / PAGE_TOKENS;
    const int nB_all = q_hi > q_lo ? (q_hi - 1) / PAGE_TOKENS - page_first + 1 : 0;      // packed pages
    const int gC_all = nA_all + nB_all;                         // first tile of the chunk itself
    int n_rows[2], n_tiles[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qt = 2 * pr + t, np = min(R, n_new - qt * R);
        n_rows[t] = max(np, 0) * G;
        n_tiles[t] = np > 0 ? gC_all + (min(qt * R + R, n_new) - 1) / TN + 1 : 0;
    }
    // This CTA's share [g0, g0 + NT) of the pair's key tiles.  From here on tiles are counted from g0: nA and gC are the
    // (possibly negative, possibly beyond NT) local indices where the packed pages and the chunk's own tiles begin.
    const int NT_all = max(n_tiles[0], n_tiles[1]);
    const int g0 = static_cast<int>(static_cast<long long>(NT_all) * sp / n_split);
    const int NT = static_cast<int>(static_cast<long long>(NT_all) * (sp + 1) / n_split) - g0;
    const int nA = nA_all - g0, gC = gC_all - g0;
#pragma unroll
    for (int t = 0; t < 2; ++t) n_tiles[t] = min(max(n_tiles[t] - g0, 0), NT);
    const int n_staged = P.use_tma ? min(max(gC, 0), NT) : NT;                // tiles written by the staging threads
    const int gb_first = max(-nA, 0), gb_end = max(min(gC, NT) - nA, gb_first);      // this CTA's packed pages [gb_first, gb_end)
    const int wait_limit = P.wait_limit > 0 ? P.wait_limit : (1 << 24);      // polls of at least ~60 ns each: a second or more

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;
    // Registers move from the issuing / copying / staging warps to the softmax warps (per group of four warps; each group
    // executes its own instruction at the head of its branch, so that the code below it is compiled for the new count).
    // ---- the packed query tiles: row r of tile t = chunk position (2 pr + t) R + r / G, head h G + r % G.  With bulk tensor
    // copies a box of (64 channels, G heads, R positions) lands as R G rows of 128 bytes in exactly that order (128-byte
    // swizzle; rows past the chunk hold zeros or the next sequence's queries and are never stored); otherwise the softmax
    // and MMA warps place 16-byte pieces (rows clamped to the chunk) while the staging warps start on the key side at once.
    if (warp < 8) {
        // =============================== softmax of query tile t ==========================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 176;" ::: "memory");
        if (!P.use_tma) {
            for (int item = tid; item < 4 * TM * 16; item += 256) {
                const int q = item >> 11, part = q & 1, r = (item >> 4) & (TM - 1), piece = item & 15;
                const int tq = n_rows[q >> 1] > 0 ? (q >> 1) : 0;       // a tile without rows aliases tile 0's (never used)
                const int rr = min(r, n_rows[tq] - 1);
                const int tok = first + (2 * pr + tq) * R + rr / G, jq = h * G + rr % G;
                const __half* src = P.QP + static_cast<long long>(part) * P.total_new * c.n_q * D + (static_cast<long long>(tok) * c.n_q + jq) * D + 8 * piece;
                cp16(smem_addr(sm_ws + WS_OFF_Q + q * TC_Q_BYTES + (r >> 3) * 2048 + piece * 128 + (r & 7) * 16), src, 16u);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ws_arrive(bar(WB_Q));
        }
        const int t = warp >> 2, wt = tid & 127;
        if (n_tiles[t] > 0) {
            const int qt = 2 * pr + t;
            const int my_r = min(wt, n_rows[t] - 1);
            const int my_tok = first + qt * R + my_r / G, my_jq = h * G + my_r % G;
            const float my_qsum = __ldcg(P.qsum + static_cast<long long>(my_tok) * c.n_q + my_jq);
            const int my_row = qt * R + my_r / G;               // this row sees the chunk's rows 0 .. my_row
            const int tile_row_lo = qt * R;                     // smallest such limit of the tile
            const unsigned tmem_row = tmem_base + (static_cast<unsigned>((warp & 3) * 32) << 16) + 256u * t;
            float m_ref = -INFINITY, l = 0.f;
            bool ok = true;
            WST_DECL;

            // One key tile.  PACKED: the keys are integer codes that carry affine factors (a packed page; the factors and the
            // set of existing keys come with the value stage; the values of a packed page are staged dequantized).  MASKED: key j exists if bit j of (live_lo, live_hi) is set and is visible to
            // this row if crow0 + j <= my_row (crow0: chunk row of the tile's first key, very negative for old positions).
            auto soft = [&](auto packed_tag, auto masked_tag, const int g, unsigned live_lo, unsigned live_hi, const int crow0) {
                constexpr bool PACKED = decltype(packed_tag)::value, MASKED = decltype(masked_tag)::value;
                const unsigned sbuf = tmem_row + 128u + 64u * (g & 1);
                WST(0);
                // one barrier per score buffer: its next phase (tile g + 2) cannot complete before this tile's probabilities are ready
                if (!__all_sync(FULLM, ws_wait(bar(WB_S + 2 * t + (g & 1)), (g >> 1) & 1, wait_limit, abort_flag))) { ok = false; return; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned char* kmeta = meta_all + (g % WS_VS) * META_STAGE;
                auto factors4 = [&](const unsigned char* side, const int j4, float2 (&f)[4]) {      // (step, offset) of keys 4 j4 .. 4 j4 + 3
                    const float4 a = reinterpret_cast<const float4*>(side)[2 * j4], b2 = reinterpret_cast<const float4*>(side)[2 * j4 + 1];
                    f[0] = make_float2(a.x, a.y); f[1] = make_float2(a.z, a.w); f[2] = make_float2(b2.x, b2.y); f[3] = make_float2(b2.z, b2.w);
                };
                if (PACKED) {
                    if (!__all_sync(FULLM, ws_wait(bar(WB_VFULL + g % WS_VS), (g / WS_VS) & 1, wait_limit, abort_flag))) { ok = false; return; }
                    const uint2 lv = live_all[g % WS_VS];
                    live_lo = lv.x; live_hi = lv.y;
                }
                WST(1);
                float s[TN];
                tc_ld64(sbuf, s);
                WST(2);
                // scores before the common factor k2 = scale * log2(e) > 0, which is folded into the exponent's multiply-add
                // below: the maximum is taken of these (three-input max), then scaled once
                // (a packed page inside the quantized range has all its keys, and all of them lie below the chunk: no mask)
                if (PACKED && (live_lo & live_hi) == 0xffffffffu) {
#pragma unroll
                    for (int j4 = 0; j4 < TN / 4; ++j4) {
                        float2 mk[4];
                        factors4(kmeta, j4, mk);
#pragma unroll
                        for (int q = 0; q < 4; ++q) s[4 * j4 + q] = fmaf(mk[q].y, my_qsum, mk[q].x * s[4 * j4 + q]);
                    }
                } else if (PACKED || MASKED) {
#pragma unroll
                    for (int j4 = 0; j4 < TN / 4; ++j4) {
                        float2 mk[4];
                        if (PACKED) factors4(kmeta, j4, mk);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int j = 4 * j4 + q;
                            float v = s[j];
                            if (PACKED) v = fmaf(mk[q].y, my_qsum, mk[q].x * v);
                            if (MASKED) {
                                const bool live = ((j < 32 ? live_lo >> j : live_hi >> (j - 32)) & 1u) != 0u;
                                if (!live || crow0 + j > my_row) v = -INFINITY;
                            }
                            s[j] = v;
                        }
                    }
                }
                float mx_raw = fmaxf(s[0], s[1]);
#pragma unroll
                for (int j = 2; j < TN; j += 2) mx_raw = max3f(mx_raw, s[j], s[j + 1]);
                const float mx = k2 * mx_raw;
                const bool raise = mx > m_ref + REF_SLACK;                 // also the first finite maximum (m_ref = -inf)
                const float new_ref = raise ? mx : m_ref;
                const float factor = raise ? fast_ex2(m_ref - new_ref) : 1.f;      // old reference -inf: factor 0, state is zero anyway
                WST(3);
                // The accumulator rows in tensor memory are touched only when the reference grew: only then is O += P V of
                // the previous tile awaited (one barrier per tile parity, so that a warp may skip any number of them).
                if (g > 0 && __any_sync(FULLM, raise)) {
                    if (!__all_sync(FULLM, ws_wait(bar(WB_PV + 2 * t + ((g - 1) & 1)), ((g - 1) >> 1) & 1, wait_limit, abort_flag))) { ok = false; return; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        float o[32];
                        tc_ld32(tmem_row + 32 * q4, o);
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] *= factor;
                        tc_st32(tmem_row + 32 * q4, o);
                    }
                }
                WST(4);
                l *= factor;
                m_ref = new_ref;
                const float ref = m_ref == -INFINITY ? 0.f : m_ref;
                // ---- probabilities as fp16 pairs over the first 32 columns of the score buffer just read
                float2 lsum = make_float2(0.f, 0.f);                       // two partial sums
#pragma unroll
                for (int half = 0; half < 2; ++half) {                     // 32 keys = 16 columns of fp16 pairs at a time
                    unsigned pk[16];
#pragma unroll
                    for (int e4 = 0; e4 < 8; ++e4) {                       // four keys = two fp16 pairs at a time
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int e = 16 * half + 2 * e4 + q;
                            // k2 s - ref in one rounding, two lanes per instruction
                            float2 pr;
                            asm("{\n\t.reg .b64 va, vm, vc, vd;\n\tmov.b64 va, {%2, %3};\n\tmov.b64 vm, {%4, %4};\n\tmov.b64 vc, {%5, %5};\n\t"
                                "fma.rn.f32x2 vd, va, vm, vc;\n\tmov.b64 {%0, %1}, vd;\n\t}"
                                : "=f"(pr.x), "=f"(pr.y) : "f"(s[2 * e]), "f"(s[2 * e + 1]), "f"(k2), "f"(-ref));
                            pr.x = fast_ex2(pr.x); pr.y = fast_ex2(pr.y);
                            // so the running sums
                            asm("{\n\t.reg .b64 va, vb, vd;\n\tmov.b64 va, {%2, %3};\n\tmov.b64 vb, {%4, %5};\n\tadd.rn.f32x2 vd, va, vb;\n\tmov.b64 {%0, %1}, vd;\n\t}"
                                : "=f"(lsum.x), "=f"(lsum.y) : "f"(lsum.x), "f"(lsum.y), "f"(pr.x), "f"(pr.y));
                            pk[2 * e4 + q] = pack_half2(pr.x, pr.y);
                        }
                    }
                    tc_st16u(sbuf + 16 * half, pk);
                }
                l += lsum.x + lsum.y;
                WST(5);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                // one barrier per tile parity: the softmax of tile g + 1 does not wait for the issuing warp, that of tile g + 2 does
                ws_arrive(bar(WB_PREADY + 2 * t + (g & 1)));
                WST(6);
            };

            constexpr int FAR_BELOW = -(1 << 30);
            for (int g = 0; g < n_tiles[t] && ok; ++g) {
                // valid keys of the tile and the chunk row of its first key (old positions: visible to every row)
                int nv = TN, crow0 = FAR_BELOW;
                bool masked = false;
                if (g < nA) { nv = min(TN, n_old_fp - (g + g0) * TN); masked = nv < TN; }
                else if (g >= gC) {
                    const int kt = g - gC;
                    nv = min(TN, n_new - kt * TN); crow0 = kt * TN;
                    // no mask needed when every key of the tile exists and lies at or below every row's own position
                    masked = nv < TN || kt * TN + TN - 1 > tile_row_lo;
                }
                const unsigned live_lo = nv >= 32 ? 0xffffffffu : (1u << nv) - 1u;
                const unsigned live_hi = nv >= TN ? 0xffffffffu : nv > 32 ? (1u << (nv - 32)) - 1u : 0u;
                // (one call per variant, so that each is expanded in place)
                if (g >= nA && g < gC) soft(std::true_type{}, std::true_type{}, g, 0u, 0u, FAR_BELOW);
                else if (masked) soft(std::false_type{}, std::true_type{}, g, live_lo, live_hi, crow0);
                else soft(std::false_type{}, std::false_type{}, g, 0u, 0u, 0);
            }
            WST_FLUSH;
            // ---- output: o = O / l for the rows that carry a query
            if (ok && !__all_sync(FULLM, ws_wait(bar(WB_PV + 2 * t + ((n_tiles[t] - 1) & 1)), ((n_tiles[t] - 1) >> 1) & 1, wait_limit, abort_flag))) ok = false;
            if (ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // alone: o = O / l; one of several CTAs of the pair: the partial (O, reference, l) for the merge
                const float inv = n_split > 1 ? 1.f : (l > 0.f ? 1.f / l : 0.f);
                float* dst = n_split > 1 ? P.part + ((static_cast<long long>(sp) * P.total_new + my_tok) * c.n_q + my_jq) * PART_W
                                         : P.O + (static_cast<long long>(my_tok) * c.n_q + my_jq) * D;
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    float o[32];
                    tc_ld32(tmem_row + 32 * q4, o);
                    if (wt < n_rows[t]) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *reinterpret_cast<float4*>(dst + 32 * q4 + i) = make_float4(o[i] * inv, o[i + 1] * inv, o[i + 2] * inv, o[i + 3] * inv);
                    }
                }
                if (n_split > 1 && wt < n_rows[t]) *reinterpret_cast<float2*>(dst + D) = make_float2(m_ref, l);
            }
        } else if (n_split > 1 && wt < n_rows[t]) {
            // none of this CTA's key tiles is the tile's: an empty partial (reference -inf, sum 0)
            const int qt = 2 * pr + t;
            const int my_tok = first + qt * R + wt / G, my_jq = h * G + wt % G;
            float* dst = P.part + ((static_cast<long long>(sp) * P.total_new + my_tok) * c.n_q + my_jq) * PART_W;
#pragma unroll
            for (int i = 0; i < D; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(0.f, 0.f, 0.f, 0.f);
            *reinterpret_cast<float2*>(dst + D) = make_float2(-INFINITY, 0.f);
        }
    }
    else if (warp < 12) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 64;" ::: "memory");
      if (P.use_tma && tid == 288) {
            const unsigned box_bytes = 128u * static_cast<unsigned>(G * R);
            ws_expect_tx(bar(WB_Q), 4u * box_bytes * ((n_tiles[0] > 0 ? 1u : 0u) + (n_tiles[1] > 0 ? 1u : 0u)));
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (n_tiles[q >> 1] == 0) continue;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
                    tma_load_3d(smem_addr(sm_ws + WS_OFF_Q + q * TC_Q_BYTES + hf * 16384), (q & 1) ? &map_q1 : &map_q0, 64 * hf, h * G,
                                first + (2 * pr + (q >> 1)) * R, bar(WB_Q));
            }
      }
      if (warp == 8 || warp == 11) {
        // =============================== MMA issue for query tile t ========================================
        // One issuing warp per query tile: with the 64-key tiles an MMA takes the pipe 48-64 cycles, about what one thread
        // needs to issue it, so a single thread for both tiles left the pipe half idle.
        const int t = warp == 8 ? 0 : 1;
        const int mine = n_tiles[t];                            // tiles of this query tile; the other one may have more
        WST_DECL;
        bool ok = __all_sync(FULLM, ws_wait(bar(WB_Q), 0u, wait_limit, abort_flag));
        WST(0);
        // Descriptors are built once; their low bits hold the start address / 16, so a byte offset is added as offset / 16.
        const bool q_swz = P.use_tma != 0;                      // query tiles written by bulk tensor copies: 128-byte-swizzled rows, two 16 KB boxes
        const unsigned long long q_desc = q_swz ? tc_desc_sw128(smem_addr(sm_ws + WS_OFF_Q + 2 * t * TC_Q_BYTES), 16, 1024)
                                                : tc_desc(smem_addr(sm_ws + WS_OFF_Q + 2 * t * TC_Q_BYTES), 128, 2048);
        const unsigned long long k_plain0 = tc_desc(smem_addr(sm_ws + WS_OFF_K), 128, 2048), k_swz0 = tc_desc_sw128(smem_addr(sm_ws + WS_OFF_K), 16, 1024);
        const unsigned long long v_plain0 = tc_desc(smem_addr(sm_ws + WS_OFF_V), 128, 1024), v_swz0 = tc_desc_sw128(smem_addr(sm_ws + WS_OFF_V), 8192, 1024);
        const unsigned acc_o = tmem_base + 256u * t;
        auto scores_of = [&](auto swz_tag, const int g, const int st) {      // lane 0: the MMAs of S_t(g)
            constexpr bool SWZ = decltype(swz_tag)::value;
            const unsigned long long kb = (SWZ ? k_swz0 : k_plain0) + static_cast<unsigned>(st * (TC_K_BYTES >> 4));
            const unsigned acc = acc_o + 128u + 64u * (g & 1);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                // swizzled: channels 0-63 and 64-127 are two boxes of 8 KB; a k-step of 16 channels is 32 bytes inside the 128-byte row
                const unsigned long long bdesc = kb + static_cast<unsigned>((SWZ ? (ks >> 2) * 8192 + (ks & 3) * 32 : ks * 256) >> 4);
                const unsigned long long adesc = q_desc + static_cast<unsigned>((q_swz ? (ks >> 2) * 16384 + (ks & 3) * 32 : ks * 256) >> 4);
                tc_mma(acc, adesc, bdesc, TC_IDESC_S, ks > 0 ? 1u : 0u);
                tc_mma(acc, adesc + static_cast<unsigned>(TC_Q_BYTES >> 4), bdesc, TC_IDESC_S, 1u);
            }
            if (!(P.drop == 1 && g == 0)) ws_commit(bar(WB_S + 2 * t + (g & 1)));
            ws_commit(bar(WB_KEMPTY + st));
        };
        // Only lane 0 runs the loop.  Order per tile g: wait for the probabilities, O_t += P_t(g) V(g), S_t(g+2) (its score
        // buffer is the one P_t(g) sits in, so it must follow that product in the pipe), then, off the critical path, the
        // wait for the value stage the next round needs.
        auto scores = [&](const int g) -> bool {                // key stage of tile g has landed (awaited by the caller)
            const int st = g % WS_KS;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (g >= mine) ws_arrive(bar(WB_KEMPTY + st));      // a tile only the other query tile reads: just release the stage
            else if (g >= gC && P.use_tma) scores_of(std::true_type{}, g, st);
            else scores_of(std::false_type{}, g, st);
            return true;
        };
        // Two streams of work, each in tile order: the scores S_t(sc) (once the key tile has landed and O += P V of tile
        // sc - 2, which reads the probabilities out of the same score buffer, has been issued) and the products O_t += P_t(pv)
        // V(pv) (once the value tile has landed and the probabilities are ready).  Neither may wait for the other: a key tile
        // written by the staging threads arrives together with its value tile, whose stage only the product of two tiles
        // before releases.  So the thread tests the barriers and issues whatever is ready.
        auto landed = [&](const int full0, const int depth, const int g) -> bool {
            unsigned ready;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ready) : "r"(bar(full0 + g % depth)), "r"(static_cast<unsigned>((g / depth) & 1)) : "memory");
            return ready != 0;
        };
        if (lane == 0 && ok) {
            int sc = 0, pv = 0, idle = 0;
            while (pv < NT) {
                bool progressed = false;
                if (pv < sc && landed(WB_VFULL, WS_VS, pv)) {
                    const int st = pv % WS_VS;
                    if (pv >= mine) {                           // a tile only the other query tile reads: just release the stage
                        ws_arrive(bar(WB_VEMPTY + st));
                        ++pv; progressed = true;
                    } else {
                        unsigned ready;
                        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                                     : "=r"(ready) : "r"(bar(WB_PREADY + 2 * t + (pv & 1))), "r"(static_cast<unsigned>((pv >> 1) & 1)) : "memory");
                        if (ready) {
                            WST(2);
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                            const bool swz = pv >= gC && P.use_tma;
                            // swizzled values: rows (keys) of 128 bytes, 8-key groups 1024 bytes apart, channel halves 8192 bytes apart: 16 keys = 2048 bytes
                            const unsigned long long vb = (swz ? v_swz0 : v_plain0) + static_cast<unsigned>(st * (TC_K_BYTES >> 4));
                            const unsigned vstep = swz ? (2048u >> 4) : (256u >> 4);
                            const unsigned prob = acc_o + 128u + 64u * (pv & 1);
#pragma unroll
                            for (int ks = 0; ks < TN / 16; ++ks)
                                tc_mma_ts(acc_o, prob + 8 * ks, vb + ks * vstep, TC_IDESC_O, (pv > 0 || ks > 0) ? 1u : 0u);
                            ws_commit(bar(WB_PV + 2 * t + (pv & 1)));
                            ws_commit(bar(WB_VEMPTY + st));
                            ++pv; progressed = true;
                            WST(3);
                        }
                    }
                }
                if (sc < NT && sc < pv + 2 && landed(WB_KFULL, WS_KS, sc)) {
                    WST(6);
                    scores(sc);
                    ++sc; progressed = true;
                    WST(4);
                }
                if (progressed) { idle = 0; continue; }
                // nothing ready: a short pause keeps the polls off the softmax warps' issue slots; bounded like every wait
                __nanosleep(40);
                if (++idle >= wait_limit) { *abort_flag = 1; ok = false; break; }
                if ((idle & 7) == 7 && *abort_flag) { ok = false; break; }
            }
        }
        __syncwarp();
        WST_FLUSH;
      } else {
        // =============================== the chunk itself: bulk tensor copies ==============================
        // Four copies per tile (keys / values x channel halves) of 64 rows x 128 bytes; rows past the end of the chunk read
        // zeros or the next sequence's rows, both masked by the softmax warps.  Warp 9 requests the key tiles, warp 10 the
        // value tiles: the two rings advance on their own (a stage is requested once its previous tile was released, which
        // for the first chunk tiles means: once the staging threads' last tiles went through).
        int armed[3] = {-1, -1, -1};                            // last tile whose copies this warp announced on each stage (<= 3 stages)
        bool ok = true;
        // Before that, warp 9 requests the records of the packed pages for the staging threads, by bulk copies into the two
        // raw buffers: record gb as soon as the staging threads have left the record two before it.  (Done here because the
        // request costs its thread several hundred cycles, which the staging threads do not have.)
        int requested[2] = {0, 0};                              // records requested so far into each raw buffer
        if (warp == 9) {
            // (the page id is read a record ahead, so that the wait for the buffer covers the load)
            auto page_id = [&](const int gb) {
                const int pg = page_first + gb;
                return (gb < gb_end && pg < c.max_pages) ? __ldg(c.page_table + static_cast<long long>(sl) * c.max_pages + pg) : -1;
            };
            int page_ahead = page_id(gb_first);
            for (int gb = gb_first; gb < gb_end && ok; ++gb) {
                const int rb = gb & 1, use = (gb - gb_first) >> 1;      // use-th record of this buffer
                const int page = page_ahead;
                page_ahead = page_id(gb + 1);
                if (use >= 1 && !__all_sync(FULLM, ws_wait(bar(WB_RAWFREE + rb), (use - 1) & 1, wait_limit, abort_flag))) { ok = false; break; }
                if (lane == 0) {
                    const int pg = page_first + gb;
                    if (page < 0 || page >= c.n_pages) {
                        atomicOr(c.dev_status, pg < c.max_pages ? WUSHKV_DEV_BAD_PAGE_ID : WUSHKV_DEV_PAGE_TABLE_FULL);
                    } else {
                        ws_expect_tx(bar(WB_RAW + rb), REC);
                        ws_bulk_g2s(smem_addr(sm_ws + WS_OFF_RAW + rb * REC), c.pages + (static_cast<long long>(page) * c.n_kv + h) * REC, REC,
                                    bar(WB_RAW + rb));
                        ++requested[rb];
                    }
                }
            }
        }
        if (ok && P.use_tma && n_staged > 0) ok = __all_sync(FULLM, ws_wait(bar(WB_STAGED), 0u, wait_limit, abort_flag));
        if (P.use_tma) {
            const bool keys = warp == 9;
            const int depth = keys ? WS_KS : WS_VS, full0 = keys ? WB_KFULL : WB_VFULL, empty0 = keys ? WB_KEMPTY : WB_VEMPTY;
            const CUtensorMap* map = keys ? &map_k : &map_v;
            unsigned char* ring = sm_ws + (keys ? WS_OFF_K : WS_OFF_V);
            WST_DECL;
            for (int g = max(gC, 0); g < NT && ok; ++g) {
                const int st = g % depth, row = first + (g - gC) * TN;
                WST(0);
                if (g >= depth && !__all_sync(FULLM, ws_wait(bar(empty0 + st), ((g / depth) - 1) & 1, wait_limit, abort_flag))) { ok = false; break; }
                WST(1);
                if (lane == 0) {
                    ws_expect_tx(bar(full0 + st), TC_K_BYTES);
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf)
                        if (!(P.drop == 2 && keys && g == gC && hf == 0))
                            tma_load_3d(smem_addr(ring + st * TC_K_BYTES) + hf * 8192, map, 64 * hf, h, row, bar(full0 + st));
                }
#pragma unroll
                for (int i = 0; i < 3; ++i) if (i == st) armed[i] = g;
#if WUSHKV_WS_TIMING
                WST(2);
                ws_wait(bar(full0 + st), (g / depth) & 1, wait_limit, abort_flag);      // measurement only: how long the copies take
                WST(3);
#endif
            }
            WST_FLUSH;
            // after a failure elsewhere: give the copies this warp announced a bounded time to land, so that none is
            // still writing shared memory when the CTA ends
            if (lane == 0 && *abort_flag) {
#pragma unroll
                for (int i = 0; i < 3; ++i)
                    if (i < depth && armed[i] >= 0)
                        for (int it = 0; it < 512 && !ws_wait(bar(full0 + i), (armed[i] / depth) & 1, 1, abort_flag); ++it) __nanosleep(2000);
            }
        }
        if (tid == 288 && *abort_flag && P.use_tma)             // the same for the query copies
            for (int it = 0; it < 512 && !ws_wait(bar(WB_Q), 0u, 1, abort_flag); ++it) __nanosleep(2000);
        if (tid == 288 && *abort_flag) {                        // and for the record copies
#pragma unroll
            for (int i = 0; i < 2; ++i)
                if (requested[i] > 0)
                    for (int it = 0; it < 64 && !ws_wait(bar(WB_RAW + i), (requested[i] - 1) & 1, 1, abort_flag); ++it) __nanosleep(2000);
        }
      }
    }
    else {
        // =============================== staging of key / value tiles by threads ===========================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 96;" ::: "memory");
        const int ptid = tid - 384;
        int raw_uses[2] = {0, 0};                               // records fetched so far into each raw buffer
        // page id of packed tile gb as the table holds it (-1 beyond the table); it is range-checked where it is used, a tile
        // later, so that nothing waits for the load
        auto page_of = [&](const int gb) -> int {
            const int pg = page_first + gb;
            return pg < c.max_pages ? __ldg(c.page_table + static_cast<long long>(sl) * c.max_pages + pg) : -1;
        };
        auto page_valid = [&](const int page) { return page >= 0 && page < c.n_pages; };
        // (the records themselves are requested by warp 9, up to two ahead; a page that cannot be read is reported there and
        // its tile is staged as absent keys here)
        int page_cur = gb_end > gb_first ? page_of(gb_first) : -1;
        bool ok = true;
        WST_DECL;
        for (int g = 0; g < n_staged && ok; ++g) {
            WST(0);
            const int ks = g % WS_KS, vs = g % WS_VS;
            unsigned char* sK = sm_ws + WS_OFF_K + ks * TC_K_BYTES;
            unsigned char* sV = sm_ws + WS_OFF_V + vs * TC_K_BYTES;
            bool mine = true;
            if (g >= WS_KS) mine = ws_wait(bar(WB_KEMPTY + ks), ((g / WS_KS) - 1) & 1, wait_limit, abort_flag);
            WST(4);
            if (mine && g >= WS_VS) mine = ws_wait(bar(WB_VEMPTY + vs), ((g / WS_VS) - 1) & 1, wait_limit, abort_flag);
            mine = __all_sync(FULLM, mine);                     // warp-uniform from here on
            WST(1);
            if (g < nA) {
                // ---- full-precision old positions: sink [0, a_hi) and recent window [c_lo, S0), bf16 rows
                for (int item = ptid; item < TN * 16 && mine; item += 128) {
                    const int r = item & (TN - 1), piece = item >> 6, idx = (g + g0) * TN + r;
                    uint4 kh = make_uint4(0, 0, 0, 0), vh = kh;
                    if (idx < n_old_fp) {
                        const long long plane = (static_cast<long long>(sl) * c.n_kv + h) * 2;
                        const unsigned short *ksrc, *vsrc;
                        if (idx < a_hi) {
                            ksrc = c.sink_kv + (plane * c.s_sink + idx) * D;
                            vsrc = c.sink_kv + ((plane + 1) * c.s_sink + idx) * D;
                        } else {
                            const int p = c_lo + (idx - a_hi);
                            ksrc = c.ring_kv + (plane * c.ring_cap + p % c.ring_cap) * D;
                            vsrc = c.ring_kv + ((plane + 1) * c.ring_cap + p % c.ring_cap) * D;
                        }
                        const uint4 kb16 = *reinterpret_cast<const uint4*>(ksrc + 8 * piece), vb16 = *reinterpret_cast<const uint4*>(vsrc + 8 * piece);
                        const unsigned kw[4] = {kb16.x, kb16.y, kb16.z, kb16.w}, vw[4] = {vb16.x, vb16.y, vb16.z, vb16.w};
                        unsigned ko[4], vo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            ko[e] = pack_half2(bf16_bits_to_float(kw[e] & 0xffff), bf16_bits_to_float(kw[e] >> 16));
                            vo[e] = pack_half2(bf16_bits_to_float(vw[e] & 0xffff), bf16_bits_to_float(vw[e] >> 16));
                        }
                        kh = make_uint4(ko[0], ko[1], ko[2], ko[3]); vh = make_uint4(vo[0], vo[1], vo[2], vo[3]);
                    }
                    *reinterpret_cast<uint4*>(sK + (r >> 3) * 2048 + piece * 128 + (r & 7) * 16) = kh;
                    *reinterpret_cast<uint4*>(sV + piece * 1024 + (r >> 3) * 128 + (r & 7) * 16) = vh;
                }
            } else if (g < gC) {
                // ---- a packed page: the record was requested one tile ahead; unpack it into integer codes (exact in fp16)
                const int gb = g - nA, rb = gb & 1;
                const bool page_ok = page_valid(page_cur);
                page_cur = gb + 1 < gb_end ? page_of(gb + 1) : -1;          // read a tile ahead: nothing waits for the page table
                if (page_ok && mine) mine = __all_sync(FULLM, ws_wait(bar(WB_RAW + rb), raw_uses[rb] & 1, wait_limit, abort_flag));
                if (page_ok) ++raw_uses[rb];
                WST(5);
                const unsigned char* raw = sm_ws + WS_OFF_RAW + rb * REC;
                const uint4 zero4 = make_uint4(0, 0, 0, 0);
                const int page_pos = (page_first + gb) * PAGE_TOKENS;
                const bool whole = page_ok && page_pos >= q_lo && page_pos + PAGE_TOKENS <= q_hi;
                if (whole && mine) unpack_page<BITS>(raw, sK, sV, ptid);
                WST(6);
#pragma unroll 4
                for (int item = ptid; item < (mine && !whole ? TN * 16 : 0); item += 128) {      // first / last page of the range
                    const int r = item & (TN - 1), kc = item >> 6;
                    const int pos = (page_first + gb) * PAGE_TOKENS + r;
                    const bool live = page_ok && pos >= q_lo && pos < q_hi;
                    uint4 kq = zero4, vq = zero4;
                    if (live) {
                        unpack_chunk8<BITS>(raw, r, kc, kq, vq);
                        // values are staged dequantized (see unpack_page)
                        const unsigned mv = *reinterpret_cast<const unsigned*>(raw + meta_location(BITS, r) + 4);
                        const unsigned step2 = __byte_perm(mv, mv, 0x1010u), offs2 = __byte_perm(mv, mv, 0x3232u);
                        unsigned* vw = reinterpret_cast<unsigned*>(&vq);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __half2 hv = __hfma2(*reinterpret_cast<const __half2*>(vw + e), *reinterpret_cast<const __half2*>(&step2),
                                                       *reinterpret_cast<const __half2*>(&offs2));
                            vw[e] = *reinterpret_cast<const unsigned*>(&hv);
                        }
                    }
                    *reinterpret_cast<uint4*>(sK + (r >> 3) * 2048 + kc * 128 + (r & 7) * 16) = kq;
                    *reinterpret_cast<uint4*>(sV + kc * 1024 + (r >> 3) * 128 + (r & 7) * 16) = vq;
                }
                if (mine && ptid < TN) {                        // warps 12 and 13: key factors and existence of key ptid
                    const int pos = (page_first + gb) * PAGE_TOKENS + ptid;
                    const bool live = page_ok && pos >= q_lo && pos < q_hi;
                    const unsigned mk = live ? *reinterpret_cast<const unsigned*>(raw + meta_location(BITS, ptid)) : 0u;
                    unsigned char* kside = meta_all + vs * META_STAGE;
                    reinterpret_cast<float2*>(kside)[ptid] = h2f2u(mk);
                    const unsigned word = __ballot_sync(FULLM, live);
                    if (lane == 0) reinterpret_cast<unsigned*>(live_all + vs)[ptid >> 5] = word;
                }
            } else {
                // ---- the chunk's own rows by 16-byte loads (testing aid; bulk tensor copies otherwise)
                const int kt = g - gC;
                for (int item = ptid; item < TN * 16 && mine; item += 128) {
                    const int r = item & (TN - 1), piece = item >> 6, row = kt * TN + r;
                    uint4 kh = make_uint4(0, 0, 0, 0), vh = kh;
                    if (row < n_new) {
                        const long long off = (static_cast<long long>(first + row) * c.n_kv + h) * D + 8 * piece;
                        kh = *reinterpret_cast<const uint4*>(P.KP + off);
                        vh = *reinterpret_cast<const uint4*>(P.VP + off);
                    }
                    *reinterpret_cast<uint4*>(sK + (r >> 3) * 2048 + piece * 128 + (r & 7) * 16) = kh;
                    *reinterpret_cast<uint4*>(sV + piece * 1024 + (r >> 3) * 128 + (r & 7) * 16) = vh;
                }
            }
            WST(2);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ok = ws_stagers_and(mine);
            WST(3);
            // (one arrival per warp: each costs its thread some tens of cycles)
            if (ok && ptid == 0) ws_arrive(bar(WB_KFULL + ks));
            if (ok && ptid == 32) ws_arrive(bar(WB_VFULL + vs));
            if (ok && ptid == 64 && g >= nA && g < gC) ws_arrive(bar(WB_RAWFREE + ((g - nA) & 1)));      // every staging thread has left the raw record
        }
        // the copy-issuing warps may start on the chunk's own tiles now: a wait for a stage's release only tells the last two
        // releases apart, so they must not look at a stage before the tiles staged here have gone through it
        WST_FLUSH;
        if (ok && ptid == 0) ws_arrive(bar(WB_STAGED));
    }

    // ---- all roles are done (or gave up)
    __syncthreads();
    if (*abort_flag) {
        // commit whatever was issued once more and give it a bounded time, so that no MMA is still writing tensor
        // memory when it is released below
        if (tid == 256) {
            atomicOr(c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
            ws_commit(bar(WB_DRAIN));
            for (int it = 0; it < 512; ++it) {
                unsigned done;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(done) : "r"(bar(WB_DRAIN)), "r"(0u), "r"(2000u) : "memory");
                if (done) break;
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// Merge of the partial results of the n_split CTAs of a tile pair: one CTA of 128 threads (one per channel) per
// (chunk token, query head).  A partial holds O relative to its own reference m (2^m was factored out of its
// probabilities) and the sum l of those probabilities; the output is sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.
__global__ void __launch_bounds__(D) prefill_merge_kernel(PrefillParams P) {
    const CacheView& c = P.c;
    const int tok = blockIdx.x, jq = blockIdx.y, ch = threadIdx.x;
    {   // a sequence the attention kernel skipped leaves no partials: its rows stay untouched here as well
        int lo = 0, hi = P.batch;
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (__ldg(P.cu_new + mid) <= tok) lo = mid; else hi = mid; }
        const int n_new = __ldg(P.cu_new + lo + 1) - __ldg(P.cu_new + lo), sl = __ldg(P.slot + lo);
        if (sl < 0 || sl >= c.n_slots || __ldg(P.seq_len + lo) < n_new) return;
    }
    const long long row = static_cast<long long>(tok) * c.n_q + jq, stride = static_cast<long long>(P.total_new) * c.n_q * PART_W;
    const float* p0 = P.part + row * PART_W;
    float M = -INFINITY;
    for (int s = 0; s < P.n_split; ++s) M = fmaxf(M, __ldcg(p0 + s * stride + D));
    float acc = 0.f, lsum = 0.f;
    for (int s = 0; s < P.n_split; ++s) {
        const float m = __ldcg(p0 + s * stride + D);
        if (m == -INFINITY) continue;
        const float w = fast_ex2(m - M);
        acc = fmaf(w, __ldcg(p0 + s * stride + ch), acc);
        lsum = fmaf(w, __ldcg(p0 + s * stride + D + 1), lsum);
    }
    P.O[row * D + ch] = lsum > 0.f ? acc / lsum : 0.f;
}

// ------------------------------------------------------------------------------------------------
// 1b. transforms of the chunk on tcgen05 (the default)
// ------------------------------------------------------------------------------------------------
// The same arithmetic as prefill_prep_kernel (bf16 x bf16 products, exact in the fp32 accumulator; T_K^{-T} as three bf16
// terms), as tcgen05.mma with the accumulator in tensor memory.  A CTA keeps its head's transform in shared memory as the
// B operand and walks over 128-token tiles:
//   warp 16  one lane requests the token tiles: two bulk tensor copies (channel halves) of 128 rows x 128 bytes into a
//            two-deep ring, the A operand as it comes;
//   warp 17  one lane issues 8 MMAs (M 128, N 128, K 16) per term into one of two 128-column accumulators;
//   warps 0-15  a thread owns 32 channels of one token of the tile (one warp alone per scheduler spends its time on
//            instruction latency): tcgen05.ld, the roundings (k' through bf16 to fp16; q' as fp16 value + fp16 remainder,
//            and their sum over the channels); the rows go through a shared-memory tile so that the stores to global memory
//            are whole 256-byte rows.
// Head slots past the query heads convert the chunk's values of one KV head to fp16 (plain loads and stores).
// Barriers come in pairs (one per ring slot), every wait is bounded.
constexpr int PT_THREADS = 576;                                  // warps 0-15 epilogue, 16 copies, 17 MMA issue
constexpr int PT_OFF_T = 0;                                      // three terms of 128 x 128 bf16, K-major core matrices
constexpr int PT_OFF_X = 3 * D * D * 2;                          // two token tiles (128-byte-swizzled rows, two 16 KB boxes each)
constexpr int PT_X_BYTES = PREP_TOK * D * 2;
enum { PB_XFULL = 0, PB_XEMPTY = 2, PB_DFULL = 4, PB_DEMPTY = 6, PB_XREADY = 8, PB_DRAIN = 10, PB_COUNT = 11 };
constexpr int PT_OUT_PITCH = D * 2 + 16;                         // bytes per staged output row (272: conflict-free 16-byte pieces)
constexpr int PT_OFF_OUT = PT_OFF_X + 2 * PT_X_BYTES;            // one fp16 output tile on its way to global memory
constexpr int PT_OFF_QS = PT_OFF_OUT + PREP_TOK * PT_OUT_PITCH;  // float[4][128]: partial sums of q' over channel quarters
constexpr int PT_MAX_SEQ = 1024;                                 // sequences whose chunk bounds are kept in shared memory (projected inputs)
constexpr int PT_OFF_SEQ = PT_OFF_QS + 4 * PREP_TOK * 4;         // int[PT_MAX_SEQ + 1] first chunk token, int[PT_MAX_SEQ] position of token 0 minus its index
constexpr int PT_OFF_BAR = PT_OFF_SEQ + (2 * PT_MAX_SEQ + 2) * 4;
constexpr int PT_OFF_MISC = PT_OFF_BAR + PB_COUNT * 8;           // [0] tensor-memory slot, [4] abort flag
constexpr int PT_SMEM = PT_OFF_MISC + 16;
constexpr unsigned PT_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((static_cast<unsigned>(D) >> 3) << 17) | ((static_cast<unsigned>(PREP_TOK) >> 4) << 24);   // fp32 <- bf16 x bf16, K-major
static_assert(PT_OFF_X % 1024 == 0, "swizzled tiles need 1024-byte alignment");

#if WUSHKV_WS_TIMING
#define PST_DECL long long pst_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long pst_last = clock64()
#define PST(slot) do { const long long now = clock64(); pst_acc[slot] += now - pst_last; pst_last = now; } while (0)
#define PST_FLUSH(base) do { if (blockIdx.x == 0 && blockIdx.y == P.c.n_kv && lane == 0) for (int i_ = 0; i_ < 8; ++i_) g_ws_t[(base) + i_] += pst_acc[i_]; } while (0)
#else
#define PST_DECL
#define PST(slot) do { } while (0)
#define PST_FLUSH(base) do { } while (0)
#endif
__global__ void __launch_bounds__(PT_THREADS, 1) prefill_prep_tc_kernel(PrefillParams P, const __grid_constant__ CUtensorMap map_k,
                                                                        const __grid_constant__ CUtensorMap map_q) {
    extern __shared__ __align__(1024) unsigned char sm_pt[];
    const int hs = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (hs >= P.c.n_kv + P.c.n_q) {
        // head slots past the query heads: the chunk's values of one KV head as fp16 (no transform), 16-byte pieces, four
        // loads in flight per thread; the CTAs of a slot take interleaved 128-token tiles like the others
        const int vh = hs - P.c.n_kv - P.c.n_q;
        for (int tok0 = static_cast<int>(blockIdx.x) * PREP_TOK; tok0 < P.total_new; tok0 += static_cast<int>(gridDim.x) * PREP_TOK) {
            uint4 v[4];
            long long off[4];
            bool in[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int item = tid + k * PT_THREADS, r = item >> 4, piece = item & 15;
                in[k] = item < PREP_TOK * 16 && tok0 + r < P.total_new;
                off[k] = (static_cast<long long>(tok0 + r) * P.c.n_kv + vh) * D + 8 * piece;
                if (in[k]) v[k] = __ldg(reinterpret_cast<const uint4*>(P.V_new + off[k]));
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (!in[k]) continue;
                const unsigned w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
                unsigned o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) o[e] = pack_half2(bf16_bits_to_float(w[e] & 0xffff), bf16_bits_to_float(w[e] >> 16));
                *reinterpret_cast<uint4*>(P.VP + off[k]) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        return;
    }
    const bool is_key = hs < P.c.n_kv;
    const int head = is_key ? hs : hs - P.c.n_kv;
    const int kvh = is_key ? head : head / P.c.G;
    const int n_terms = is_key ? 1 : 3;
    const int n_heads = is_key ? P.c.n_kv : P.c.n_q;
    const float* T = (is_key ? P.c.T_K : P.c.T_K_invT) + static_cast<long long>(kvh) * D * D;
    const unsigned bar0 = smem_addr(sm_pt + PT_OFF_BAR);
    auto bar = [&](int i) -> unsigned { return bar0 + 8u * static_cast<unsigned>(i); };
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(sm_pt + PT_OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm_pt + PT_OFF_MISC + 4);
#if WUSHKV_WS_TIMING
    const long long t_entry = clock64();
#endif
    const int n_my_tiles = (P.total_new + PREP_TOK - 1) / PREP_TOK > static_cast<int>(blockIdx.x)
                               ? ((P.total_new + PREP_TOK - 1) / PREP_TOK - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
    if (n_my_tiles == 0) return;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < PB_COUNT; ++i) {
            // accumulator released, and projected rows normalised and rotated, by the 512 epilogue threads
            const unsigned count = (i == PB_DEMPTY || i == PB_DEMPTY + 1 || i == PB_XREADY || i == PB_XREADY + 1) ? 512u : 1u;
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(i)), "r"(count) : "memory");
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // projected inputs: where every sequence's chunk starts and the position of its first token, for the row fix-up
    int* seq_first = reinterpret_cast<int*>(sm_pt + PT_OFF_SEQ);
    int* seq_base = seq_first + PT_MAX_SEQ + 1;
    const bool seq_in_smem = P.pro.rope != nullptr && P.batch <= PT_MAX_SEQ;
    if (seq_in_smem) {
        for (int bq = tid; bq <= P.batch; bq += PT_THREADS) {
            const int f0 = __ldg(P.cu_new + bq);
            seq_first[bq] = f0;
            if (bq < P.batch) seq_base[bq] = __ldg(P.seq_len + bq) - (__ldg(P.cu_new + bq + 1) - f0) - f0;
        }
    }
    // the transform as the B operand: element (i, j) of term `term` at (i / 8) * 2048 + (j / 8) * 128 + (i % 8) * 16 + (j % 8) * 2
    for (int idx = tid; idx < D * D; idx += PT_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        float x = __ldg(T + idx);
        const int off = (i >> 3) * 2048 + (j >> 3) * 128 + (i & 7) * 16 + (j & 7) * 2;
#pragma unroll
        for (int term = 0; term < 3; ++term) {
            if (term < n_terms) {
                const unsigned short hb = float_to_bf16_bits(x);
                *reinterpret_cast<unsigned short*>(sm_pt + PT_OFF_T + term * (D * D * 2) + off) = hb;
                x -= bf16_bits_to_float(hb);
            }
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;
    const int wait_limit = P.wait_limit > 0 ? P.wait_limit : (1 << 24);
    const bool fix_rows = P.pro.rope != nullptr;                // projected inputs: Algorithm 2 lines 1-2 on the staged rows
#if WUSHKV_WS_TIMING
    if (tid == 0 && blockIdx.x == 0 && blockIdx.y == gridDim.y - 1) g_ws_t[8] += clock64() - t_entry;
#endif

    if (warp == 16) {
        // ---- token tiles
        int armed[2] = {-1, -1};
        if (lane == 0) {
            const CUtensorMap* map = is_key ? &map_k : &map_q;
            for (int i = 0; i < n_my_tiles; ++i) {
                const int s = i & 1, tok0 = (static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x)) * PREP_TOK;
                if (i >= 2 && !ws_wait(bar(PB_XEMPTY + s), ((i >> 1) - 1) & 1, wait_limit, abort_flag)) break;
                ws_expect_tx(bar(PB_XFULL + s), PT_X_BYTES);
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
                    if (!(P.drop == 3 && i == 0 && hf == 0))    // testing aid: announced, never issued
                        tma_load_3d(smem_addr(sm_pt + PT_OFF_X + s * PT_X_BYTES + hf * 16384), map, 64 * hf, head, tok0, bar(PB_XFULL + s));
                if (s == 0) armed[0] = i; else armed[1] = i;
            }
            if (*abort_flag) {                                  // give announced copies a bounded time to land
#pragma unroll
                for (int s = 0; s < 2; ++s)
                    if (armed[s] >= 0) for (int it = 0; it < 512 && !ws_wait(bar(PB_XFULL + s), (armed[s] >> 1) & 1, 1, abort_flag); ++it) __nanosleep(2000);
            }
        }
        __syncwarp();
    } else if (warp == 17) {
        // ---- MMA issue
        if (lane == 0) {
            const unsigned long long t_desc = tc_desc(smem_addr(sm_pt + PT_OFF_T), 128, 2048);
            const unsigned long long x_desc = tc_desc_sw128(smem_addr(sm_pt + PT_OFF_X), 16, 1024);
            PST_DECL;
            for (int i = 0; i < n_my_tiles; ++i) {
                const int s = i & 1;
                PST(0);
                if (!ws_wait(bar((fix_rows ? PB_XREADY : PB_XFULL) + s), (i >> 1) & 1, wait_limit, abort_flag)) break;
                PST(1);
                if (i >= 2 && !ws_wait(bar(PB_DEMPTY + s), ((i >> 1) - 1) & 1, wait_limit, abort_flag)) break;
                PST(2);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned acc = tmem_base + 128u * s;
                for (int term = 0; term < n_terms; ++term) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        tc_mma(acc, x_desc + static_cast<unsigned>((s * PT_X_BYTES + (ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                               t_desc + static_cast<unsigned>((term * (D * D * 2) + ks * 256) >> 4), PT_IDESC, (term > 0 || ks > 0) ? 1u : 0u);
                }
                ws_commit(bar(PB_DFULL + s));
                ws_commit(bar(PB_XEMPTY + s));
                PST(3);
            }
            PST_FLUSH(16);
        }
        __syncwarp();
    } else {
        // ---- epilogue: 16 warps; warp w reads rows 32 (w % 4) .. + 31 (its lanes of tensor memory), channels 32 (w / 4) .. + 31
        constexpr int EPI = 512;
        const int row = 32 * (warp & 3) + lane, cq = warp >> 2;
        const unsigned tmem_row = tmem_base + (static_cast<unsigned>((warp & 3) * 32) << 16) + 32u * cq;
        const long long lo_off = static_cast<long long>(P.total_new) * n_heads * D;
        float* qs_part = reinterpret_cast<float*>(sm_pt + PT_OFF_QS);      // [4][128] partial channel sums
        bool ok = true;
        PST_DECL;
        // AND over the 512 epilogue threads (they meet at named barriers, so they give up together)
        auto together = [&](const bool mine) -> bool {
            unsigned all;
            asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 3, 512, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(all) : "r"(mine ? 1u : 0u) : "memory");
            return all != 0;
        };
        // Projected inputs: the rows of tile i, as the bulk tensor copies left them (128-byte-swizzled rows, channels 0-63 and
        // 64-127 in two boxes), are normalised and rotated in place (Algorithm 2 lines 1-2: fp32, one rounding to bf16)
        // before the MMAs may read them.
        Prologue pro = P.pro;
        pro.weight = is_key ? P.pro.weight : P.q_weight;
        auto fix_tile = [&](const int i) -> bool {
            const int s = i & 1, tok0 = (static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x)) * PREP_TOK;
            PST(5);
            if (!together(ws_wait(bar(PB_XFULL + s), (i >> 1) & 1, wait_limit, abort_flag))) return false;
            PST(6);
            unsigned char* xs = sm_pt + PT_OFF_X + s * PT_X_BYTES;
            // four threads per row: thread q holds channels 16 q .. 16 q + 15 (two 16-byte chunks of the first box) and their
            // rotation partners 64 + 16 q .. (the same chunks of the second box), so that a pair never leaves the thread
            const int r = tid >> 2, q = tid & 3;
            const bool valid = tok0 + r < P.total_new;      // rows past the chunk (zeros) go through the arithmetic and are not stored
            const int tok = valid ? tok0 + r : P.total_new - 1;
            {
                int lo = 0, hi = P.batch, pos;              // the token's sequence by bisection of the chunk bounds, then its position
                if (seq_in_smem) {
                    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (seq_first[mid] <= tok) lo = mid; else hi = mid; }
                    pos = seq_base[lo] + tok;
                } else {
                    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (__ldg(P.cu_new + mid) <= tok) lo = mid; else hi = mid; }
                    const int f0 = __ldg(P.cu_new + lo), n_b = __ldg(P.cu_new + lo + 1) - f0;
                    pos = __ldg(P.seq_len + lo) - n_b + (tok - f0);
                }
                pos = prologue_position(pro, pos, P.c.dev_status, q == 0 && valid);
                uint4* cell[4];                             // [box][chunk]
                uint4 raw[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    cell[k] = reinterpret_cast<uint4*>(xs + (k >> 1) * 16384 + r * 128 + (((2 * q + (k & 1)) ^ (r & 7)) << 4));
                    raw[k] = *cell[k];
                }
                const float4* tab = reinterpret_cast<const float4*>(pro.rope + static_cast<long long>(pos) * (D / 2) + 16 * q);
                float4 cs[8];                               // (cos, sin) of pairs 16 q .. 16 q + 15, two per load
#pragma unroll
                for (int k = 0; k < 8; ++k) cs[k] = __ldg(tab + k);
                float x[4][8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const unsigned w4[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) { x[k][2 * e] = bf16_bits_to_float(w4[e] & 0xffff); x[k][2 * e + 1] = bf16_bits_to_float(w4[e] >> 16); }
                }
                if (pro.normalise) {
                    float ss = 0.f;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
#pragma unroll
                        for (int e = 0; e < 8; ++e) ss = fmaf(x[k][e], x[k][e], ss);
                    ss += __shfl_xor_sync(FULLM, ss, 1);
                    ss += __shfl_xor_sync(FULLM, ss, 2);
                    const float rn = ss > 0.f ? 1.f / sqrtf(ss * (1.f / D) + pro.eps) : 0.f;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        float wv[8] = {1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f};
                        if (pro.weight) {
                            const float4* wp = reinterpret_cast<const float4*>(pro.weight + static_cast<long long>(head) * D + 64 * (k >> 1) + 16 * q + 8 * (k & 1));
                            const float4 wa = __ldg(wp), wb = __ldg(wp + 1);
                            wv[0] = wa.x; wv[1] = wa.y; wv[2] = wa.z; wv[3] = wa.w; wv[4] = wb.x; wv[5] = wb.y; wv[6] = wb.z; wv[7] = wb.w;
                        }
#pragma unroll
                        for (int e = 0; e < 8; ++e) x[k][e] *= pro.weight ? rn * wv[e] : rn;
                    }
                }
#pragma unroll
                for (int k = 0; k < 2; ++k) {               // chunk k of the first box with chunk k of the second
                    unsigned oa[4], ob[4];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float4 c2 = cs[4 * k + (e >> 1)];
                        const float co = (e & 1) ? c2.z : c2.x, si = (e & 1) ? c2.w : c2.y;
                        const float av = x[k][e], bv = x[2 + k][e];
                        const unsigned ya = float_to_bf16_bits(fmaf(av, co, -bv * si)), yb = float_to_bf16_bits(fmaf(av, si, bv * co));
                        if (e & 1) { oa[e >> 1] |= ya << 16; ob[e >> 1] |= yb << 16; } else { oa[e >> 1] = ya; ob[e >> 1] = yb; }
                    }
                    if (valid) {
                        *cell[k] = make_uint4(oa[0], oa[1], oa[2], oa[3]);
                        *cell[2 + k] = make_uint4(ob[0], ob[1], ob[2], ob[3]);
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ws_arrive(bar(PB_XREADY + s));
            PST(7);
            return true;
        };
        if (fix_rows) ok = fix_tile(0);
        for (int i = 0; i < n_my_tiles && ok; ++i) {
            const int s = i & 1, tok0 = (static_cast<int>(blockIdx.x) + i * static_cast<int>(gridDim.x)) * PREP_TOK;
            if (fix_rows && i + 1 < n_my_tiles && !fix_tile(i + 1)) { ok = false; break; }
            PST(0);
            if (!together(ws_wait(bar(PB_DFULL + s), (i >> 1) & 1, wait_limit, abort_flag))) { ok = false; break; }
            PST(1);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float o[32];
            tc_ld32(tmem_row + 128u * s, o);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            ws_arrive(bar(PB_DEMPTY + s));                      // the accumulator is free again
            float sum = 0.f;
            unsigned hi[16], lo[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                if (is_key) {                                   // the cache holds bf16(k')
                    hi[e] = pack_half2(bf16_bits_to_float(float_to_bf16_bits(o[2 * e])), bf16_bits_to_float(float_to_bf16_bits(o[2 * e + 1])));
                    lo[e] = 0u;
                } else {                                        // q' as fp16 value + fp16 rounding remainder
                    hi[e] = pack_half2(o[2 * e], o[2 * e + 1]);
                    const float2 hv = h2f2u(hi[e]);
                    lo[e] = pack_half2(o[2 * e] - hv.x, o[2 * e + 1] - hv.y);
                    const float2 lv = h2f2u(lo[e]);
                    sum += (hv.x + lv.x) + (hv.y + lv.y);
                }
            }
            unsigned char* stage = sm_pt + PT_OFF_OUT + row * PT_OUT_PITCH + 64 * cq;
            // the staged tile leaves as whole rows: 16 consecutive threads per 256-byte row
            auto flush = [&](const unsigned (&w)[16], __half* base) {
#pragma unroll
                for (int e = 0; e < 16; e += 4) *reinterpret_cast<uint4*>(stage + 4 * e) = make_uint4(w[e], w[e + 1], w[e + 2], w[e + 3]);
                asm volatile("bar.sync 2, 512;" ::: "memory");
#pragma unroll
                for (int item = tid; item < PREP_TOK * 16; item += EPI) {
                    const int r = item >> 4, piece = item & 15;
                    if (tok0 + r < P.total_new)
                        *reinterpret_cast<uint4*>(base + (static_cast<long long>(tok0 + r) * n_heads + head) * D + 8 * piece) =
                            *reinterpret_cast<const uint4*>(sm_pt + PT_OFF_OUT + r * PT_OUT_PITCH + 16 * piece);
                }
                asm volatile("bar.sync 2, 512;" ::: "memory");
            };
            if (!is_key) qs_part[cq * PREP_TOK + row] = sum;
            PST(2);
            flush(hi, is_key ? P.KP : P.QP);
            PST(3);
            if (!is_key) {
                flush(lo, P.QP + lo_off);
                PST(4);
                if (cq == 0 && tok0 + row < P.total_new)
                    P.qsum[static_cast<long long>(tok0 + row) * P.c.n_q + head] =
                        (qs_part[row] + qs_part[PREP_TOK + row]) + (qs_part[2 * PREP_TOK + row] + qs_part[3 * PREP_TOK + row]);
            }
        }
        if (warp == 0) PST_FLUSH(0);
    }

    __syncthreads();
#if WUSHKV_WS_TIMING
    if (tid == 0 && blockIdx.x == 0 && blockIdx.y == gridDim.y - 1) g_ws_t[9] += clock64() - t_entry;
#endif
    if (*abort_flag && tid == 544) {                            // the issuing thread: let whatever was issued finish (bounded) before the release
        atomicOr(P.c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
        ws_commit(bar(PB_DRAIN));
        for (int it = 0; it < 512 && !ws_wait(bar(PB_DRAIN), 0u, 1, abort_flag); ++it) __nanosleep(2000);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct PrefillPlan { size_t off_kp, off_vp, off_qp, off_qsum, off_part, total; int max_split; };
bool make_prefill_plan(const CacheView& c, int total_new, PrefillPlan& pl) {
    if (total_new <= 0) return false;
    size_t off = 0;
    pl.off_kp = off;   off = align256(off + static_cast<size_t>(total_new) * c.n_kv * D * sizeof(__half));
    pl.off_vp = off;   off = align256(off + static_cast<size_t>(total_new) * c.n_kv * D * sizeof(__half));
    pl.off_qp = off;   off = align256(off + 2 * static_cast<size_t>(total_new) * c.n_q * D * sizeof(__half));
    pl.off_qsum = off; off = align256(off + static_cast<size_t>(total_new) * c.n_q * sizeof(float));
    // Partial results of the warp-specialised attention kernel when a call has too few tile pairs to fill the GPU: at
    // least ceil(total_new / (2 R)) pairs per KV head exist, so at most sm_count / that many CTAs per pair are worth it.
    const int R = 128 / c.G;
    const long long min_ctas = (static_cast<long long>(total_new) + 2 * R - 1) / (2 * R) * c.n_kv;
    pl.max_split = static_cast<int>(std::max<long long>(1, std::min<long long>(16, sm_count() / std::max<long long>(min_ctas, 1))));
    pl.off_part = off;
    if (pl.max_split > 1) off = align256(off + static_cast<size_t>(pl.max_split) * total_new * c.n_q * 132 * sizeof(float));
    pl.total = off;
    return true;
}

}  // namespace
}  // namespace wushkv

using namespace wushkv;

extern "C" size_t wushkv_prefill_workspace_bytes(const wushkv_cache* cache, int32_t batch, int32_t total_new) {
    CacheView v;
    if (make_view(cache, v) != WUSHKV_OK || batch <= 0) return 0;
    PrefillPlan pl;
    if (!make_prefill_plan(v, total_new, pl)) return 0;
    return pl.total;
}

static int prefill_attn_impl(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                             const int32_t* cu_new, int32_t total_new, int32_t max_new,
                             const uint16_t* K_new, const uint16_t* V_new, const uint16_t* Q_new, float* O,
                             void* workspace, size_t workspace_bytes, void* stream, const wushkv_prologue* prologue) {
    PrefillParams P;
    const int rc = make_view(cache, P.c);
    if (rc != WUSHKV_OK) return rc;
    P.pro = Prologue{nullptr, 0, 0, nullptr, 0.f};
    P.q_weight = nullptr;
    if (prologue) {
        if (!make_prologue(prologue, prologue->k_norm_weight, P.pro) || (reinterpret_cast<uintptr_t>(prologue->q_norm_weight) & 15)) return WUSHKV_EINVAL;
        P.q_weight = prologue->q_norm_weight;
    }
    if (batch <= 0 || !slot || !seq_len || !cu_new || total_new < 0 || max_new < 0 || max_new > total_new) return WUSHKV_EINVAL;
    if (total_new == 0) return WUSHKV_OK;
    if (!K_new || !V_new || !Q_new || !O || !workspace || !aligned(K_new, 16) || !aligned(V_new, 16) || !aligned(Q_new, 16) ||
        !aligned(O, 16) || !aligned(workspace, 256))
        return WUSHKV_EINVAL;
    PrefillPlan pl;
    if (!make_prefill_plan(P.c, total_new, pl)) return WUSHKV_EINVAL;
    if (workspace_bytes < pl.total) return WUSHKV_ECAPACITY;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    P.batch = batch; P.total_new = total_new; P.slot = slot; P.seq_len = seq_len; P.cu_new = cu_new;
    P.K_new = K_new; P.V_new = V_new; P.Q_new = Q_new; P.O = O;
    P.use_tma = 0;
    P.n_split = 1;
    P.part = nullptr;
    P.wait_limit = static_cast<int>(std::min<long long>(std::max<long long>(knobs().wait_limit, 0), 1 << 30));
    P.drop = knobs().drop_prefill;
    P.KP = reinterpret_cast<__half*>(ws + pl.off_kp);
    P.VP = reinterpret_cast<__half*>(ws + pl.off_vp);
    P.QP = reinterpret_cast<__half*>(ws + pl.off_qp);
    P.qsum = reinterpret_cast<float*>(ws + pl.off_qsum);
    P.tiles_per_seq = (max_new + BM - 1) / BM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem_prep = static_cast<size_t>(PREP_TOK + 3 * D) * PREP_PITCH * sizeof(unsigned short);
    if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(prefill_prep_kernel), static_cast<int>(smem_prep))) return WUSHKV_ECUDA;
    {   // about one wave of CTAs: each keeps its head's transform resident and walks over token tiles
        const int n_tok_tiles = (total_new + PREP_TOK - 1) / PREP_TOK, slots = P.c.n_kv + P.c.n_q;
        const int per_slot = std::max(1, std::min(n_tok_tiles, sm_count() / slots));
        // the tcgen05 kernel, fed by bulk tensor copies of the bf16 rows as they come (projected rows are normalised and
        // rotated in shared memory before the MMAs read them)
        CUtensorMap in_k, in_q;
        const bool tc_prep = !knobs().prefill_legacy && !knobs().prefill_no_tma &&
                             make_row_tensor_map(in_k, true, K_new, P.c.n_kv, total_new, PREP_TOK) &&
                             make_row_tensor_map(in_q, true, Q_new, P.c.n_q, total_new, PREP_TOK) &&
                             opt_in_dynamic_smem(reinterpret_cast<const void*>(prefill_prep_tc_kernel), PT_SMEM);
        if (tc_prep) {      // head slots: key heads, query heads, then one per KV head for the values
            const int slots_tc = slots + P.c.n_kv, per_slot_tc = std::max(1, std::min(n_tok_tiles, sm_count() / slots_tc));
            prefill_prep_tc_kernel<<<dim3(per_slot_tc, slots_tc), PT_THREADS, PT_SMEM, st>>>(P, in_k, in_q);
        }
#if WUSHKV_WS_TIMING
        if (tc_prep) {
            cudaDeviceSynchronize();
            unsigned long long t[32];
            cudaMemcpyFromSymbol(t, g_ws_t, sizeof(t));
            std::fprintf(stderr, "prep timing epilogue:");
            for (int i = 0; i < 10; ++i) std::fprintf(stderr, " %llu", t[i]);
            std::fprintf(stderr, "\nprep timing mma:");
            for (int i = 16; i < 24; ++i) std::fprintf(stderr, " %llu", t[i]);
            std::fprintf(stderr, "\n");
            std::memset(t, 0, sizeof(t));
            cudaMemcpyToSymbol(g_ws_t, t, sizeof(t));
        }
#endif
        else prefill_prep_kernel<<<dim3(per_slot, slots), 256, smem_prep, st>>>(P);
    }
    if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
    if (!knobs().prefill_legacy) {              // tcgen05 path: the G heads of a KV head share a 128-row tile
        const int R = TM / P.c.G;
        P.tiles_per_seq = (max_new + R - 1) / R;
        const dim3 grid_tc(static_cast<unsigned>(batch) * P.tiles_per_seq, P.c.n_kv);
        // tensor maps of the chunk's fp16 keys and values, [token][head][128 channels], boxes of 64 tokens x 64 channels
        // written as 128-byte-swizzled rows; without the driver entry point the kernel stages with 16-byte copies
        CUtensorMap map_k, map_v;
        const bool mk = make_row_tensor_map(map_k, false, P.KP, P.c.n_kv, total_new, TN);
        const bool mv = make_row_tensor_map(map_v, false, P.VP, P.c.n_kv, total_new, TN);
        P.use_tma = (mk && mv && !knobs().prefill_no_tma) ? 1 : 0;
        if (!knobs().prefill_one_tile) {        // warp-specialised kernel: a pair of query tiles per CTA
            // few pairs (a short chunk): several CTAs per pair, each over a share of the key tiles, then a merge
            const long long n_pairs = static_cast<long long>(batch) * ((P.tiles_per_seq + 1) / 2) * P.c.n_kv;
            int n_split = static_cast<int>(std::max<long long>(1, std::min<long long>(pl.max_split, sm_count() / std::max<long long>(n_pairs, 1))));
            if (knobs().prefill_split > 0) n_split = std::min(knobs().prefill_split, pl.max_split);
            P.n_split = n_split;
            P.part = reinterpret_cast<float*>(ws + pl.off_part);
            const dim3 grid_ws(static_cast<unsigned>(batch) * ((P.tiles_per_seq + 1) / 2) * n_split, P.c.n_kv);
            // the query operands (value, remainder) as [token][query head][128 channels]: a box is one tile's (G heads, R positions)
            CUtensorMap map_q0, map_q1;
            const bool mq = make_row_tensor_map(map_q0, false, P.QP, P.c.n_q, total_new, R, P.c.G) &&
                            make_row_tensor_map(map_q1, false, P.QP + static_cast<size_t>(total_new) * P.c.n_q * D, P.c.n_q, total_new, R, P.c.G);
            if (!mq) P.use_tma = 0;
            auto launch_ws = [&](auto kernel, const int smem) -> bool {
                if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(kernel), smem)) return false;
                kernel<<<grid_ws, WS_THREADS, smem, st>>>(P, map_k, map_v, map_q0, map_q1);
                return true;
            };
            const bool ok = P.c.bits == 2   ? launch_ws(prefill_attn_ws_kernel<2>, ws_smem(2))
                            : P.c.bits == 3 ? launch_ws(prefill_attn_ws_kernel<3>, ws_smem(3))
                                            : launch_ws(prefill_attn_ws_kernel<4>, ws_smem(4));
            if (!ok) return WUSHKV_ECUDA;
            if (n_split > 1) prefill_merge_kernel<<<dim3(total_new, P.c.n_q), D, 0, st>>>(P);
#if WUSHKV_WS_TIMING
            {
                cudaDeviceSynchronize();
                unsigned long long t[32];
                cudaMemcpyFromSymbol(t, g_ws_t, sizeof(t));
                std::fprintf(stderr, "ws timing softmax:");
                for (int i = 0; i < 16; ++i) std::fprintf(stderr, " %llu", t[i]);
                std::fprintf(stderr, "\nws timing mma:");
                for (int i = 16; i < 32; ++i) std::fprintf(stderr, " %llu", t[i]);
                std::fprintf(stderr, "\n");
                std::memset(t, 0, sizeof(t));
                cudaMemcpyToSymbol(g_ws_t, t, sizeof(t));
            }
#endif
            return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
        }
        auto launch = [&](auto kernel) -> bool {
            if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(kernel), TC_SMEM)) return false;
            kernel<<<grid_tc, TM, TC_SMEM, st>>>(P, map_k, map_v);
            return true;
        };
        const bool ok = P.c.bits == 2 ? launch(prefill_attn_tc_kernel<2>) : P.c.bits == 3 ? launch(prefill_attn_tc_kernel<3>)
                                                                                         : launch(prefill_attn_tc_kernel<4>);
        if (!ok) return WUSHKV_ECUDA;
        return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
    }
    const dim3 grid(static_cast<unsigned>(batch) * P.tiles_per_seq, P.c.n_q);
    const size_t smem_attn = sizeof(TileSmem);
    if (P.c.bits == 2) {
        if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(prefill_attn_kernel<2>), static_cast<int>(smem_attn))) return WUSHKV_ECUDA;
        prefill_attn_kernel<2><<<grid, PF_THREADS, smem_attn, st>>>(P);
    } else if (P.c.bits == 3) {
        if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(prefill_attn_kernel<3>), static_cast<int>(smem_attn))) return WUSHKV_ECUDA;
        prefill_attn_kernel<3><<<grid, PF_THREADS, smem_attn, st>>>(P);
    } else {
        if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(prefill_attn_kernel<4>), static_cast<int>(smem_attn))) return WUSHKV_ECUDA;
        prefill_attn_kernel<4><<<grid, PF_THREADS, smem_attn, st>>>(P);
    }
    return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
}

extern "C" int wushkv_prefill_attn(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                   const int32_t* cu_new, int32_t total_new, int32_t max_new,
                                   const uint16_t* K_new, const uint16_t* V_new, const uint16_t* Q_new, float* O,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    return prefill_attn_impl(cache, batch, slot, seq_len, cu_new, total_new, max_new, K_new, V_new, Q_new, O, workspace, workspace_bytes,
                             stream, nullptr);
}

extern "C" int wushkv_prefill_attn_projected(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                             const int32_t* cu_new, int32_t total_new, int32_t max_new,
                                             const uint16_t* K_proj, const uint16_t* V_new, const uint16_t* Q_proj,
                                             const wushkv_prologue* prologue, float* O,
                                             void* workspace, size_t workspace_bytes, void* stream) {
    if (!prologue) return WUSHKV_EINVAL;
    return prefill_attn_impl(cache, batch, slot, seq_len, cu_new, total_new, max_new, K_proj, V_new, Q_proj, O, workspace, workspace_bytes,
                             stream, prologue);
}
