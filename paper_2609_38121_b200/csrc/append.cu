// Quantize-on-append (Algorithm 2 lines 3-4 and 9-12; quantizer: Section 5.3 Eq. 6).
//
// Three kernels, chosen by wushkv_append from the shape of the call:
//   append_chunk_kernel  prefill chunks (max_new >= 128): key transform on tcgen05, four lanes per vector
//                        for the quantizer (described where it is defined, further down);
//   append_token_kernel  one token per sequence (a decode step): one CTA per sequence, single launch;
//   append_rows_kernel   everything else, and the chunk path when WUSHKV_APPEND_PATH=cuda.
// The last two share the warp-per-vector path: one warp owns one (new token, KV head) pair.  It computes k' = T_K k on
// CUDA cores against a transposed copy of T_K in shared memory (keys only), then for k' and for v:
// finds the clip range (min, max and the two order statistics around rank kappa*(d-1) of |x| by
// repeated warp-wide maximum extraction), derives the fp16 step / offset, rounds the codes with
// the STORED step and offset, and scatters the codes into the fragment-ordered page record.
// The bf16 copies for the sink buffer and the recent ring are written by the same warp.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>

#include "host_common.h"
#include "prologue.cuh"
#include "layout.cuh"

namespace wushkv {

constexpr unsigned FULL = 0xffffffffu;
constexpr int TT_STRIDE = 132;   // floats per row of the transposed transform in shared memory
// The decode kernel feeds (probability x value step) to the tensor core in fp16 with 2^6 of headroom:
// a stored value step at or beyond this limit can saturate there, so the append flags it.
constexpr float VALUE_STEP_LIMIT = 1024.f;

struct ClipRule {     // how the step and offset of a group are chosen
    int rounds;       // Eq. 6: extraction rounds of quantile_kappa(|x|): the last yields a[lo], the one before a[lo+1]
    float frac;       // Eq. 6: pos - lo of the linear interpolation
    float quest;      // Eq. 5 (QuEST) when > 0: 2 alpha_b / ((2^b - 1) sqrt(d)), the step per unit norm; 0 selects Eq. 6
};

struct AppendParams {
    CacheView c;
    int batch, total_new, tokens_per_cta;
    const int* slot;
    int* seq_len;
    const int* cu_new;
    const unsigned short* K_new;
    const unsigned short* V_new;
    ClipRule rule_k, rule_v;
    int wait_limit;          // poll limit of the chunk kernel's MMA barrier wait (0: default, about two seconds)
    int drop_mma_commit;     // testing aid: the first tile's MMAs are never committed to their barrier
    Prologue pro;            // pro.rope != nullptr: K_new holds projected keys, normalised and rotated here (Algorithm 2 lines 1-2)
    int use_tma;             // 1: the chunk kernel stages its key / value tiles with bulk tensor copies (128-byte-swizzled rows)
};

__device__ __forceinline__ void cswap_desc(unsigned& a, unsigned& b) {
    const unsigned hi = max(a, b), lo = min(a, b);
    a = hi; b = lo;
}

__device__ __forceinline__ unsigned order_key(float x) {       // monotone float -> uint map
    const unsigned u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float order_key_inv(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Eq. 6 for the 128-vector held as x[4] per lane (channels 4*lane .. 4*lane+3).  Returns the four
// codes of this lane and the stored (fp16) step and offset.
template <int BITS>
__device__ __forceinline__ void quantize_vec(const float (&x)[4], ClipRule rule, int lane, int (&code)[4],
                                             __half& step_h, __half& xmin_h, int* value_status = nullptr) {
    constexpr int LEVELS = (1 << BITS) - 1;
    if (rule.quest > 0.f) {
        // Eq. 5: step from the group's norm, bin index floor(x / step) in [-2^(b-1), 2^(b-1) - 1], offset -step (2^b - 1) / 2
        float ss = x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3];
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(FULL, ss, o);
        step_h = __float2half_rn(fminf(rule.quest * sqrtf(ss), 65504.f));
        const float step_s = __half2float(step_h);
        xmin_h = __float2half_rn(-0.5f * static_cast<float>(LEVELS) * step_s);
        if (value_status != nullptr && step_s >= VALUE_STEP_LIMIT && lane == 0) atomicOr(value_status, WUSHKV_DEV_VALUE_RANGE);
        const float inv = step_s > 0.f ? __frcp_rn(step_s) : 0.f;
        constexpr float HALF = static_cast<float>(1 << (BITS - 1));
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float t = floorf(x[e] * inv) + HALF;
            code[e] = step_s > 0.f ? static_cast<int>(fminf(fmaxf(t, 0.f), static_cast<float>(LEVELS))) : 0;
        }
        if (!(step_s > 0.f)) xmin_h = __float2half_rn(0.f);
        return;
    }
    // ---- the two order statistics of |x| around rank kappa*(d-1)
    unsigned u0 = __float_as_uint(x[0]) & 0x7fffffffu, u1 = __float_as_uint(x[1]) & 0x7fffffffu;
    unsigned u2 = __float_as_uint(x[2]) & 0x7fffffffu, u3 = __float_as_uint(x[3]) & 0x7fffffffu;
    cswap_desc(u0, u1); cswap_desc(u2, u3); cswap_desc(u0, u2); cswap_desc(u1, u3); cswap_desc(u1, u2);
    unsigned a_lo = 0, a_hi = 0;
    for (int r = 0; r < rule.rounds; ++r) {
        const unsigned m = __reduce_max_sync(FULL, u0);
        const unsigned owners = __ballot_sync(FULL, u0 == m);
        if (lane == __ffs(owners) - 1) { u0 = u1; u1 = u2; u2 = u3; u3 = 0; }
        a_hi = a_lo;
        a_lo = m;
    }
    if (rule.rounds == 1) a_hi = a_lo;
    const float alo = __uint_as_float(a_lo), ahi = __uint_as_float(a_hi);
    const float q = alo + rule.frac * (ahi - alo);
    // ---- extremes of x
    const float lmin = fminf(fminf(x[0], x[1]), fminf(x[2], x[3]));
    const float lmax = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    const float vmin = order_key_inv(__reduce_min_sync(FULL, order_key(lmin)));
    const float vmax = order_key_inv(__reduce_max_sync(FULL, order_key(lmax)));
    const float x_min = fmaxf(vmin, -q);
    const float x_max = fminf(vmax, q);
    const float step = __fdiv_rn(x_max - x_min, static_cast<float>(LEVELS));
    step_h = __float2half_rn(fminf(fmaxf(step, -65504.f), 65504.f));
    xmin_h = __float2half_rn(fminf(fmaxf(x_min, -65504.f), 65504.f));
    const float step_s = __half2float(step_h), xmin_s = __half2float(xmin_h);
    if (value_status != nullptr && step_s >= VALUE_STEP_LIMIT && lane == 0) atomicOr(value_status, WUSHKV_DEV_VALUE_RANGE);
    const float inv = step_s > 0.f ? __frcp_rn(step_s) : 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float t = rintf((x[e] - xmin_s) * inv);
        code[e] = static_cast<int>(fminf(fmaxf(t, 0.f), static_cast<float>(LEVELS)));
    }
}

// Scatter one token's K codes (lane holds channels 4*lane..+3) into the record; r = token row in page.
// Channel 4 lane + e sits in k-step s = lane >> 3, channel half hh = (lane >> 2) & 1, byte 2 ((lane >> 1) & 1) + (e & 1)
// of the word of fragment lane t = 2 (lane & 1) + (e >> 1).
template <int BITS>
__device__ __forceinline__ void store_k_codes(unsigned char* rec, int r, const int (&code)[4], int lane) {
    constexpr bool PLANES = BITS == 3;                  // 3 bits: low two bits here (2-bit layout), high bit below
    constexpr bool TWO = BITS == 2 || BITS == 3;
    const int bi = r >> 4, rr = r & 15, g = rr & 7, rs = rr >> 3;
    const int s = lane >> 3, b0 = 2 * ((lane >> 1) & 1);
    const int sh = 8 * b0 + (TWO ? 2 * s : 4 * (s & 1));
    const unsigned lowmask = PLANES ? 3u : 0xFu;
    unsigned wa = ((static_cast<unsigned>(code[0]) & lowmask) << sh) | ((static_cast<unsigned>(code[1]) & lowmask) << (8 + sh));   // t = 2 (lane & 1)
    unsigned wb = ((static_cast<unsigned>(code[2]) & lowmask) << sh) | ((static_cast<unsigned>(code[3]) & lowmask) << (8 + sh));   // t = 2 (lane & 1) + 1
    wa |= __shfl_xor_sync(FULL, wa, 2);  wb |= __shfl_xor_sync(FULL, wb, 2);       // the other byte pair
    wa |= __shfl_xor_sync(FULL, wa, 8);  wb |= __shfl_xor_sync(FULL, wb, 8);       // the fields / nibbles of the same byte
    if (TWO) { wa |= __shfl_xor_sync(FULL, wa, 16); wb |= __shfl_xor_sync(FULL, wb, 16); }
    const int hh = (lane >> 2) & 1, ta = 2 * (lane & 1), j = rs + 2 * hh;
    const bool writer = TWO ? (lane & 26) == 0 : (lane & 10) == 0;
    if (writer) {
        unsigned char* p = rec + bi * code_block_bytes(BITS) + (BITS == 4 ? 512 * (lane >> 4) : 0) + 16 * (4 * g + ta) + 4 * j;
        *reinterpret_cast<unsigned*>(p) = wa;
        *reinterpret_cast<unsigned*>(p + 16) = wb;
    }
    if (PLANES) {                                       // 1-bit plane: word rs of lane (g,t), byte b, bit 2s + hh
        const int shb = 8 * b0 + 2 * s + hh;
        unsigned ha = ((static_cast<unsigned>(code[0]) >> 2) << shb) | ((static_cast<unsigned>(code[1]) >> 2) << (8 + shb));
        unsigned hb = ((static_cast<unsigned>(code[2]) >> 2) << shb) | ((static_cast<unsigned>(code[3]) >> 2) << (8 + shb));
#pragma unroll
        for (int o = 2; o <= 16; o <<= 1) { ha |= __shfl_xor_sync(FULL, ha, o); hb |= __shfl_xor_sync(FULL, hb, o); }
        if ((lane & 30) == 0) {
            unsigned char* p = rec + k_hi_offset(3) + bi * 256 + 8 * (4 * g + ta) + 4 * rs;
            *reinterpret_cast<unsigned*>(p) = ha;
            *reinterpret_cast<unsigned*>(p + 8) = hb;
        }
    }
}

template <int BITS>
__device__ __forceinline__ void store_v_codes(unsigned char* rec, int r, const int (&code)[4], int lane) {
    constexpr bool PLANES = BITS == 3;
    constexpr bool TWO = BITS == 2 || BITS == 3;
    const int bi = r >> 4, rr = r & 15, ps = rr >> 3, t = (rr & 7) >> 1, hi = rr & 1;
    const int i = lane >> 2;                            // channel block of this lane's channels
    const int sh = TWO ? 2 * i : 4 * (i & 3);
    const unsigned lowmask = PLANES ? 3u : 0xFu;
    unsigned wa = ((static_cast<unsigned>(code[0]) & lowmask) << sh) | ((static_cast<unsigned>(code[1]) & lowmask) << (16 + sh));
    unsigned wb = ((static_cast<unsigned>(code[2]) & lowmask) << sh) | ((static_cast<unsigned>(code[3]) & lowmask) << (16 + sh));
    wa |= __shfl_xor_sync(FULL, wa, 4);  wb |= __shfl_xor_sync(FULL, wb, 4);
    wa |= __shfl_xor_sync(FULL, wa, 8);  wb |= __shfl_xor_sync(FULL, wb, 8);
    if (TWO) { wa |= __shfl_xor_sync(FULL, wa, 16); wb |= __shfl_xor_sync(FULL, wb, 16); }
    const int rsel = (lane & 3) >> 1, g0 = 4 * (lane & 1);
    unsigned char* base;
    bool writer;
    if (TWO) {
        writer = lane < 4;
        base = rec + v_codes_offset(BITS) + bi * 512 + 4 * (2 * ps + rsel) + 2 * hi;
    } else {
        writer = (lane & 12) == 0;
        base = rec + v_codes_offset(4) + bi * 1024 + 512 * ps + 4 * (2 * rsel + (lane >> 4)) + 2 * hi;
    }
    if (writer) {
        *reinterpret_cast<unsigned short*>(base + 16 * (4 * (g0 + 0) + t)) = static_cast<unsigned short>(wa & 0xffffu);
        *reinterpret_cast<unsigned short*>(base + 16 * (4 * (g0 + 1) + t)) = static_cast<unsigned short>(wa >> 16);
        *reinterpret_cast<unsigned short*>(base + 16 * (4 * (g0 + 2) + t)) = static_cast<unsigned short>(wb & 0xffffu);
        *reinterpret_cast<unsigned short*>(base + 16 * (4 * (g0 + 3) + t)) = static_cast<unsigned short>(wb >> 16);
    }
    if (PLANES) {                                       // 1-bit plane: half-word hi of word ps of lane (g,t), bit v1_bit(rsel, i)
        const int shb = v1_bit(rsel, i);
        unsigned ha = ((static_cast<unsigned>(code[0]) >> 2) << shb) | ((static_cast<unsigned>(code[1]) >> 2) << (16 + shb));
        unsigned hb = ((static_cast<unsigned>(code[2]) >> 2) << shb) | ((static_cast<unsigned>(code[3]) >> 2) << (16 + shb));
#pragma unroll
        for (int o = 2; o <= 16; o <<= 1) { ha |= __shfl_xor_sync(FULL, ha, o); hb |= __shfl_xor_sync(FULL, hb, o); }
        if (lane < 2) {
            unsigned char* hbase = rec + v_hi_offset(3) + bi * 256 + 4 * ps + 2 * hi;
            *reinterpret_cast<unsigned short*>(hbase + 8 * (4 * (g0 + 0) + t)) = static_cast<unsigned short>(ha & 0xffffu);
            *reinterpret_cast<unsigned short*>(hbase + 8 * (4 * (g0 + 1) + t)) = static_cast<unsigned short>(ha >> 16);
            *reinterpret_cast<unsigned short*>(hbase + 8 * (4 * (g0 + 2) + t)) = static_cast<unsigned short>(hb & 0xffffu);
            *reinterpret_cast<unsigned short*>(hbase + 8 * (4 * (g0 + 3) + t)) = static_cast<unsigned short>(hb >> 16);
        }
    }
}

// Where a new token goes; false (with a status bit) if it cannot be stored.
struct TokenSlot {
    int b, slot, pos, s_final;
    unsigned char* rec;      // this head's record of the token's page
    int r;                   // row inside the page
};

__device__ __forceinline__ bool locate_token(const AppendParams& P, int token, int head, TokenSlot& ts) {
    int lo = 0, hi = P.batch;                 // largest b with cu_new[b] <= token
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(P.cu_new + mid) <= token) lo = mid; else hi = mid;
    }
    ts.b = lo;
    ts.slot = __ldg(P.slot + lo);
    const int s0 = __ldg(P.seq_len + lo);
    const int first = __ldg(P.cu_new + lo), last = __ldg(P.cu_new + lo + 1);
    ts.pos = s0 + (token - first);
    ts.s_final = s0 + (last - first);
    if (ts.slot < 0 || ts.slot >= P.c.n_slots || s0 < 0) { atomicOr(P.c.dev_status, WUSHKV_DEV_BAD_SLOT); return false; }
    const int pidx = ts.pos / PAGE_TOKENS;
    if (pidx >= P.c.max_pages) { atomicOr(P.c.dev_status, WUSHKV_DEV_PAGE_TABLE_FULL); return false; }
    const int page = __ldg(P.c.page_table + static_cast<long long>(ts.slot) * P.c.max_pages + pidx);
    if (page < 0 || page >= P.c.n_pages) { atomicOr(P.c.dev_status, WUSHKV_DEV_BAD_PAGE_ID); return false; }
    ts.rec = P.c.pages + (static_cast<long long>(page) * P.c.n_kv + head) * record_bytes(P.c.bits);
    ts.r = ts.pos % PAGE_TOKENS;
    return true;
}

// bf16 copies for the sink buffer and the recent ring (Section 4.4): which = 0 keys, 1 values.
__device__ __forceinline__ void store_window_copy(const AppendParams& P, const TokenSlot& ts, int head, int which,
                                                  uint2 four_bf16, int lane) {
    const CacheView& c = P.c;
    if (ts.pos < c.s_sink) {
        unsigned short* dst = c.sink_kv + (((static_cast<long long>(ts.slot) * c.n_kv + head) * 2 + which) * c.s_sink + ts.pos) * D;
        reinterpret_cast<uint2*>(dst)[lane] = four_bf16;
    }
    if (ts.pos >= ts.s_final - c.ring_cap) {
        unsigned short* dst = c.ring_kv + (((static_cast<long long>(ts.slot) * c.n_kv + head) * 2 + which) * c.ring_cap + ts.pos % c.ring_cap) * D;
        reinterpret_cast<uint2*>(dst)[lane] = four_bf16;
    }
}

template <int BITS>
__global__ void __launch_bounds__(256) append_rows_kernel(AppendParams P) {
    extern __shared__ __align__(16) float Tt[];          // Tt[j * TT_STRIDE + i] = T[i][j]
    const int head = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const float* T = P.c.T_K + static_cast<long long>(head) * D * D;
    for (int idx = threadIdx.x; idx < D * D; idx += blockDim.x) {
        const int i = idx >> 7, j = idx & 127;
        Tt[j * TT_STRIDE + i] = __ldg(T + idx);
    }
    __syncthreads();
    const int tok0 = blockIdx.x * P.tokens_per_cta;
    const int tok1 = min(tok0 + P.tokens_per_cta, P.total_new);
    for (int token = tok0 + warp; token < tok1; token += nwarps) {
        TokenSlot ts;
        if (!locate_token(P, token, head, ts)) continue;
        const long long row = (static_cast<long long>(token) * P.c.n_kv + head) * D;
        // ---------------- keys: k' = T k (Algorithm 2 line 3), fp32 accumulation of exact bf16 products
        const uint2 kraw = __ldg(reinterpret_cast<const uint2*>(P.K_new + row) + lane);
        float kin[4] = {bf16_bits_to_float(kraw.x & 0xffff), bf16_bits_to_float(kraw.x >> 16),
                        bf16_bits_to_float(kraw.y & 0xffff), bf16_bits_to_float(kraw.y >> 16)};
        if (P.pro.rope) norm_rope_warp(kin, lane, P.pro, head, prologue_position(P.pro, ts.pos, P.c.dev_status, lane == 0));
        float x[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int jj = 0; jj < 32; ++jj) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float kj = __shfl_sync(FULL, kin[e], jj);
                const float4 tt = *reinterpret_cast<const float4*>(Tt + (4 * jj + e) * TT_STRIDE + 4 * lane);
                x[0] = fmaf(tt.x, kj, x[0]); x[1] = fmaf(tt.y, kj, x[1]);
                x[2] = fmaf(tt.z, kj, x[2]); x[3] = fmaf(tt.w, kj, x[3]);
            }
        }
        int code[4];
        __half step_h, xmin_h;
        quantize_vec<BITS>(x, P.rule_k, lane, code, step_h, xmin_h);
        store_k_codes<BITS>(ts.rec, ts.r, code, lane);
        __half* meta = reinterpret_cast<__half*>(ts.rec + meta_location(BITS, ts.r));
        if (lane == 0) { meta[0] = step_h; meta[1] = xmin_h; }
        uint2 kb;
        kb.x = float_to_bf16_bits(x[0]) | (static_cast<unsigned>(float_to_bf16_bits(x[1])) << 16);
        kb.y = float_to_bf16_bits(x[2]) | (static_cast<unsigned>(float_to_bf16_bits(x[3])) << 16);
        store_window_copy(P, ts, head, 0, kb, lane);
        // ---------------- values: already in the folded basis, no transform
        const uint2 vraw = __ldg(reinterpret_cast<const uint2*>(P.V_new + row) + lane);
        float v[4] = {bf16_bits_to_float(vraw.x & 0xffff), bf16_bits_to_float(vraw.x >> 16),
                      bf16_bits_to_float(vraw.y & 0xffff), bf16_bits_to_float(vraw.y >> 16)};
        quantize_vec<BITS>(v, P.rule_v, lane, code, step_h, xmin_h, P.c.dev_status);
        store_v_codes<BITS>(ts.rec, ts.r, code, lane);
        if (lane == 0) { meta[2] = step_h; meta[3] = xmin_h; }
        store_window_copy(P, ts, head, 1, vraw, lane);
    }
}

// Decode-time append: exactly one new token per sequence (or none).  One CTA of four warps per (KV head,
// sequence); the CTAs of a sequence form a thread-block cluster.  Every warp computes 32 outputs of
// k' = T_K k as row dot products (the rows of T_K come straight from L2, 64 KB per CTA, so the read is
// spread over n_kv SMs per sequence instead of one), then one warp quantizes and packs the key, another
// the value.  The cluster is the only reader of its sequence's length, so it also advances it: every CTA
// reads the old length, the cluster meets at its barrier, then the first CTA stores the new one.
template <int BITS>
__global__ void __launch_bounds__(128) append_token_kernel(AppendParams P) {
    __shared__ __align__(16) float kin_s[D];             // input key
    __shared__ __align__(16) float kp_s[D];              // transformed key
    // Launched programmatically: the CTAs may be resident before the kernel ahead in the stream has
    // finished, so wait for it (and its memory) first; then let the next kernel's CTAs come in early
    // too (that kernel waits for this one itself).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int head = blockIdx.x, b = blockIdx.y;
    const int n_kv = P.c.n_kv;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int first = __ldg(P.cu_new + b), n_new = __ldg(P.cu_new + b + 1) - first;
    const int s0 = n_new > 0 ? P.seq_len[b] : 0;         // written by this cluster: not through the read-only path
    // every CTA of the sequence has read the old length once all have arrived here
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    bool ok = n_new == 1;
    if (n_new > 1 && threadIdx.x == 0 && head == 0) atomicOr(P.c.dev_status, WUSHKV_DEV_BAD_COUNT);   // the host promised one token per sequence
    int slot0 = 0, page = -1;
    if (ok) {
        slot0 = __ldg(P.slot + b);                       // the page lookup does not depend on the transform: start it now
        if (slot0 >= 0 && slot0 < P.c.n_slots && s0 >= 0 && s0 / PAGE_TOKENS < P.c.max_pages)
            page = __ldg(P.c.page_table + static_cast<long long>(slot0) * P.c.max_pages + s0 / PAGE_TOKENS);
    }
    if (ok) {
        const long long row0 = (static_cast<long long>(first) * n_kv + head) * D;
        // the warp that will quantize the value vector requests it now; it is used after the transform
        uint2 v_pre = make_uint2(0u, 0u);
        if (warp == 1) v_pre = __ldg(reinterpret_cast<const uint2*>(P.V_new + row0) + lane);
        kin_s[threadIdx.x] = bf16_bits_to_float(__ldg(P.K_new + row0 + threadIdx.x));
        __syncthreads();
        if (P.pro.rope) {                                // projected keys: Norm and RoPE first
            if (warp == 0) {
                float4* kv = reinterpret_cast<float4*>(kin_s) + lane;
                const float4 v = *kv;
                float x[4] = {v.x, v.y, v.z, v.w};
                norm_rope_warp(x, lane, P.pro, head, prologue_position(P.pro, s0, P.c.dev_status, lane == 0 && head == 0));
                *kv = make_float4(x[0], x[1], x[2], x[3]);
            }
            __syncthreads();
        }
        // k'[i] = sum_j T[i][j] k[j]: a warp takes 32 consecutive rows; every row is read as one coalesced
        // 512-byte line (lane L holds columns 4L..4L+3), the 32 partial sums per lane are then reduced across
        // lanes with a transposing butterfly.
        {
            const int r0 = warp * 32;
            const float4 kv = *reinterpret_cast<const float4*>(kin_s + 4 * lane);
            const float4* Tbase = reinterpret_cast<const float4*>(P.c.T_K + (static_cast<long long>(head) * D + r0) * D) + lane;
            float part[32];
#pragma unroll
            for (int r = 0; r < 32; ++r) {
                const float4 t = __ldg(Tbase + r * (D / 4));
                part[r] = fmaf(t.x, kv.x, fmaf(t.y, kv.y, fmaf(t.z, kv.z, t.w * kv.w)));
            }
            kp_s[r0 + lane] = warp_transpose_reduce(part, lane);
        }
        __syncthreads();
        TokenSlot ts;
        ts.b = b; ts.slot = slot0; ts.pos = s0; ts.s_final = s0 + 1;
        if (ts.slot < 0 || ts.slot >= P.c.n_slots || s0 < 0) { if (threadIdx.x == 0 && head == 0) atomicOr(P.c.dev_status, WUSHKV_DEV_BAD_SLOT); ok = false; }
        if (ok) {
            const int pidx = ts.pos / PAGE_TOKENS;
            if (pidx >= P.c.max_pages) { if (threadIdx.x == 0 && head == 0) atomicOr(P.c.dev_status, WUSHKV_DEV_PAGE_TABLE_FULL); ok = false; }
            else if (page < 0 || page >= P.c.n_pages) { if (threadIdx.x == 0 && head == 0) atomicOr(P.c.dev_status, WUSHKV_DEV_BAD_PAGE_ID); ok = false; }
        }
        if (ok && warp < 2) {
            const int which = warp;                      // warp 0: key, warp 1: value
            ts.r = ts.pos % PAGE_TOKENS;
            ts.rec = P.c.pages + (static_cast<long long>(page) * n_kv + head) * record_bytes(BITS);
            float x[4];
            uint2 copy;
            if (which == 0) {
                const float4 kp = *reinterpret_cast<const float4*>(kp_s + 4 * lane);
                x[0] = kp.x; x[1] = kp.y; x[2] = kp.z; x[3] = kp.w;
                copy.x = float_to_bf16_bits(x[0]) | (static_cast<unsigned>(float_to_bf16_bits(x[1])) << 16);
                copy.y = float_to_bf16_bits(x[2]) | (static_cast<unsigned>(float_to_bf16_bits(x[3])) << 16);
            } else {
                copy = v_pre;
                x[0] = bf16_bits_to_float(copy.x & 0xffff); x[1] = bf16_bits_to_float(copy.x >> 16);
                x[2] = bf16_bits_to_float(copy.y & 0xffff); x[3] = bf16_bits_to_float(copy.y >> 16);
            }
            int code[4];
            __half step_h, xmin_h;
            quantize_vec<BITS>(x, which ? P.rule_v : P.rule_k, lane, code, step_h, xmin_h, which ? P.c.dev_status : nullptr);
            if (which == 0) store_k_codes<BITS>(ts.rec, ts.r, code, lane); else store_v_codes<BITS>(ts.rec, ts.r, code, lane);
            __half* meta = reinterpret_cast<__half*>(ts.rec + meta_location(BITS, ts.r));
            if (lane == 0) { meta[2 * which] = step_h; meta[2 * which + 1] = xmin_h; }
            store_window_copy(P, ts, head, which, copy, lane);
        }
    }
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    // the conditions that clear `ok` are the same for every head of the sequence, so the first CTA decides for all
    if (ok && head == 0 && threadIdx.x == 0) P.seq_len[b] = s0 + 1;
}

// ------------------------------------------------------------------------------------------------
// Chunk (prefill) append: the key transform K' = K T_K^T of 128 tokens x one KV head is ONE
// tcgen05 tile: A = the 128 x 128 bf16 key tile, B = T_K (bf16, [out][in] is already the K-major B
// operand), D = 128 x 128 fp32 in tensor memory (lane = token, column = output channel).  bf16 x bf16
// products are exact in fp32, so the result differs from the CUDA-core paths only by summation order.
// A CTA keeps its head's T_K resident in shared memory and walks over token tiles.  The key tile (straight
// into the operand layout) and the tile's value rows arrive by 16-byte cp.async copies; while the tensor
// core works on the keys, the warps quantize the values out of shared memory (they are parked in the part
// of the fp32 tile that stays free until the MMAs are done); the fp32 keys then come back through
// tcgen05.ld into shared memory and are quantized the same way: four lanes per vector, each keeping the
// largest 8 or 16 of its 32 entries with sorting networks on registers (quad_quantize).
//
// Shared-memory operand layout (no swizzle, K-major "interleaved"): the tile is cut into core matrices
// of 8 rows x 16 bytes (8 bf16) stored as 128 contiguous bytes; core matrix (row group rg, k chunk kc)
// sits at rg * SBO + kc * LBO with LBO = 128 B and SBO = 2048 B.  One MMA consumes K = 16, i.e. two
// k chunks, so the descriptor start address advances by 256 B per k-step.
// ------------------------------------------------------------------------------------------------
constexpr int TC_TILE = 128;                 // tokens per tile (MMA M)
constexpr int TC_LBO = 128, TC_SBO = 2048;   // bytes
constexpr int TC_X_PITCH = 136;              // floats per row of the fp32 key tile (== 8 mod 32: conflict-free quad reads)
constexpr int TC_THREADS = 512;
constexpr int TC_SMEM_B = 32768;                                   // T_K as bf16 operand
constexpr int TC_SMEM_X = TC_TILE * TC_X_PITCH * 4;                // fp32 keys; its first 32 KB double as the A operand
constexpr int TC_SMEM_A = TC_TILE * D * 2;                         // the A operand
constexpr int TC_V_PITCH = 288;                                    // bytes per staged value row (72 words: quad reads spread over all banks)
static_assert(TC_SMEM_A + TC_TILE * TC_V_PITCH <= TC_SMEM_X, "the staged value rows must fit behind the A operand");
constexpr int TC_SMEM_ROWS = TC_TILE * 32;                          // per-row token lookup (RowInfo)
constexpr int TC_SMEM_TOTAL = TC_SMEM_B + TC_SMEM_X + TC_SMEM_ROWS + 64;

__device__ __forceinline__ unsigned long long umma_smem_desc(unsigned smem_addr) {
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((smem_addr >> 4) & 0x3FFFu);            // start address
    d |= static_cast<unsigned long long>((TC_LBO >> 4) & 0x3FFFu) << 16;         // leading (k chunk) byte offset
    d |= static_cast<unsigned long long>((TC_SBO >> 4) & 0x3FFFu) << 32;         // stride (row group) byte offset
    d |= 1ull << 46;                                                             // descriptor version of sm_100
    return d;                                                                    // base offset 0, no swizzle
}
// The same for an operand written by a bulk tensor copy: rows of 128 bytes with the 128-byte swizzle, groups of 8 rows
// 1024 bytes apart; a k-step of 16 channels advances the start address by 32 bytes inside the row.
__device__ __forceinline__ unsigned long long umma_smem_desc_sw128(unsigned smem_addr) {
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((smem_addr >> 4) & 0x3FFFu);
    d |= 1ull << 16;
    d |= static_cast<unsigned long long>(1024u >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
__device__ __forceinline__ void tma_tile_3d(unsigned dst, const CUtensorMap* map, int c0, int c1, int c2, unsigned bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = 128
constexpr unsigned UMMA_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ unsigned smem_addr_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros without reading
__device__ __forceinline__ void cp_async16(unsigned dst, const void* src, unsigned src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// ---- quad-per-vector quantizer of the chunk path --------------------------------------------------
// Four adjacent lanes own one 128-vector, 32 entries each.  The clipping quantile needs the two
// order statistics around rank kappa*(d-1) of |x|, i.e. the `rounds`-th and (`rounds`-1)-th largest;
// each lane keeps the KK largest of its entries with bitonic networks on registers and the quad merges
// the four lists with two exchanges.  All network indices are compile-time constants.
struct RowInfo {                 // where one token of the tile goes (filled once per tile and head)
    long long rec_off;           // byte offset of the head's record in the page pool, < 0: skip the token
    int r, pos, s_final, slot;
    int pad[2];
};

__device__ __forceinline__ void ce_desc_u(unsigned& a, unsigned& b) {
    const unsigned hi = max(a, b), lo = min(a, b);
    a = hi; b = lo;
}
// Sorting networks with the fewest known comparators (19 for 8 keys: Batcher's odd-even merge sort;
// 60 for 16 keys: Green's network), descending; both checked exhaustively with the 0-1 principle.
__device__ __forceinline__ void sort_desc(unsigned (&a)[8]) {
    ce_desc_u(a[0], a[1]); ce_desc_u(a[2], a[3]); ce_desc_u(a[0], a[2]); ce_desc_u(a[1], a[3]); ce_desc_u(a[1], a[2]); ce_desc_u(a[4], a[5]); ce_desc_u(a[6], a[7]); ce_desc_u(a[4], a[6]);
    ce_desc_u(a[5], a[7]); ce_desc_u(a[5], a[6]); ce_desc_u(a[0], a[4]); ce_desc_u(a[2], a[6]); ce_desc_u(a[2], a[4]); ce_desc_u(a[1], a[5]); ce_desc_u(a[3], a[7]); ce_desc_u(a[3], a[5]);
    ce_desc_u(a[1], a[2]); ce_desc_u(a[3], a[4]); ce_desc_u(a[5], a[6]);
}
__device__ __forceinline__ void sort_desc(unsigned (&a)[16]) {
    ce_desc_u(a[0], a[13]); ce_desc_u(a[1], a[12]); ce_desc_u(a[2], a[15]); ce_desc_u(a[3], a[14]); ce_desc_u(a[4], a[8]); ce_desc_u(a[5], a[6]); ce_desc_u(a[7], a[11]); ce_desc_u(a[9], a[10]);
    ce_desc_u(a[0], a[5]); ce_desc_u(a[1], a[7]); ce_desc_u(a[2], a[9]); ce_desc_u(a[3], a[4]); ce_desc_u(a[6], a[13]); ce_desc_u(a[8], a[14]); ce_desc_u(a[10], a[15]); ce_desc_u(a[11], a[12]);
    ce_desc_u(a[0], a[1]); ce_desc_u(a[2], a[3]); ce_desc_u(a[4], a[5]); ce_desc_u(a[6], a[8]); ce_desc_u(a[7], a[9]); ce_desc_u(a[10], a[11]); ce_desc_u(a[12], a[13]); ce_desc_u(a[14], a[15]);
    ce_desc_u(a[0], a[2]); ce_desc_u(a[1], a[3]); ce_desc_u(a[4], a[10]); ce_desc_u(a[5], a[11]); ce_desc_u(a[6], a[7]); ce_desc_u(a[8], a[9]); ce_desc_u(a[12], a[14]); ce_desc_u(a[13], a[15]);
    ce_desc_u(a[1], a[2]); ce_desc_u(a[3], a[12]); ce_desc_u(a[4], a[6]); ce_desc_u(a[5], a[7]); ce_desc_u(a[8], a[10]); ce_desc_u(a[9], a[11]); ce_desc_u(a[13], a[14]);
    ce_desc_u(a[1], a[4]); ce_desc_u(a[2], a[6]); ce_desc_u(a[5], a[8]); ce_desc_u(a[7], a[10]); ce_desc_u(a[9], a[13]); ce_desc_u(a[11], a[14]);
    ce_desc_u(a[2], a[4]); ce_desc_u(a[3], a[6]); ce_desc_u(a[9], a[12]); ce_desc_u(a[11], a[13]);
    ce_desc_u(a[3], a[5]); ce_desc_u(a[6], a[8]); ce_desc_u(a[7], a[9]); ce_desc_u(a[10], a[12]);
    ce_desc_u(a[3], a[4]); ce_desc_u(a[5], a[6]); ce_desc_u(a[7], a[8]); ce_desc_u(a[9], a[10]); ce_desc_u(a[11], a[12]);
    ce_desc_u(a[6], a[7]); ce_desc_u(a[8], a[9]);
}
template <int N>
__device__ __forceinline__ void bitonic_merge_desc(unsigned (&a)[N]) {      // bitonic sequence -> descending
#pragma unroll
    for (int j = N >> 1; j > 0; j >>= 1)
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const int l = i ^ j;
            if (l > i) ce_desc_u(a[i], a[l]);
        }
}
template <int N>
__device__ __forceinline__ void keep_largest(unsigned (&top)[N], const unsigned (&other)[N]) {   // both descending
#pragma unroll
    for (int i = 0; i < N; ++i) top[i] = max(top[i], other[N - 1 - i]);
    bitonic_merge_desc<N>(top);
}

// Clip range, stored step / offset and the 32 codes of this lane's entries x[32] (Eq. 6); all four
// lanes of the quad return the same step_h / xmin_h.
template <int BITS, int KK>
__device__ __forceinline__ void quad_quantize(const float (&x)[32], ClipRule rule, int (&code)[32], __half& step_h, __half& xmin_h,
                                              int* value_status = nullptr, bool flag_lane = false) {
    constexpr int LEVELS = (1 << BITS) - 1;
    if constexpr (KK < 0) {                     // Eq. 5 (see quantize_vec); a compile-time choice keeps it out of the Eq. 6 kernels
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) ss = fmaf(x[i], x[i], ss);
        ss += __shfl_xor_sync(FULL, ss, 1);
        ss += __shfl_xor_sync(FULL, ss, 2);
        step_h = __float2half_rn(fminf(rule.quest * sqrtf(ss), 65504.f));
        const float step_s = __half2float(step_h);
        xmin_h = __float2half_rn(step_s > 0.f ? -0.5f * static_cast<float>(LEVELS) * step_s : 0.f);
        if (value_status != nullptr && flag_lane && step_s >= VALUE_STEP_LIMIT) atomicOr(value_status, WUSHKV_DEV_VALUE_RANGE);
        const float inv = step_s > 0.f ? __frcp_rn(step_s) : 0.f;
        constexpr float HALF = static_cast<float>(1 << (BITS - 1));
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float t = fminf(fmaxf(floorf(x[i] * inv) + HALF, 0.f), static_cast<float>(LEVELS));
            code[i] = step_s > 0.f ? static_cast<int>(t) : 0;
        }
    } else {
    unsigned top[KK];
#pragma unroll
    for (int g0 = 0; g0 < 32; g0 += KK) {
        unsigned tmp[KK];
#pragma unroll
        for (int i = 0; i < KK; ++i) tmp[i] = __float_as_uint(x[g0 + i]) & 0x7fffffffu;
        sort_desc(tmp);
        if (g0 == 0) {
#pragma unroll
            for (int i = 0; i < KK; ++i) top[i] = tmp[i];
        } else {
            keep_largest<KK>(top, tmp);
        }
    }
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
        unsigned other[KK];
#pragma unroll
        for (int i = 0; i < KK; ++i) other[i] = __shfl_xor_sync(FULL, top[i], off);
        keep_largest<KK>(top, other);
    }
    unsigned a_lo = 0, a_hi = 0;
#pragma unroll
    for (int i = 0; i < KK; ++i) {
        if (i == rule.rounds - 1) a_lo = top[i];
        if (i == rule.rounds - 2) a_hi = top[i];
    }
    if (rule.rounds == 1) a_hi = a_lo;
    const float alo = __uint_as_float(a_lo), ahi = __uint_as_float(a_hi);
    const float q = alo + rule.frac * (ahi - alo);
    float lmin = x[0], lmax = x[0];
#pragma unroll
    for (int i = 1; i < 32; ++i) { lmin = fminf(lmin, x[i]); lmax = fmaxf(lmax, x[i]); }
    lmin = fminf(lmin, __shfl_xor_sync(FULL, lmin, 1)); lmax = fmaxf(lmax, __shfl_xor_sync(FULL, lmax, 1));
    lmin = fminf(lmin, __shfl_xor_sync(FULL, lmin, 2)); lmax = fmaxf(lmax, __shfl_xor_sync(FULL, lmax, 2));
    const float x_min = fmaxf(lmin, -q);
    const float x_max = fminf(lmax, q);
    const float step = __fdiv_rn(x_max - x_min, static_cast<float>(LEVELS));
    step_h = __float2half_rn(fminf(fmaxf(step, -65504.f), 65504.f));
    xmin_h = __float2half_rn(fminf(fmaxf(x_min, -65504.f), 65504.f));
    const float step_s = __half2float(step_h), xmin_s = __half2float(xmin_h);
    if (value_status != nullptr && flag_lane && step_s >= VALUE_STEP_LIMIT) atomicOr(value_status, WUSHKV_DEV_VALUE_RANGE);
    const float inv = step_s > 0.f ? __frcp_rn(step_s) : 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        // clamp, then round to nearest even by adding 1.5 * 2^23: the code is in the low mantissa bits
        const float t = fminf(fmaxf((x[i] - xmin_s) * inv, 0.f), static_cast<float>(LEVELS));
        code[i] = static_cast<int>(__float_as_uint(t + 12582912.f) & 0xFu);
    }
    }
}

// KK_K / KK_V: list length of the quad quantizer for keys / values (8 or 16, >= the rule's rounds), 0 for
// the warp-per-vector quantizer (any kappa), or -1 for the QuEST rule (Eq. 5, no order statistics).
template <int BITS, int KK_K, int KK_V>
__global__ void __launch_bounds__(TC_THREADS, 2) append_chunk_kernel(AppendParams P, const __grid_constant__ CUtensorMap map_k,
                                                                     const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ __align__(1024) unsigned char tc_smem[];
    unsigned char* sB = tc_smem;
    unsigned char* sA = tc_smem + TC_SMEM_B;                         // A operand, later overwritten by the fp32 tile
    float* sX = reinterpret_cast<float*>(tc_smem + TC_SMEM_B);
    unsigned char* sV = tc_smem + TC_SMEM_B + TC_SMEM_A;             // value rows of the tile, until the fp32 tile arrives
    unsigned long long* mbar = reinterpret_cast<unsigned long long*>(tc_smem + TC_SMEM_B + TC_SMEM_X);
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(tc_smem + TC_SMEM_B + TC_SMEM_X + 16);
    RowInfo* rows = reinterpret_cast<RowInfo*>(tc_smem + TC_SMEM_B + TC_SMEM_X + 64);
    const int head = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_tiles = (P.total_new + TC_TILE - 1) / TC_TILE;

    // ---- one-time set-up: tensor memory, barrier, T_K as bf16 operand
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr_u32(tmem_slot)), "r"(128u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const unsigned tbar = smem_addr_u32(mbar) + 8;           // completion of a tile's bulk tensor copies
    unsigned tphase = 0;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr_u32(mbar)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    {
        const float* T = P.c.T_K + static_cast<long long>(head) * D * D;
        const int r8 = lane & 7, cq = lane >> 3;
        for (int item = warp; item < 64; item += TC_THREADS / 32) {     // 16 row groups x 4 groups of 4 k chunks
            const int rg = item >> 2, kc = (item & 3) * 4 + cq;
            const float4* src = reinterpret_cast<const float4*>(T + (rg * 8 + r8) * D + kc * 8);
            const float4 a = __ldg(src), b = __ldg(src + 1);
            uint4 v;
            v.x = float_to_bf16_bits(a.x) | (static_cast<unsigned>(float_to_bf16_bits(a.y)) << 16);
            v.y = float_to_bf16_bits(a.z) | (static_cast<unsigned>(float_to_bf16_bits(a.w)) << 16);
            v.z = float_to_bf16_bits(b.x) | (static_cast<unsigned>(float_to_bf16_bits(b.y)) << 16);
            v.w = float_to_bf16_bits(b.z) | (static_cast<unsigned>(float_to_bf16_bits(b.w)) << 16);
            *reinterpret_cast<uint4*>(sB + rg * TC_SBO + kc * TC_LBO + r8 * 16) = v;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;
    unsigned phase = 0;
    bool failed = false;

    for (int tile = blockIdx.x; tile < n_tiles && !failed; tile += gridDim.x) {
        const int tok0 = tile * TC_TILE;
        // ---- A operand: key rows of this tile (zero rows past the end of the batch), and the value rows of the
        // tile into the part of the fp32 tile that is free until the MMAs are done; both as 16-byte
        // asynchronous copies, so that no register waits for them
        if (P.use_tma) {
            // four bulk tensor copies: keys and values x channel halves, 128 rows of 128 bytes each (rows past the end of
            // the batch read zeros); the values go to the part of the fp32 tile that is free until the MMAs are done
            if (tid == 0) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tbar), "r"(KK_V != 0 ? 4u * 16384u : 2u * 16384u) : "memory");
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    tma_tile_3d(smem_addr_u32(sA) + hf * 16384, &map_k, 64 * hf, head, tok0, tbar);
                    if (KK_V != 0) tma_tile_3d(smem_addr_u32(sV) + hf * 16384, &map_v, 64 * hf, head, tok0, tbar);
                }
            }
        } else {
            const int r8 = lane & 7, cq = lane >> 3;
            for (int item = warp; item < 64; item += TC_THREADS / 32) {
                const int rg = item >> 2, kc = (item & 3) * 4 + cq;
                const int tok = tok0 + rg * 8 + r8;
                const bool in_range = tok < P.total_new;
                cp_async16(smem_addr_u32(sA + rg * TC_SBO + kc * TC_LBO + r8 * 16),
                           P.K_new + (static_cast<long long>(in_range ? tok : 0) * P.c.n_kv + head) * D + kc * 8, in_range ? 16u : 0u);
            }
            if (KK_V != 0) {
                for (int item = tid; item < TC_TILE * 16; item += TC_THREADS) {
                    const int row = item >> 4, ch = item & 15;
                    const bool in_range = tok0 + row < P.total_new;
                    cp_async16(smem_addr_u32(sV + row * TC_V_PITCH + ch * 16),
                               P.V_new + (static_cast<long long>(in_range ? tok0 + row : 0) * P.c.n_kv + head) * D + ch * 8, in_range ? 16u : 0u);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (tid < TC_TILE) {                                  // where each token of the tile goes
            RowInfo ri;
            ri.rec_off = -1; ri.r = 0; ri.pos = 0; ri.s_final = 0; ri.slot = 0; ri.pad[0] = ri.pad[1] = 0;
            TokenSlot ts;
            if (tok0 + tid < P.total_new && locate_token(P, tok0 + tid, head, ts)) {
                ri.rec_off = ts.rec - P.c.pages; ri.r = ts.r; ri.pos = ts.pos; ri.s_final = ts.s_final; ri.slot = ts.slot;
            }
            rows[tid] = ri;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        if (P.use_tma) {                                      // bounded wait for the tile's bulk copies
            bool arrived = false;
            const int tma_wait_limit = P.wait_limit > 0 ? P.wait_limit : (1 << 22);
            for (int it = 0; it < tma_wait_limit && !arrived; ++it) {
                unsigned ok;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(tbar), "r"(tphase), "r"(200u) : "memory");
                arrived = ok != 0;
            }
            tphase ^= 1u;
            if (!__syncthreads_and(arrived ? 1 : 0)) {
                if (tid == 0) atomicOr(P.c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
                failed = true;
                break;
            }
        }
        if (P.pro.rope) {
            // Projected keys: normalise and rotate the staged tile in place (Algorithm 2 lines 1-2).  Four threads
            // share a row; thread q of a row owns channels 16q..16q+15 and their rotation partners 64+16q..64+16q+15,
            // i.e. k chunks 2q, 2q+1, 8+2q, 9+2q of the operand layout.
            __syncthreads();                                  // the copies and the row records of the other threads
            const int row = tid >> 2, q = tid & 3;
            const RowInfo ri = rows[row];
            unsigned char* base = sA + (row >> 3) * TC_SBO + (row & 7) * 16;
            uint4 raw[4];
            raw[0] = *reinterpret_cast<const uint4*>(base + (2 * q) * TC_LBO);
            raw[1] = *reinterpret_cast<const uint4*>(base + (2 * q + 1) * TC_LBO);
            raw[2] = *reinterpret_cast<const uint4*>(base + (8 + 2 * q) * TC_LBO);
            raw[3] = *reinterpret_cast<const uint4*>(base + (9 + 2 * q) * TC_LBO);
            float a[16], b[16];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const unsigned wa[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w}, wb[4] = {raw[2 + k].x, raw[2 + k].y, raw[2 + k].z, raw[2 + k].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    a[8 * k + 2 * e] = bf16_bits_to_float(wa[e] & 0xffff); a[8 * k + 2 * e + 1] = bf16_bits_to_float(wa[e] >> 16);
                    b[8 * k + 2 * e] = bf16_bits_to_float(wb[e] & 0xffff); b[8 * k + 2 * e + 1] = bf16_bits_to_float(wb[e] >> 16);
                }
            }
            if (P.pro.normalise) {
                float ss = 0.f;
#pragma unroll
                for (int e = 0; e < 16; ++e) ss = fmaf(a[e], a[e], fmaf(b[e], b[e], ss));
                ss += __shfl_xor_sync(FULL, ss, 1);
                ss += __shfl_xor_sync(FULL, ss, 2);
                const float r = ss > 0.f ? 1.f / sqrtf(ss * (1.f / D) + P.pro.eps) : 0.f;
                if (P.pro.weight) {
                    const float4* wa = reinterpret_cast<const float4*>(P.pro.weight + static_cast<long long>(head) * D + 16 * q);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float4 u = __ldg(wa + e), v = __ldg(wa + 16 + e);
                        a[4 * e] *= r * u.x; a[4 * e + 1] *= r * u.y; a[4 * e + 2] *= r * u.z; a[4 * e + 3] *= r * u.w;
                        b[4 * e] *= r * v.x; b[4 * e + 1] *= r * v.y; b[4 * e + 2] *= r * v.z; b[4 * e + 3] *= r * v.w;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) { a[e] *= r; b[e] *= r; }
                }
            }
            const int pos = prologue_position(P.pro, ri.pos, P.c.dev_status, ri.rec_off >= 0 && q == 0);
            const float4* tab = reinterpret_cast<const float4*>(P.pro.rope + static_cast<long long>(pos) * (D / 2) + 16 * q);
            unsigned outa[8], outb[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float4 cs = __ldg(tab + e);             // (cos, sin) of pairs 16q + 2e, 16q + 2e + 1
                const float ya0 = fmaf(a[2 * e], cs.x, -b[2 * e] * cs.y), yb0 = fmaf(a[2 * e], cs.y, b[2 * e] * cs.x);
                const float ya1 = fmaf(a[2 * e + 1], cs.z, -b[2 * e + 1] * cs.w), yb1 = fmaf(a[2 * e + 1], cs.w, b[2 * e + 1] * cs.z);
                outa[e] = float_to_bf16_bits(ya0) | (static_cast<unsigned>(float_to_bf16_bits(ya1)) << 16);
                outb[e] = float_to_bf16_bits(yb0) | (static_cast<unsigned>(float_to_bf16_bits(yb1)) << 16);
            }
            *reinterpret_cast<uint4*>(base + (2 * q) * TC_LBO) = make_uint4(outa[0], outa[1], outa[2], outa[3]);
            *reinterpret_cast<uint4*>(base + (2 * q + 1) * TC_LBO) = make_uint4(outa[4], outa[5], outa[6], outa[7]);
            *reinterpret_cast<uint4*>(base + (8 + 2 * q) * TC_LBO) = make_uint4(outb[0], outb[1], outb[2], outb[3]);
            *reinterpret_cast<uint4*>(base + (9 + 2 * q) * TC_LBO) = make_uint4(outb[4], outb[5], outb[6], outb[7]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // generic-proxy writes -> visible to the tensor core
        __syncthreads();
        // ---- one thread issues the 8 k-steps and commits them to the barrier
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const unsigned long long adesc = umma_smem_desc(smem_addr_u32(sA)), bdesc = umma_smem_desc(smem_addr_u32(sB));
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const unsigned accumulate = ks > 0 ? 1u : 0u;
                // swizzled A: channels 0-63 and 64-127 are two boxes of 16 KB, a k-step is 32 bytes inside the 128-byte row
                const unsigned long long a_ks = P.use_tma ? umma_smem_desc_sw128(smem_addr_u32(sA) + (ks >> 2) * 16384 + (ks & 3) * 32)
                                                          : adesc + static_cast<unsigned long long>(ks * 2 * TC_LBO >> 4);
                asm volatile(
                    "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                    "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                    ::"r"(tmem_base), "l"(a_ks),
                      "l"(bdesc + static_cast<unsigned long long>(ks * 2 * TC_LBO >> 4)), "r"(UMMA_IDESC), "r"(accumulate),
                      "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
            }
            if (!(P.drop_mma_commit && tile == 0))       // (testing aid: without the commit the wait below runs into its limit)
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr_u32(mbar)) : "memory");
        }
        // ---- while the tensor core runs: values of this tile (no transform)
        if (KK_V != 0) {
            constexpr int KQ = KK_V != 0 ? KK_V : 8;
            const int row = 8 * warp + (lane >> 2), qd = lane & 3;
            const RowInfo ri = rows[row];
            const bool live = ri.rec_off >= 0;
            const unsigned char* vrow = sV + row * TC_V_PITCH + 8 * qd;
            float x[32];
            uint2 raw[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                // channels 16k + 4qd .. +3: byte 32k + 8qd of the row; in a swizzled tile the row is 2 x 128 bytes (two
                // boxes) and its 16-byte pieces are XOR-ed with the row index
                const int o = 32 * k + 8 * qd;
                const unsigned char* src = P.use_tma ? sV + (o >> 7) * 16384 + row * 128 + ((((o & 127) >> 4) ^ (row & 7)) << 4) + (o & 15)
                                                     : vrow + 32 * k;
                raw[k] = live ? *reinterpret_cast<const uint2*>(src) : make_uint2(0u, 0u);
                x[4 * k + 0] = bf16_bits_to_float(raw[k].x & 0xffff); x[4 * k + 1] = bf16_bits_to_float(raw[k].x >> 16);
                x[4 * k + 2] = bf16_bits_to_float(raw[k].y & 0xffff); x[4 * k + 3] = bf16_bits_to_float(raw[k].y >> 16);
            }
            int code[32];
            __half step_h, xmin_h;
            quad_quantize<BITS, KQ>(x, P.rule_v, code, step_h, xmin_h, P.c.dev_status, live && qd == 0);
            unsigned hplane[4] = {0u, 0u, 0u, 0u};           // 3 bits: the 1-bit plane's half-words, both row halves joined
            if (BITS == 3) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    unsigned h0 = 0, h1 = 0;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        h0 |= static_cast<unsigned>(code[4 * k + e] >> 2) << v1_bit(0, k);
                        h1 |= static_cast<unsigned>(code[4 * k + e] >> 2) << v1_bit(1, k);
                    }
                    const unsigned mine = (qd >> 1) ? h1 : h0;
                    hplane[e] = mine | __shfl_xor_sync(FULL, mine, 2);     // lane qd ^ 2 holds the other row half of the same rows
                }
            }
            if (live) {
                unsigned char* rec = P.c.pages + ri.rec_off;
                const int bi = ri.r >> 4, rr = ri.r & 15, ps = rr >> 3, t = (rr & 7) >> 1, hi = rr & 1;
#pragma unroll
                for (int e = 0; e < 4; ++e) {                 // channel residue c16 = 4 qd + e: one half-word per 8 (or 4) channel blocks
                    const int c16 = 4 * qd + e, g = c16 & 7, rsel = c16 >> 3;
                    if (BITS == 2 || BITS == 3) {
                        unsigned hw = 0;
#pragma unroll
                        for (int k = 0; k < 8; ++k) hw |= static_cast<unsigned>(code[4 * k + e] & 3) << (2 * k);
                        *reinterpret_cast<unsigned short*>(rec + v_codes_offset(BITS) + bi * 512 + 16 * (4 * g + t) + 4 * (2 * ps + rsel) + 2 * hi) =
                            static_cast<unsigned short>(hw);
                        if (BITS == 3 && qd < 2)
                            *reinterpret_cast<unsigned short*>(rec + v_hi_offset(3) + bi * 256 + 8 * (4 * g + t) + 4 * ps + 2 * hi) =
                                static_cast<unsigned short>(hplane[e]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            unsigned hw = 0;
#pragma unroll
                            for (int k = 0; k < 4; ++k) hw |= static_cast<unsigned>(code[4 * (4 * j + k) + e]) << (4 * k);
                            *reinterpret_cast<unsigned short*>(rec + v_codes_offset(4) + bi * 1024 + 512 * ps + 16 * (4 * g + t) + 4 * (2 * rsel + j) + 2 * hi) =
                                static_cast<unsigned short>(hw);
                        }
                    }
                }
                if (qd == 0) {
                    __half* meta = reinterpret_cast<__half*>(rec + meta_location(BITS, ri.r));
                    meta[2] = step_h; meta[3] = xmin_h;
                }
                const CacheView& c = P.c;
                const long long plane = (static_cast<long long>(ri.slot) * c.n_kv + head) * 2 + 1;
                if (ri.pos < c.s_sink) {
                    unsigned short* dst = c.sink_kv + (plane * c.s_sink + ri.pos) * D + 4 * qd;
#pragma unroll
                    for (int k = 0; k < 8; ++k) *reinterpret_cast<uint2*>(dst + 16 * k) = raw[k];
                }
                if (ri.pos >= ri.s_final - c.ring_cap) {
                    unsigned short* dst = c.ring_kv + (plane * c.ring_cap + ri.pos % c.ring_cap) * D + 4 * qd;
#pragma unroll
                    for (int k = 0; k < 8; ++k) *reinterpret_cast<uint2*>(dst + 16 * k) = raw[k];
                }
            }
        } else {
            for (int v = warp; v < TC_TILE; v += TC_THREADS / 32) {
                const int token = tok0 + v;
                if (token >= P.total_new) break;
                TokenSlot ts;
                if (!locate_token(P, token, head, ts)) continue;
                const uint2 vraw = __ldg(reinterpret_cast<const uint2*>(P.V_new + (static_cast<long long>(token) * P.c.n_kv + head) * D) + lane);
                float x[4] = {bf16_bits_to_float(vraw.x & 0xffff), bf16_bits_to_float(vraw.x >> 16),
                              bf16_bits_to_float(vraw.y & 0xffff), bf16_bits_to_float(vraw.y >> 16)};
                int code[4];
                __half step_h, xmin_h;
                quantize_vec<BITS>(x, P.rule_v, lane, code, step_h, xmin_h, P.c.dev_status);
                store_v_codes<BITS>(ts.rec, ts.r, code, lane);
                __half* meta = reinterpret_cast<__half*>(ts.rec + meta_location(BITS, ts.r));
                if (lane == 0) { meta[2] = step_h; meta[3] = xmin_h; }
                store_window_copy(P, ts, head, 1, vraw, lane);
            }
        }
        // ---- wait for the MMAs (bounded), then tensor memory -> shared memory
        {
            bool done = false;
            const int mma_wait_limit = P.wait_limit > 0 ? P.wait_limit : (1 << 20);
            for (int it = 0; it < mma_wait_limit && !done; ++it) {
                unsigned ok;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(smem_addr_u32(mbar)), "r"(phase), "r"(2000u) : "memory");
                done = ok != 0;
            }
            if (!__syncthreads_and(done ? 1 : 0)) {          // uniform decision for the whole CTA
                if (tid == 0) {
                    atomicOr(P.c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
                    // commit whatever was issued once more and give it a bounded time, so that no MMA is still
                    // writing tensor memory when it is released below
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr_u32(mbar)) : "memory");
                }
                for (int it = 0; it < 512; ++it) {
                    unsigned ok;
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                                 : "=r"(ok) : "r"(smem_addr_u32(mbar)), "r"(phase), "r"(2000u) : "memory");
                    if (ok) break;
                }
                failed = true;
                break;
            }
            phase ^= 1u;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        {
            const int q = warp & 3, cg = warp >> 2;          // lane quadrant of this warp, 32-column group
            unsigned r[32];
            const unsigned taddr = tmem_base + (static_cast<unsigned>(q * 32) << 16) + static_cast<unsigned>(cg * 32);
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                  "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                  "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                  "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            float* dst = sX + (q * 32 + lane) * TC_X_PITCH + cg * 32;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(dst + 4 * j) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        // ---- keys of this tile: quantize the fp32 rows
        if (KK_K != 0) {
            constexpr int KQ = KK_K != 0 ? KK_K : 8;
            const int row = 8 * warp + (lane >> 2), qd = lane & 3;
            const RowInfo ri = rows[row];
            const bool live = ri.rec_off >= 0;
            float x[32];                                      // entry 4k + j: channel 16k + 2qd + (j & 1) + 8 (j >> 1)
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float2 a = *reinterpret_cast<const float2*>(sX + row * TC_X_PITCH + 16 * k + 2 * qd);
                const float2 b = *reinterpret_cast<const float2*>(sX + row * TC_X_PITCH + 16 * k + 2 * qd + 8);
                x[4 * k + 0] = a.x; x[4 * k + 1] = a.y; x[4 * k + 2] = b.x; x[4 * k + 3] = b.y;
            }
            int code[32];
            __half step_h, xmin_h;
            quad_quantize<BITS, KQ>(x, P.rule_k, code, step_h, xmin_h);
            if (live) {
                unsigned char* rec = P.c.pages + ri.rec_off;
                const int bi = ri.r >> 4, rr = ri.r & 15, g = rr & 7, rs = rr >> 3;
                // entry 4k + j is byte j of the word of channel half k & 1, field / nibble of k-step k >> 1
                if (BITS == 2 || BITS == 3) {
                    unsigned w[2] = {0u, 0u};
#pragma unroll
                    for (int k = 0; k < 8; ++k)
#pragma unroll
                        for (int j = 0; j < 4; ++j) w[k & 1] |= static_cast<unsigned>(code[4 * k + j] & 3) << (8 * j + 2 * (k >> 1));
                    unsigned char* p = rec + bi * 512 + 16 * (4 * g + qd) + 4 * rs;
                    *reinterpret_cast<unsigned*>(p) = w[0];
                    *reinterpret_cast<unsigned*>(p + 8) = w[1];
                    if (BITS == 3) {                          // 1-bit plane: byte j, bit 2 (k >> 1) + (k & 1) = k
                        unsigned wh = 0u;
#pragma unroll
                        for (int k = 0; k < 8; ++k)
#pragma unroll
                            for (int j = 0; j < 4; ++j) wh |= static_cast<unsigned>(code[4 * k + j] >> 2) << (8 * j + k);
                        *reinterpret_cast<unsigned*>(rec + k_hi_offset(3) + bi * 256 + 8 * (4 * g + qd) + 4 * rs) = wh;
                    }
                } else {
                    unsigned w[2][2] = {{0u, 0u}, {0u, 0u}};      // [512-byte half][channel half]
#pragma unroll
                    for (int k = 0; k < 8; ++k)
#pragma unroll
                        for (int j = 0; j < 4; ++j) w[k >> 2][k & 1] |= static_cast<unsigned>(code[4 * k + j]) << (8 * j + 4 * ((k >> 1) & 1));
#pragma unroll
                    for (int pq = 0; pq < 2; ++pq) {
                        unsigned char* p = rec + bi * 1024 + 512 * pq + 16 * (4 * g + qd) + 4 * rs;
                        *reinterpret_cast<unsigned*>(p) = w[pq][0];
                        *reinterpret_cast<unsigned*>(p + 8) = w[pq][1];
                    }
                }
                if (qd == 0) {
                    __half* meta = reinterpret_cast<__half*>(rec + meta_location(BITS, ri.r));
                    meta[0] = step_h; meta[1] = xmin_h;
                }
                const CacheView& c = P.c;
                const long long plane = (static_cast<long long>(ri.slot) * c.n_kv + head) * 2 + 0;
                const bool to_sink = ri.pos < c.s_sink, to_ring = ri.pos >= ri.s_final - c.ring_cap;
                if (to_sink || to_ring) {
                    unsigned short* d_sink = c.sink_kv + (plane * c.s_sink + ri.pos) * D + 2 * qd;
                    unsigned short* d_ring = c.ring_kv + (plane * c.ring_cap + ri.pos % c.ring_cap) * D + 2 * qd;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const unsigned lo = float_to_bf16_bits(x[4 * k + 0]) | (static_cast<unsigned>(float_to_bf16_bits(x[4 * k + 1])) << 16);
                        const unsigned hi2 = float_to_bf16_bits(x[4 * k + 2]) | (static_cast<unsigned>(float_to_bf16_bits(x[4 * k + 3])) << 16);
                        if (to_sink) { *reinterpret_cast<unsigned*>(d_sink + 16 * k) = lo; *reinterpret_cast<unsigned*>(d_sink + 16 * k + 8) = hi2; }
                        if (to_ring) { *reinterpret_cast<unsigned*>(d_ring + 16 * k) = lo; *reinterpret_cast<unsigned*>(d_ring + 16 * k + 8) = hi2; }
                    }
                }
            }
        } else {
            for (int v = warp; v < TC_TILE; v += TC_THREADS / 32) {
                const int token = tok0 + v;
                if (token >= P.total_new) break;
                TokenSlot ts;
                if (!locate_token(P, token, head, ts)) continue;
                const float4 kp = *reinterpret_cast<const float4*>(sX + v * TC_X_PITCH + 4 * lane);
                float x[4] = {kp.x, kp.y, kp.z, kp.w};
                int code[4];
                __half step_h, xmin_h;
                quantize_vec<BITS>(x, P.rule_k, lane, code, step_h, xmin_h);
                store_k_codes<BITS>(ts.rec, ts.r, code, lane);
                __half* meta = reinterpret_cast<__half*>(ts.rec + meta_location(BITS, ts.r));
                if (lane == 0) { meta[0] = step_h; meta[1] = xmin_h; }
                uint2 kb;
                kb.x = float_to_bf16_bits(x[0]) | (static_cast<unsigned>(float_to_bf16_bits(x[1])) << 16);
                kb.y = float_to_bf16_bits(x[2]) | (static_cast<unsigned>(float_to_bf16_bits(x[3])) << 16);
                store_window_copy(P, ts, head, 0, kb, lane);
            }
        }
        __syncthreads();                                      // the fp32 tile becomes the next A operand
    }
    // ---- release tensor memory (also after a timeout: nothing of this CTA is in flight any more or ever will complete)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
}

// Advances the lengths after a rows / chunk append.  A sequence one of whose tokens could not be stored
// (bad slot, page table too short, page id outside the pool: the append kernel flagged it and skipped
// that token) keeps its old length.
__global__ void advance_len_kernel(CacheView c, int batch, const int* slot, int* seq_len, const int* cu_new) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int n_new = cu_new[b + 1] - cu_new[b];
    if (n_new <= 0) return;
    const int s0 = seq_len[b], sl = slot[b];
    if (sl < 0 || sl >= c.n_slots || s0 < 0) return;
    const int p0 = s0 / PAGE_TOKENS, p1 = (s0 + n_new - 1) / PAGE_TOKENS;
    if (p1 >= c.max_pages) return;
    for (int p = p0; p <= p1; ++p) {
        const int page = c.page_table[static_cast<long long>(sl) * c.max_pages + p];
        if (page < 0 || page >= c.n_pages) return;
    }
    seq_len[b] = s0 + n_new;
}

__global__ void unpack_debug_kernel(CacheView c, int slot, int head, int which, int pos0, int n,
                                    unsigned char* codes, float* scale, float* zero) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n * D) return;
    const int tok = idx >> 7, ch = idx & 127;
    const int pos = pos0 + tok;
    const int pidx = pos / PAGE_TOKENS, r = pos % PAGE_TOKENS;
    if (pidx >= c.max_pages) { atomicOr(c.dev_status, WUSHKV_DEV_PAGE_TABLE_FULL); return; }
    const int page = c.page_table[static_cast<long long>(slot) * c.max_pages + pidx];
    if (page < 0 || page >= c.n_pages) { atomicOr(c.dev_status, WUSHKV_DEV_BAD_PAGE_ID); return; }
    const unsigned char* rec = c.pages + (static_cast<long long>(page) * c.n_kv + head) * record_bytes(c.bits);
    int off, bit;
    if (which == 0) k_code_location(c.bits, r, ch, off, bit); else v_code_location(c.bits, r, ch, off, bit);
    const unsigned byte = rec[off + (bit >> 3)];          // little-endian half-words: bit 8.. is the second byte
    unsigned code = (byte >> (bit & 7)) & ((1u << (c.bits == 3 ? 2 : c.bits)) - 1u);
    if (c.bits == 3) {                                    // the third bit lives in the 1-bit plane
        if (which == 0) k_hi_location(r, ch, off, bit); else v_hi_location(r, ch, off, bit);
        code |= ((static_cast<unsigned>(rec[off + (bit >> 3)]) >> (bit & 7)) & 1u) << 2;
    }
    codes[idx] = static_cast<unsigned char>(code);
    if (ch == 0) {
        const __half* meta = reinterpret_cast<const __half*>(rec + meta_location(c.bits, r));
        scale[tok] = __half2float(meta[2 * which]);
        zero[tok] = __half2float(meta[2 * which + 1]);
    }
}

// alpha_b of Eq. 5: the endpoint of the evenly spaced 2^b-level grid with the least mean squared error on a
// standard Gaussian (the paper prints no value).  Ternary search on the closed-form error.
static double quest_grid_mse(double alpha, int bits) {
    const int n = 1 << bits;
    const double step = 2.0 * alpha / (n - 1), s2pi = std::sqrt(2.0 * 3.14159265358979323846);
    auto pdf = [&](double t) { return std::isinf(t) ? 0.0 : std::exp(-0.5 * t * t) / s2pi; };
    auto cdf = [&](double t) { return 0.5 * std::erfc(-t / std::sqrt(2.0)); };
    double mse = 0.0;
    for (int k = 0; k < n; ++k) {
        const double c = -alpha + k * step;
        const double a = k == 0 ? -INFINITY : c - 0.5 * step, b = k == n - 1 ? INFINITY : c + 0.5 * step;
        const double m0 = cdf(b) - cdf(a), m1 = pdf(a) - pdf(b);
        const double m2 = m0 + (std::isinf(a) ? 0.0 : a * pdf(a)) - (std::isinf(b) ? 0.0 : b * pdf(b));
        mse += m2 - 2.0 * c * m1 + c * c * m0;
    }
    return mse;
}
static double quest_alpha(int bits) {
    double lo = 1e-3, hi = 8.0;
    for (int it = 0; it < 200; ++it) {
        const double a = lo + (hi - lo) / 3.0, b = hi - (hi - lo) / 3.0;
        if (quest_grid_mse(a, bits) < quest_grid_mse(b, bits)) hi = b; else lo = a;
    }
    return 0.5 * (lo + hi);
}
static ClipRule make_quest_rule(int bits) {
    static double alpha[5] = {0, 0, 0, 0, 0};          // per bit width, computed on first use
    if (alpha[bits] == 0) alpha[bits] = quest_alpha(bits);
    ClipRule r;
    r.rounds = 1; r.frac = 0.f;
    r.quest = static_cast<float>(2.0 * alpha[bits] / (((1 << bits) - 1) * std::sqrt(static_cast<double>(D))));
    return r;
}

static ClipRule make_rule(float kappa) {
    const double pos = static_cast<double>(kappa) * (D - 1);
    int lo = static_cast<int>(std::floor(pos));
    lo = std::min(std::max(lo, 0), D - 1);
    ClipRule r;
    r.quest = 0.f;
    if (lo >= D - 1) { r.rounds = 1; r.frac = 0.f; }
    else { r.rounds = D - lo; r.frac = static_cast<float>(pos - lo); }
    return r;
}

}  // namespace wushkv

using namespace wushkv;

static int append_impl(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                       const int32_t* cu_new, int32_t total_new, int32_t max_new,
                       const uint16_t* K_new, const uint16_t* V_new, const wushkv_prologue* prologue, void* stream) {
    AppendParams P;
    const int rc = make_view(cache, P.c);
    if (rc != WUSHKV_OK) return rc;
    P.pro = Prologue{nullptr, 0, 0, nullptr, 0.f};
    P.use_tma = 0;
    if (prologue && !make_prologue(prologue, prologue->k_norm_weight, P.pro)) return WUSHKV_EINVAL;
    if (batch <= 0 || !slot || !seq_len || !cu_new || total_new < 0 || max_new < 0 || max_new > total_new) return WUSHKV_EINVAL;
    if (total_new == 0) return WUSHKV_OK;
    if (!K_new || !V_new || !aligned(K_new, 16) || !aligned(V_new, 16)) return WUSHKV_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    P.batch = batch; P.total_new = total_new;
    P.slot = slot; P.seq_len = seq_len; P.cu_new = cu_new;
    P.K_new = K_new; P.V_new = V_new;
    if (cache->quantizer == WUSHKV_QUANTIZER_QUEST) {
        P.rule_k = P.rule_v = make_quest_rule(cache->bits);
    } else {
        P.rule_k = make_rule(cache->kappa_k);
        P.rule_v = make_rule(cache->kappa_v);
    }
    P.wait_limit = static_cast<int>(std::min<long long>(std::max<long long>(knobs().wait_limit, 0), 1 << 30));
    P.drop_mma_commit = knobs().drop_chunk_mma;
    if (max_new == 1 && P.c.n_kv <= 8 && batch <= 65535) {    // decode-time append: a cluster of one CTA per KV head for every sequence, single launch
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = P.c.n_kv;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(P.c.n_kv, batch);
        cfg.blockDim = dim3(128);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        const cudaError_t e1 = P.c.bits == 2 ? cudaLaunchKernelEx(&cfg, append_token_kernel<2>, P)
                             : P.c.bits == 3 ? cudaLaunchKernelEx(&cfg, append_token_kernel<3>, P)
                                             : cudaLaunchKernelEx(&cfg, append_token_kernel<4>, P);
        return e1 == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
    }
    const bool force_cuda = knobs().append_path_cuda != 0;             // testing aid: CUDA-core path for chunks too
    if (max_new >= TC_TILE && !force_cuda) {    // prefill chunk: tensor-core transform
        const int n_tiles = (total_new + TC_TILE - 1) / TC_TILE;
        const int per_head = std::max(1, std::min(n_tiles, 2 * sm_count() / P.c.n_kv));
        const dim3 grid_tc(per_head, P.c.n_kv);
        // list length of the quad quantizer: the rule's rounds must fit (kappa >= ~0.945 -> 8, >= ~0.882 -> 16)
        const int need = std::max(P.rule_k.rounds, P.rule_v.rounds);
        const bool quest = P.rule_k.quest > 0.f;
        const int kk_k = quest ? -1 : need > 16 ? 0 : (P.rule_k.rounds <= 8 ? 8 : 16);
        const int kk_v = quest ? -1 : need > 16 ? 0 : (P.rule_v.rounds <= 8 ? 8 : 16);
        // tensor maps of the new keys and values (not for projected keys, whose tile is rewritten in place in the plain layout)
        CUtensorMap map_k, map_v;
        const bool mk = make_row_tensor_map(map_k, true, K_new, P.c.n_kv, total_new, TC_TILE);
        const bool mv = make_row_tensor_map(map_v, true, V_new, P.c.n_kv, total_new, TC_TILE);
        P.use_tma = (mk && mv && !P.pro.rope && !knobs().append_no_tma) ? 1 : 0;
        auto launch = [&](auto kernel) -> bool {
            if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(kernel), TC_SMEM_TOTAL)) return false;
            kernel<<<grid_tc, TC_THREADS, TC_SMEM_TOTAL, st>>>(P, map_k, map_v);
            return true;
        };
        bool ok;
        if (P.c.bits == 2) {
            if (kk_k < 0) ok = launch(append_chunk_kernel<2, -1, -1>);
            else if (kk_k == 0) ok = launch(append_chunk_kernel<2, 0, 0>);
            else if (kk_k == 8 && kk_v == 8) ok = launch(append_chunk_kernel<2, 8, 8>);
            else if (kk_k == 8) ok = launch(append_chunk_kernel<2, 8, 16>);
            else if (kk_v == 8) ok = launch(append_chunk_kernel<2, 16, 8>);
            else ok = launch(append_chunk_kernel<2, 16, 16>);
        } else if (P.c.bits == 3) {
            if (kk_k < 0) ok = launch(append_chunk_kernel<3, -1, -1>);
            else if (kk_k == 0) ok = launch(append_chunk_kernel<3, 0, 0>);
            else if (kk_k == 8 && kk_v == 8) ok = launch(append_chunk_kernel<3, 8, 8>);
            else if (kk_k == 8) ok = launch(append_chunk_kernel<3, 8, 16>);
            else if (kk_v == 8) ok = launch(append_chunk_kernel<3, 16, 8>);
            else ok = launch(append_chunk_kernel<3, 16, 16>);
        } else {
            if (kk_k < 0) ok = launch(append_chunk_kernel<4, -1, -1>);
            else if (kk_k == 0) ok = launch(append_chunk_kernel<4, 0, 0>);
            else if (kk_k == 8 && kk_v == 8) ok = launch(append_chunk_kernel<4, 8, 8>);
            else if (kk_k == 8) ok = launch(append_chunk_kernel<4, 8, 16>);
            else if (kk_v == 8) ok = launch(append_chunk_kernel<4, 16, 8>);
            else ok = launch(append_chunk_kernel<4, 16, 16>);
        }
        if (!ok) return WUSHKV_ECUDA;
        if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
        advance_len_kernel<<<(batch + 127) / 128, 128, 0, st>>>(P.c, batch, slot, seq_len, cu_new);
        return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
    }
    // enough CTAs to fill the machine, but at least 8 tokens each to amortise the transform load
    const int want_ctas = std::max(1, 2 * sm_count() / P.c.n_kv);
    int tpc = (total_new + want_ctas - 1) / want_ctas;
    tpc = std::max(8, ((tpc + 7) / 8) * 8);
    P.tokens_per_cta = tpc;
    const dim3 grid((total_new + tpc - 1) / tpc, P.c.n_kv);
    const size_t smem = static_cast<size_t>(D) * TT_STRIDE * sizeof(float);
    if (P.c.bits == 2) {
        if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(append_rows_kernel<2>), static_cast<int>(smem))) return WUSHKV_ECUDA;
        append_rows_kernel<2><<<grid, 256, smem, st>>>(P);
    } else if (P.c.bits == 3) {
        if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(append_rows_kernel<3>), static_cast<int>(smem))) return WUSHKV_ECUDA;
        append_rows_kernel<3><<<grid, 256, smem, st>>>(P);
    } else {
        if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(append_rows_kernel<4>), static_cast<int>(smem))) return WUSHKV_ECUDA;
        append_rows_kernel<4><<<grid, 256, smem, st>>>(P);
    }
    if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
    advance_len_kernel<<<(batch + 127) / 128, 128, 0, st>>>(P.c, batch, slot, seq_len, cu_new);
    if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
    return WUSHKV_OK;
}

extern "C" int wushkv_append(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                             const int32_t* cu_new, int32_t total_new, int32_t max_new,
                             const uint16_t* K_new, const uint16_t* V_new, void* stream) {
    return append_impl(cache, batch, slot, seq_len, cu_new, total_new, max_new, K_new, V_new, nullptr, stream);
}

extern "C" int wushkv_append_projected(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                                       const int32_t* cu_new, int32_t total_new, int32_t max_new,
                                       const uint16_t* K_proj, const uint16_t* V_new, const wushkv_prologue* prologue, void* stream) {
    if (!prologue) return WUSHKV_EINVAL;
    return append_impl(cache, batch, slot, seq_len, cu_new, total_new, max_new, K_proj, V_new, prologue, stream);
}

// cosines and sines of position * theta^(-2j/d) in double precision, rounded to fp32
__global__ void rope_table_kernel(double theta, int n_pos, float2* table) {
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<long long>(n_pos) * (D / 2)) return;
    const int j = static_cast<int>(idx % (D / 2));
    const double pos = static_cast<double>(idx / (D / 2));
    double sn, cs;
    sincos(pos * pow(theta, -2.0 * j / D), &sn, &cs);
    table[idx] = make_float2(static_cast<float>(cs), static_cast<float>(sn));
}

extern "C" int wushkv_build_rope_table(double theta, int32_t n_positions, int32_t d, float* table, void* stream) {
    if (!(theta > 0.0) || n_positions <= 0 || d != D || !table || !aligned(table, 16)) return WUSHKV_EINVAL;
    const long long n = static_cast<long long>(n_positions) * (D / 2);
    rope_table_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(theta, n_positions, reinterpret_cast<float2*>(table));
    return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
}

extern "C" int wushkv_unpack_debug(const wushkv_cache* cache, int32_t slot, int32_t kv_head, int32_t which,
                                   int32_t pos0, int32_t n, uint8_t* codes, float* scale, float* zero, void* stream) {
    CacheView v;
    const int rc = make_view(cache, v);
    if (rc != WUSHKV_OK) return rc;
    if (slot < 0 || slot >= v.n_slots || kv_head < 0 || kv_head >= v.n_kv || (which != 0 && which != 1) || pos0 < 0 || n < 0 ||
        !codes || !scale || !zero)
        return WUSHKV_EINVAL;
    if (n == 0) return WUSHKV_OK;
    const long long total = static_cast<long long>(n) * D;
    unpack_debug_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        v, slot, kv_head, which, pos0, n, codes, scale, zero);
    return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
}
