// Decode attention over the packed cache (Algorithm 2 lines 3 and 5; Eq. 2; Eq. 3; Section 4.4).
//
// Three launches on the caller's stream:
//   1. decode_prep_kernel   q' = T_K^{-T} q per query head (Algorithm 2 line 3), written (a) as fp32
//                           for the bf16 windows and (b) as fp16 mma B-fragments, pre-scaled by the
//                           power of two that each packed code field carries.
//   2. decode_main_kernel   one CTA per (sequence, KV head, split of the quantized range) plus one
//                           CTA per (sequence, KV head) for the bf16 sink / recent windows.  Each warp
//                           streams whole 64-token page records into shared memory with bulk async
//                           copies (mbarrier ring), turns code words into fp16 A-fragments with one
//                           AND per register, and runs both contractions (q'.k and p.v) on
//                           mma.sync.m16n8k16 with fp32 accumulation.  The affine part of Eq. 6 is
//                           factored out of the contractions:
//                               q'.k_hat = Delta_k (q'.c_k) + x_min_k sum(q'),
//                               o        = sum_s (p_s Delta_v,s) c_v,s + (sum_s p_s x_min_v,s) 1.
//                           Softmax is online (running max / sum) per warp, merged per CTA.
//   3. decode_combine_kernel merges the per-split (max, sum, o) partials into O.
//
// No kernel waits on another CTA.  The only waits are on this warp's own copy barriers, bounded by
// an iteration limit after which the kernel records WUSHKV_DEV_COPY_TIMEOUT and drains.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>

#include "host_common.h"
#include "layout.cuh"

namespace wushkv {

constexpr unsigned FULL = 0xffffffffu;
constexpr int PART_STRIDE = 132;          // floats per partial: [0]=max (log2 domain) [1]=sum [4..131]=o
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LO_SCALE = 2048.f;        // the "lo" fp16 column carries (x - fp16(x)) * 2^11
constexpr float PV_SCALE = 16.f;          // p * Delta_v is fed to the tensor core as fp16(p Delta_v 2^4)
constexpr int MAIN_WARPS = 4;

struct DecodeParams {
    CacheView c;
    int batch;
    const int* slot;
    const int* seq_len;
    const unsigned short* Q;
    float* O;
    uint4* qfrag;      // [batch][n_kv][4][32] uint4: B fragments of the 8 k-steps
    float* qscal;      // [batch][n_q][2]: (score multiplier, x_min multiplier) in the log2 domain
    float* qcomp;      // [batch][n_q][128]: q' * sm_scale * log2(e), fp32, for the bf16 windows
    float* part;       // [batch][n_q][n_chunks + 1][PART_STRIDE]
    int n_chunks;      // splits of the quantized range; split index n_chunks is the window split
    int chunk_pages;
};

// shift of the code field used by k-step / channel block idx (0..7) inside its 16-bit lane, after
// the optional whole-word shift: the fp16 value of the masked field is code * 2^(field_shift - 24)
template <int BITS>
__host__ __device__ constexpr int field_shift(int idx) {
    return BITS == 2 ? (idx < 5 ? 2 * idx : 2 * (idx - 5)) : 4 * (idx & 1);
}

// ------------------------------------------------------------------------------------------------
// 1. query preparation
// ------------------------------------------------------------------------------------------------
template <int BITS, int MODE>
__global__ void __launch_bounds__(128) decode_prep_kernel(DecodeParams P) {
    __shared__ float q_s[8][D];
    __shared__ float red_max[8][4];
    __shared__ float red_sum[8][4];
    const int h = blockIdx.x, b = blockIdx.y, G = P.c.G;
    const int i = threadIdx.x, lane = i & 31, warp = i >> 5;
    for (int g = 0; g < G; ++g)
        q_s[g][i] = bf16_bits_to_float(P.Q[(static_cast<long long>(b) * P.c.n_q + h * G + g) * D + i]);
    __syncthreads();
    float acc[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) acc[g] = 0.f;
    const float4* Trow = reinterpret_cast<const float4*>(P.c.T_K_invT + (static_cast<long long>(h) * D + i) * D);
    for (int j4 = 0; j4 < D / 4; ++j4) {
        const float4 t = __ldg(Trow + j4);
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            if (g < G) {
                const float4 qv = *reinterpret_cast<const float4*>(&q_s[g][4 * j4]);
                acc[g] = fmaf(t.x, qv.x, acc[g]); acc[g] = fmaf(t.y, qv.y, acc[g]);
                acc[g] = fmaf(t.z, qv.z, acc[g]); acc[g] = fmaf(t.w, qv.w, acc[g]);
            }
        }
    }
    const int s = i >> 4;
    const float pos_scale = exp2f(-static_cast<float>(field_shift<BITS>(s)));
    const float k2 = P.c.sm_scale * LOG2E;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < G) {
            P.qcomp[(static_cast<long long>(b) * P.c.n_q + h * G + g) * D + i] = acc[g] * k2;
            float mx = fabsf(acc[g]) * pos_scale, sm = acc[g];
            for (int o = 16; o > 0; o >>= 1) {
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
                sm += __shfl_xor_sync(FULL, sm, o);
            }
            if (lane == 0) { red_max[g][warp] = mx; red_sum[g][warp] = sm; }
        }
    }
    __syncthreads();
    float beta[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        beta[g] = 1.f;
        if (g < G) {
            const float mx = fmaxf(fmaxf(red_max[g][0], red_max[g][1]), fmaxf(red_max[g][2], red_max[g][3]));
            int e = 0;
            if (mx > 0.f && mx < 3e38f) frexpf(mx, &e);          // mx < 2^e
            e = max(min(e, 100), -100);
            beta[g] = exp2f(static_cast<float>(14 - e));         // scaled entries stay below 2^14
            if (i == 0) {
                const float sum = red_sum[g][0] + red_sum[g][1] + red_sum[g][2] + red_sum[g][3];
                float* qs = P.qscal + (static_cast<long long>(b) * P.c.n_q + h * G + g) * 2;
                qs[0] = k2 * 16777216.f / beta[g];
                qs[1] = k2 * sum;
            }
        }
    }
    // B fragments: column n of the mma holds, for MODE 0, head n>>1 as its fp16 value (n even) or the
    // scaled rounding remainder (n odd); for MODE 1, head n.
    const int r16 = i & 15, r = r16 >> 3, t = (r16 & 7) >> 1, hf = r16 & 1;
    unsigned short* frag = reinterpret_cast<unsigned short*>(P.qfrag + (static_cast<long long>(b) * P.c.n_kv + h) * 128);
#pragma unroll
    for (int n = 0; n < 8; ++n) {
        const int head = (MODE == 0) ? (n >> 1) : n;
        float val = 0.f;
        if (head < G) {
            const float x = acc[head] * pos_scale * beta[head];
            const __half hi = __float2half_rn(x);
            val = (MODE == 0 && (n & 1)) ? (x - __half2float(hi)) * LO_SCALE : x;
        }
        const int lane_dst = 4 * n + t;
        frag[((((s >> 1) * 32 + lane_dst) * 4 + (s & 1) * 2 + r) << 1) + hf] = __half_as_ushort(__float2half_rn(val));
    }
}

// ------------------------------------------------------------------------------------------------
// 2. main kernel helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the limit.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity) {
    for (int it = 0; it < (1 << 22); ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_copy_g2s(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds128(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void mma16816(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned movmatrix_trans(unsigned a) {
    unsigned d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ unsigned pack_h2(float lo, float hi) {      // lo -> bits 0..15, hi -> bits 16..31, saturating
    unsigned d;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float h_lo(unsigned u) { return __half2float(__ushort_as_half(static_cast<unsigned short>(u & 0xffffu))); }
__device__ __forceinline__ float h_hi(unsigned u) { return __half2float(__ushort_as_half(static_cast<unsigned short>(u >> 16))); }

// Field idx (0..7) of a code word as an fp16x2 A-fragment register.  `w` is the raw word, `ws` the
// same word shifted right so that the upper fields fall into the low bits of each 16-bit lane.
template <int BITS>
__device__ __forceinline__ unsigned field(unsigned w, unsigned ws, int idx) {
    if (BITS == 2) {
        constexpr unsigned M0 = 0x00030003u;
        return idx < 5 ? (w & (M0 << (2 * idx))) : (ws & (M0 << (2 * (idx - 5))));
    } else {
        constexpr unsigned M0 = 0x000F000Fu;
        return idx < 2 ? (w & (M0 << (4 * idx))) : (ws & (M0 << (4 * (idx - 2))));
    }
}
template <int BITS> __device__ __forceinline__ unsigned pre_shift(unsigned w) { return BITS == 2 ? (w >> 10) : (w >> 8); }

// Per-warp running softmax state.  MODE 0: one head per thread (head t, value and rounding remainder
// in the two accumulator columns).  MODE 1: two heads per thread (2t, 2t+1).
template <int MODE>
struct WarpState {
    static constexpr int NH = MODE == 0 ? 1 : 2;
    float m[NH], l[NH], z[NH];
    float o[8][4];
};

// Writes this warp's partial (max, sum, o[128]) of every head into shared scratch [warp][head][PART_STRIDE].
template <int BITS, int MODE>
__device__ __forceinline__ void spill_warp_state(WarpState<MODE>& st, float* scratch_warp, int lane, int G) {
    const int g = lane >> 2, t = lane & 3;
    constexpr int NH = WarpState<MODE>::NH;
#pragma unroll
    for (int k = 0; k < NH; ++k) {
        float l = st.l[k], z = st.z[k];
        l += __shfl_xor_sync(FULL, l, 4);  z += __shfl_xor_sync(FULL, z, 4);
        l += __shfl_xor_sync(FULL, l, 8);  z += __shfl_xor_sync(FULL, z, 8);
        l += __shfl_xor_sync(FULL, l, 16); z += __shfl_xor_sync(FULL, z, 16);
        const int head = MODE == 0 ? t : 2 * t + k;
        if (head < G) {
            float* dst = scratch_warp + head * PART_STRIDE;
            if (g == 0) { dst[0] = st.m[k]; dst[1] = l; }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float osc = exp2f(static_cast<float>(24 - field_shift<BITS>(i))) / PV_SCALE;
                float lo_ch, hi_ch;
                if (MODE == 0) {
                    lo_ch = (st.o[i][0] + st.o[i][1] * (1.f / LO_SCALE)) * osc + z;
                    hi_ch = (st.o[i][2] + st.o[i][3] * (1.f / LO_SCALE)) * osc + z;
                } else {
                    lo_ch = st.o[i][k] * osc + z;
                    hi_ch = st.o[i][2 + k] * osc + z;
                }
                dst[4 + 16 * i + g] = lo_ch;
                dst[4 + 16 * i + g + 8] = hi_ch;
            }
        }
    }
}

// Merge the per-warp partials in shared scratch and write this CTA's partial to global memory.
__device__ __forceinline__ void merge_and_store(const float* scratch, int nwarps, int G, float* part_base,
                                                long long head_stride, int tid, int nthreads) {
    for (int idx = tid; idx < G * D; idx += nthreads) {
        const int head = idx >> 7, ch = idx & 127;
        float m = -INFINITY;
        for (int w = 0; w < nwarps; ++w) m = fmaxf(m, scratch[(w * 8 + head) * PART_STRIDE]);
        float l = 0.f, o = 0.f;
        for (int w = 0; w < nwarps; ++w) {
            const float* p = scratch + (w * 8 + head) * PART_STRIDE;
            const float sc = (p[0] == -INFINITY) ? 0.f : exp2f(p[0] - m);
            l += sc * p[1];
            o += sc * p[4 + ch];
        }
        float* dst = part_base + head * head_stride;
        if (ch == 0) { dst[0] = m; dst[1] = l; }
        dst[4 + ch] = o;
    }
}

// ------------------------------------------------------------------------------------------------
// bf16 windows (sink + recent ring), CUDA cores, fp32
// ------------------------------------------------------------------------------------------------
__device__ void window_split(const DecodeParams& P, int b, int h, int slot, int S, int nq, float* scratch) {
    const CacheView& c = P.c;
    const int G = c.G;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int n_sink = min(S, c.s_sink);
    const int recent_lo = c.s_sink + nq;
    const int n_recent = max(0, S - recent_lo);
    float q[8][4];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < G) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(P.qcomp + (static_cast<long long>(b) * c.n_q + h * G + g) * D) + lane);
            q[g][0] = v.x; q[g][1] = v.y; q[g][2] = v.z; q[g][3] = v.w;
        } else {
            q[g][0] = q[g][1] = q[g][2] = q[g][3] = 0.f;
        }
    }
    float m[8], l[8], o[8][4];
#pragma unroll
    for (int g = 0; g < 8; ++g) { m[g] = -INFINITY; l[g] = 0.f; o[g][0] = o[g][1] = o[g][2] = o[g][3] = 0.f; }
    const long long head_base = (static_cast<long long>(slot) * c.n_kv + h) * 2;
    for (int w = warp; w < n_sink + n_recent; w += nwarps) {
        const unsigned short *kp, *vp;
        if (w < n_sink) {
            kp = c.sink_kv + ((head_base + 0) * c.s_sink + w) * D;
            vp = c.sink_kv + ((head_base + 1) * c.s_sink + w) * D;
        } else {
            const int row = (recent_lo + (w - n_sink)) % c.ring_cap;
            kp = c.ring_kv + ((head_base + 0) * c.ring_cap + row) * D;
            vp = c.ring_kv + ((head_base + 1) * c.ring_cap + row) * D;
        }
        const uint2 kr = __ldg(reinterpret_cast<const uint2*>(kp) + lane);
        const uint2 vr = __ldg(reinterpret_cast<const uint2*>(vp) + lane);
        const float k0 = bf16_bits_to_float(kr.x & 0xffff), k1 = bf16_bits_to_float(kr.x >> 16);
        const float k2 = bf16_bits_to_float(kr.y & 0xffff), k3 = bf16_bits_to_float(kr.y >> 16);
        const float v0 = bf16_bits_to_float(vr.x & 0xffff), v1 = bf16_bits_to_float(vr.x >> 16);
        const float v2 = bf16_bits_to_float(vr.y & 0xffff), v3 = bf16_bits_to_float(vr.y >> 16);
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            if (g < G) {
                float s = q[g][0] * k0 + q[g][1] * k1 + q[g][2] * k2 + q[g][3] * k3;
                for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(FULL, s, off);
                const float mn = fmaxf(m[g], s);
                const float sc = exp2f(m[g] - mn);            // m = -inf on the first token: sc = 0
                const float p = exp2f(s - mn);
                l[g] = l[g] * sc + p;
                o[g][0] = o[g][0] * sc + p * v0; o[g][1] = o[g][1] * sc + p * v1;
                o[g][2] = o[g][2] * sc + p * v2; o[g][3] = o[g][3] * sc + p * v3;
                m[g] = mn;
            }
        }
    }
    float* mine = scratch + warp * 8 * PART_STRIDE;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < G) {
            float* dst = mine + g * PART_STRIDE;
            if (lane == 0) { dst[0] = m[g]; dst[1] = l[g]; }
            *reinterpret_cast<float4*>(dst + 4 + 4 * lane) = make_float4(o[g][0], o[g][1], o[g][2], o[g][3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// main kernel
// ------------------------------------------------------------------------------------------------
template <int BITS, int MODE, int STAGES>
__global__ void __launch_bounds__(MAIN_WARPS * 32) decode_main_kernel(DecodeParams P) {
    constexpr int REC = record_bytes(BITS);
    constexpr int CB = code_block_bytes(BITS);
    constexpr int NH = WarpState<MODE>::NH;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* stage_base = smem;                                               // [MAIN_WARPS][STAGES][REC]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + MAIN_WARPS * STAGES * REC);
    float* scratch = reinterpret_cast<float*>(smem);                                // reused after the stream is drained
    const CacheView& c = P.c;
    const int b = blockIdx.z, h = blockIdx.y, chunk = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = c.G;
    const int slot = __ldg(P.slot + b);
    const int S = __ldg(P.seq_len + b);
    const int n_splits = P.n_chunks + 1;
    float* part_base = P.part + ((static_cast<long long>(b) * c.n_q + h * G) * n_splits + chunk) * PART_STRIDE;
    const long long head_stride = static_cast<long long>(n_splits) * PART_STRIDE;
    if (slot < 0 || slot >= c.n_slots) {
        if (tid == 0) atomicOr(c.dev_status, WUSHKV_DEV_BAD_SLOT);
        return;
    }
    const int nq = (S > 0) ? n_quantized(S - c.lag, c.s_sink, c.s_keep, c.s_flush) : 0;

    if (chunk == P.n_chunks) {          // ---- the bf16 windows
        window_split(P, b, h, slot, max(S, 0), nq, scratch);
        __syncthreads();
        merge_and_store(scratch, MAIN_WARPS, G, part_base, head_stride, tid, blockDim.x);
        return;
    }
    if (nq <= 0) return;
    const int q_lo = c.s_sink, q_hi = c.s_sink + nq;
    const int first_page = q_lo / PAGE_TOKENS, last_page = (q_hi - 1) / PAGE_TOKENS;
    const int pg0 = first_page + chunk * P.chunk_pages;
    const int pg1 = min(pg0 + P.chunk_pages, last_page + 1);
    if (pg0 >= pg1) return;

    // ---- barriers
    const unsigned bar0 = smem_u32(bars + warp * STAGES);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const unsigned stage0 = smem_u32(stage_base + warp * STAGES * REC);
    const int* ptab = c.page_table + static_cast<long long>(slot) * c.max_pages;

    unsigned bad_stage = 0;             // lane 0: bit s set if the page staged in s could not be fetched
    auto issue = [&](int pg, int s) {   // lane 0 only
        const int page = (pg < c.max_pages) ? __ldg(ptab + pg) : -1;
        if (page < 0 || page >= c.n_pages) {
            atomicOr(c.dev_status, pg < c.max_pages ? WUSHKV_DEV_BAD_PAGE_ID : WUSHKV_DEV_PAGE_TABLE_FULL);
            bad_stage |= 1u << s;
            mbar_arrive(bar0 + 8 * s);
        } else {
            bad_stage &= ~(1u << s);
            const unsigned char* src = c.pages + (static_cast<long long>(page) * c.n_kv + h) * REC;
            mbar_expect_tx(bar0 + 8 * s, REC);
            bulk_copy_g2s(stage0 + s * REC, src, REC, bar0 + 8 * s);
        }
    };
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            const int pg = pg0 + warp + s * MAIN_WARPS;
            if (pg < pg1) issue(pg, s);
        }
    }

    // ---- query fragments and per-head scalars
    unsigned qf[8][2];
    {
        const uint4* src = P.qfrag + (static_cast<long long>(b) * c.n_kv + h) * 128;
#pragma unroll
        for (int s2 = 0; s2 < 4; ++s2) {
            const uint4 v = __ldg(src + s2 * 32 + lane);
            qf[2 * s2][0] = v.x; qf[2 * s2][1] = v.y; qf[2 * s2 + 1][0] = v.z; qf[2 * s2 + 1][1] = v.w;
        }
    }
    float fmul[NH], gadd[NH];
#pragma unroll
    for (int k = 0; k < NH; ++k) {
        const int head = MODE == 0 ? t : 2 * t + k;
        fmul[k] = gadd[k] = 0.f;
        if (head < G) {
            const float2 v = __ldg(reinterpret_cast<const float2*>(P.qscal + (static_cast<long long>(b) * c.n_q + h * G + head) * 2));
            fmul[k] = v.x; gadd[k] = v.y;
        }
    }

    WarpState<MODE> st;
#pragma unroll
    for (int k = 0; k < NH; ++k) { st.m[k] = -INFINITY; st.l[k] = 0.f; st.z[k] = 0.f; }
#pragma unroll
    for (int i = 0; i < 8; ++i) st.o[i][0] = st.o[i][1] = st.o[i][2] = st.o[i][3] = 0.f;

    bool timed_out = false;
    int it = 0;
    for (int pg = pg0 + warp; pg < pg1; pg += MAIN_WARPS, ++it) {
        const int s = it % STAGES;
        const unsigned parity = (it / STAGES) & 1;
        // a phase that one lane saw complete is complete for all: keep the decision warp-uniform
        if (!__any_sync(FULL, mbar_wait_bounded(bar0 + 8 * s, parity))) { timed_out = true; break; }
        const bool bad = __shfl_sync(FULL, (bad_stage >> s) & 1u, 0) != 0;
        if (!bad) {
            const unsigned rec = stage0 + s * REC;
            const int pos0 = pg * PAGE_TOKENS;
            const bool full_page = (pos0 >= q_lo) && (pos0 + PAGE_TOKENS <= q_hi);
            // ---------------- scores of the 64 tokens
            float sc[4][2 * NH];          // [block][row g: heads..., row g+8: heads...]
            unsigned vmeta[4][2];         // fp16x2 (Delta_v, x_min_v) of rows g, g+8
#pragma unroll
            for (int bi = 0; bi < 4; ++bi) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                if (BITS == 2) {
                    const uint4 kw = lds128(rec + bi * CB + 16 * lane);
                    const unsigned sx = pre_shift<2>(kw.x), sy = pre_shift<2>(kw.y), sz = pre_shift<2>(kw.z), sw = pre_shift<2>(kw.w);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma16816(acc, field<2>(kw.x, sx, ks), field<2>(kw.z, sz, ks), field<2>(kw.y, sy, ks), field<2>(kw.w, sw, ks),
                                 qf[ks][0], qf[ks][1]);
                } else {
                    const uint4 ka = lds128(rec + bi * CB + 16 * lane);          // row g:   W0..W3
                    const uint4 kb = lds128(rec + bi * CB + 512 + 16 * lane);    // row g+8: W0..W3
                    const unsigned a0s = pre_shift<4>(ka.x), a1s = pre_shift<4>(ka.y), a2s = pre_shift<4>(ka.z), a3s = pre_shift<4>(ka.w);
                    const unsigned b0s = pre_shift<4>(kb.x), b1s = pre_shift<4>(kb.y), b2s = pre_shift<4>(kb.z), b3s = pre_shift<4>(kb.w);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma16816(acc, field<4>(ka.x, a0s, ks), field<4>(kb.x, b0s, ks), field<4>(ka.y, a1s, ks), field<4>(kb.y, b1s, ks),
                                 qf[ks][0], qf[ks][1]);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma16816(acc, field<4>(ka.z, a2s, ks), field<4>(kb.z, b2s, ks), field<4>(ka.w, a3s, ks), field<4>(kb.w, b3s, ks),
                                 qf[4 + ks][0], qf[4 + ks][1]);
                }
                const uint4 mt = lds128(rec + meta_offset(BITS) + 128 * bi + 16 * g);   // rows g (x,y) and g+8 (z,w)
                float kd0 = h_lo(mt.x), km0 = h_hi(mt.x), kd1 = h_lo(mt.z), km1 = h_hi(mt.z);
                unsigned vm0 = mt.y, vm1 = mt.w;
                bool ok0 = true, ok1 = true;
                if (!full_page) {
                    const int p0 = pos0 + bi * 16 + g, p1 = p0 + 8;
                    ok0 = (p0 >= q_lo) && (p0 < q_hi);
                    ok1 = (p1 >= q_lo) && (p1 < q_hi);
                    if (!ok0) vm0 = 0u;
                    if (!ok1) vm1 = 0u;
                }
                vmeta[bi][0] = vm0; vmeta[bi][1] = vm1;
                if (MODE == 0) {
                    const float d0 = acc[0] + acc[1] * (1.f / LO_SCALE), d1 = acc[2] + acc[3] * (1.f / LO_SCALE);
                    const float s0 = fmaf(d0 * kd0, fmul[0], km0 * gadd[0]);
                    const float s1 = fmaf(d1 * kd1, fmul[0], km1 * gadd[0]);
                    sc[bi][0] = ok0 ? s0 : -INFINITY;
                    sc[bi][1] = ok1 ? s1 : -INFINITY;
                } else {
                    const float s00 = fmaf(acc[0] * kd0, fmul[0], km0 * gadd[0]);
                    const float s01 = fmaf(acc[1] * kd0, fmul[1], km0 * gadd[1]);
                    const float s10 = fmaf(acc[2] * kd1, fmul[0], km1 * gadd[0]);
                    const float s11 = fmaf(acc[3] * kd1, fmul[1], km1 * gadd[1]);
                    sc[bi][0] = ok0 ? s00 : -INFINITY; sc[bi][1] = ok0 ? s01 : -INFINITY;
                    sc[bi][2] = ok1 ? s10 : -INFINITY; sc[bi][3] = ok1 ? s11 : -INFINITY;
                }
            }
            // ---------------- running maximum of the page, rescale if it grew
            float mref[NH], mnew[NH];
            bool grew = false;
#pragma unroll
            for (int k = 0; k < NH; ++k) {
                float mx;
                if (MODE == 0) mx = fmaxf(fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])),
                                          fmaxf(fmaxf(sc[2][0], sc[2][1]), fmaxf(sc[3][0], sc[3][1])));
                else mx = fmaxf(fmaxf(fmaxf(sc[0][k], sc[0][2 + k]), fmaxf(sc[1][k], sc[1][2 + k])),
                                fmaxf(fmaxf(sc[2][k], sc[2][2 + k]), fmaxf(sc[3][k], sc[3][2 + k])));
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 16));
                mnew[k] = fmaxf(st.m[k], mx);
                grew |= mnew[k] > st.m[k];
                mref[k] = (mnew[k] == -INFINITY) ? 0.f : mnew[k];     // all-masked so far: any finite reference works
            }
            if (__any_sync(FULL, grew)) {
                float scl[NH];
#pragma unroll
                for (int k = 0; k < NH; ++k) {
                    scl[k] = exp2f(st.m[k] - mref[k]);                // old max -inf: state is all zero, factor 0
                    st.l[k] *= scl[k]; st.z[k] *= scl[k];
                    st.m[k] = mnew[k];
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (MODE == 0) { st.o[i][0] *= scl[0]; st.o[i][1] *= scl[0]; st.o[i][2] *= scl[0]; st.o[i][3] *= scl[0]; }
                    else { st.o[i][0] *= scl[0]; st.o[i][1] *= scl[1]; st.o[i][2] *= scl[0]; st.o[i][3] *= scl[1]; }
                }
            }
            // ---------------- probabilities, value reduction
#pragma unroll
            for (int bi = 0; bi < 4; ++bi) {
                const float vd0 = h_lo(vmeta[bi][0]), vn0 = h_hi(vmeta[bi][0]);
                const float vd1 = h_lo(vmeta[bi][1]), vn1 = h_hi(vmeta[bi][1]);
                unsigned r0, r1;
                if (MODE == 0) {
                    const float p0 = exp2f(sc[bi][0] - mref[0]), p1 = exp2f(sc[bi][1] - mref[0]);
                    st.l[0] += p0 + p1;
                    st.z[0] = fmaf(p0, vn0, fmaf(p1, vn1, st.z[0]));
                    const float w0 = p0 * vd0 * PV_SCALE, w1 = p1 * vd1 * PV_SCALE;
                    const float w0h = __half2float(__float2half_rn(w0)), w1h = __half2float(__float2half_rn(w1));
                    r0 = pack_h2(w0, (w0 - w0h) * LO_SCALE);
                    r1 = pack_h2(w1, (w1 - w1h) * LO_SCALE);
                } else {
                    const float p00 = exp2f(sc[bi][0] - mref[0]), p01 = exp2f(sc[bi][1] - mref[1]);
                    const float p10 = exp2f(sc[bi][2] - mref[0]), p11 = exp2f(sc[bi][3] - mref[1]);
                    st.l[0] += p00 + p10; st.l[1] += p01 + p11;
                    st.z[0] = fmaf(p00, vn0, fmaf(p10, vn1, st.z[0]));
                    st.z[1] = fmaf(p01, vn0, fmaf(p11, vn1, st.z[1]));
                    r0 = pack_h2(p00 * vd0 * PV_SCALE, p01 * vd0 * PV_SCALE);
                    r1 = pack_h2(p10 * vd1 * PV_SCALE, p11 * vd1 * PV_SCALE);
                }
                const unsigned b01 = movmatrix_trans(r0), b23 = movmatrix_trans(r1);
                if (BITS == 2) {
                    const uint4 vw = lds128(rec + v_codes_offset(2) + bi * CB + 16 * lane);
                    const unsigned sx = pre_shift<2>(vw.x), sy = pre_shift<2>(vw.y), sz = pre_shift<2>(vw.z), sw = pre_shift<2>(vw.w);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        mma16816(st.o[i], field<2>(vw.x, sx, i), field<2>(vw.y, sy, i), field<2>(vw.z, sz, i), field<2>(vw.w, sw, i), b01, b23);
                } else {
                    const uint4 va = lds128(rec + v_codes_offset(4) + bi * CB + 16 * lane);         // tokens 2t,2t+1
                    const uint4 vb = lds128(rec + v_codes_offset(4) + bi * CB + 512 + 16 * lane);   // tokens 2t+8,2t+9
                    const unsigned a0s = pre_shift<4>(va.x), a1s = pre_shift<4>(va.y), a2s = pre_shift<4>(va.z), a3s = pre_shift<4>(va.w);
                    const unsigned b0s = pre_shift<4>(vb.x), b1s = pre_shift<4>(vb.y), b2s = pre_shift<4>(vb.z), b3s = pre_shift<4>(vb.w);
#pragma unroll
                    for (int k = 0; k < 4; ++k)     // channel blocks 0..3: words (rsel, j=0)
                        mma16816(st.o[k], field<4>(va.x, a0s, k), field<4>(va.z, a2s, k), field<4>(vb.x, b0s, k), field<4>(vb.z, b2s, k), b01, b23);
#pragma unroll
                    for (int k = 0; k < 4; ++k)     // channel blocks 4..7: words (rsel, j=1)
                        mma16816(st.o[4 + k], field<4>(va.y, a1s, k), field<4>(va.w, a3s, k), field<4>(vb.y, b1s, k), field<4>(vb.w, b3s, k), b01, b23);
                }
            }
        }
        __syncwarp();
        const int next = pg + STAGES * MAIN_WARPS;
        if (lane == 0 && next < pg1) issue(next, s);
    }
    if (timed_out) {
        if (lane == 0) atomicOr(c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
        // give copies that may still be in flight a bounded time to land before the staging area is reused
        for (int k = 0; k < 1000; ++k) __nanosleep(1000);
    }
    __syncthreads();                    // every warp has drained its stages: the staging area becomes scratch
    spill_warp_state<BITS, MODE>(st, scratch + warp * 8 * PART_STRIDE, lane, G);
    __syncthreads();
    merge_and_store(scratch, MAIN_WARPS, G, part_base, head_stride, tid, blockDim.x);
}

// ------------------------------------------------------------------------------------------------
// 3. combine
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) decode_combine_kernel(DecodeParams P) {
    const CacheView& c = P.c;
    const int j = blockIdx.x, b = blockIdx.y, ch = threadIdx.x;
    const int S = __ldg(P.seq_len + b);
    const int slot = __ldg(P.slot + b);
    float* out = P.O + (static_cast<long long>(b) * c.n_q + j) * D;
    if (slot < 0 || slot >= c.n_slots || S <= 0) { out[ch] = 0.f; return; }
    const int nq = n_quantized(S - c.lag, c.s_sink, c.s_keep, c.s_flush);
    int valid_chunks = 0;
    if (nq > 0) {
        const int first_page = c.s_sink / PAGE_TOKENS, last_page = (c.s_sink + nq - 1) / PAGE_TOKENS;
        valid_chunks = min((last_page - first_page) / P.chunk_pages + 1, P.n_chunks);
    }
    const int n_splits = P.n_chunks + 1;
    const float* base = P.part + (static_cast<long long>(b) * c.n_q + j) * n_splits * PART_STRIDE;
    float m = base[P.n_chunks * PART_STRIDE];
    for (int s = 0; s < valid_chunks; ++s) m = fmaxf(m, base[s * PART_STRIDE]);
    float l = 0.f, o = 0.f;
    for (int s = 0; s <= valid_chunks; ++s) {
        const float* p = base + (s < valid_chunks ? s : P.n_chunks) * PART_STRIDE;
        const float scl = (p[0] == -INFINITY) ? 0.f : exp2f(p[0] - m);
        l += scl * p[1];
        o += scl * p[4 + ch];
    }
    out[ch] = l > 0.f ? o / l : 0.f;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct DecodePlan {
    int chunk_pages, n_chunks;
    size_t off_qfrag, off_qscal, off_qcomp, off_part, total;
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool make_plan(const CacheView& c, int batch, int max_seq_len, DecodePlan& pl) {
    if (batch <= 0 || max_seq_len <= 0) return false;
    const long long pages_max = (static_cast<long long>(max_seq_len) + PAGE_TOKENS - 1) / PAGE_TOKENS;
    const long long total_pages = pages_max * batch * c.n_kv;
    long long cp = 0;
    if (const char* e = std::getenv("WUSHKV_CHUNK_PAGES")) cp = std::atoll(e);
    if (cp <= 0) {
        const long long want_ctas = 8LL * sm_count();          // a few waves of CTAs for balance
        cp = (total_pages + want_ctas - 1) / want_ctas;
        cp = std::max<long long>(cp, 2 * MAIN_WARPS);
    }
    cp = std::min<long long>(cp, pages_max);
    pl.chunk_pages = static_cast<int>(cp);
    pl.n_chunks = static_cast<int>((pages_max + cp - 1) / cp);
    size_t off = 0;
    pl.off_qfrag = off; off = align_up(off + static_cast<size_t>(batch) * c.n_kv * 128 * sizeof(uint4), 256);
    pl.off_qscal = off; off = align_up(off + static_cast<size_t>(batch) * c.n_q * 2 * sizeof(float), 256);
    pl.off_qcomp = off; off = align_up(off + static_cast<size_t>(batch) * c.n_q * D * sizeof(float), 256);
    pl.off_part = off;  off = align_up(off + static_cast<size_t>(batch) * c.n_q * (pl.n_chunks + 1) * PART_STRIDE * sizeof(float), 256);
    pl.total = off;
    return true;
}

static cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;

template <int BITS, int MODE>
static int launch_decode(const DecodeParams& P, cudaStream_t st) {
    constexpr int STAGES = BITS == 2 ? 4 : 3;
    constexpr size_t SMEM = static_cast<size_t>(MAIN_WARPS) * STAGES * record_bytes(BITS) + MAIN_WARPS * STAGES * 8;
    static_assert(SMEM >= static_cast<size_t>(MAIN_WARPS) * 8 * PART_STRIDE * sizeof(float), "scratch must fit in the staging area");
    decode_prep_kernel<BITS, MODE><<<dim3(P.c.n_kv, P.batch), 128, 0, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
    if (cudaFuncSetAttribute(decode_main_kernel<BITS, MODE, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM)) != cudaSuccess)
        return WUSHKV_ECUDA;
    if (g_prof_start) cudaEventRecord(g_prof_start, st);
    decode_main_kernel<BITS, MODE, STAGES><<<dim3(P.n_chunks + 1, P.c.n_kv, P.batch), MAIN_WARPS * 32, SMEM, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
    if (g_prof_stop) cudaEventRecord(g_prof_stop, st);
    decode_combine_kernel<<<dim3(P.c.n_q, P.batch), 128, 0, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return WUSHKV_ECUDA;
    return WUSHKV_OK;
}

}  // namespace wushkv

using namespace wushkv;

extern "C" size_t wushkv_decode_workspace_bytes(const wushkv_cache* cache, int32_t batch, int32_t max_seq_len) {
    CacheView v;
    if (make_view(cache, v) != WUSHKV_OK) return 0;
    DecodePlan pl;
    if (!make_plan(v, batch, max_seq_len, pl)) return 0;
    return pl.total;
}

extern "C" int wushkv_decode_attn(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                  int32_t max_seq_len, const uint16_t* Q, float* O,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    DecodeParams P;
    const int rc = make_view(cache, P.c);
    if (rc != WUSHKV_OK) return rc;
    if (!slot || !seq_len || !Q || !O || !workspace || !aligned(Q, 16) || !aligned(O, 16) || !aligned(workspace, 256)) return WUSHKV_EINVAL;
    DecodePlan pl;
    if (!make_plan(P.c, batch, max_seq_len, pl)) return WUSHKV_EINVAL;
    if (batch > 65535 || pl.n_chunks + 1 > 0x7fffffff) return WUSHKV_EINVAL;
    if (workspace_bytes < pl.total) return WUSHKV_ECAPACITY;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    P.batch = batch; P.slot = slot; P.seq_len = seq_len; P.Q = Q; P.O = O;
    P.qfrag = reinterpret_cast<uint4*>(ws + pl.off_qfrag);
    P.qscal = reinterpret_cast<float*>(ws + pl.off_qscal);
    P.qcomp = reinterpret_cast<float*>(ws + pl.off_qcomp);
    P.part = reinterpret_cast<float*>(ws + pl.off_part);
    P.n_chunks = pl.n_chunks; P.chunk_pages = pl.chunk_pages;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool mode0 = P.c.G <= 4;
    if (P.c.bits == 2) return mode0 ? launch_decode<2, 0>(P, st) : launch_decode<2, 1>(P, st);
    return mode0 ? launch_decode<4, 0>(P, st) : launch_decode<4, 1>(P, st);
}

extern "C" int wushkv_set_profile_events(void* start, void* stop) {
    if ((start == nullptr) != (stop == nullptr)) return WUSHKV_EINVAL;
    g_prof_start = static_cast<cudaEvent_t>(start);
    g_prof_stop = static_cast<cudaEvent_t>(stop);
    return WUSHKV_OK;
}

extern "C" size_t wushkv_step_staging_bytes(const wushkv_cache* cache, int32_t batch) {
    CacheView v;
    if (make_view(cache, v) != WUSHKV_OK || batch <= 0) return 0;
    const size_t kv = align_up(static_cast<size_t>(batch) * v.n_kv * D * 2, 256);
    const size_t q = align_up(static_cast<size_t>(batch) * v.n_q * D * 2, 256);
    const size_t o = align_up(static_cast<size_t>(batch) * v.n_q * D * 4, 256);
    return 2 * kv + q + o;
}

extern "C" int wushkv_decode_step_host(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                                       const int32_t* cu_new, int32_t max_seq_len,
                                       const uint16_t* K_new_host, const uint16_t* V_new_host, const uint16_t* Q_host,
                                       float* O_host, void* staging, size_t staging_bytes,
                                       void* workspace, size_t workspace_bytes, void* stream) {
    CacheView v;
    const int rc = make_view(cache, v);
    if (rc != WUSHKV_OK) return rc;
    if (batch <= 0 || !K_new_host || !V_new_host || !Q_host || !O_host || !staging || !aligned(staging, 256)) return WUSHKV_EINVAL;
    if (staging_bytes < wushkv_step_staging_bytes(cache, batch)) return WUSHKV_ECAPACITY;
    const size_t kv_bytes = static_cast<size_t>(batch) * v.n_kv * D * 2, kv = align_up(kv_bytes, 256);
    const size_t q_bytes = static_cast<size_t>(batch) * v.n_q * D * 2, q = align_up(q_bytes, 256);
    const size_t o_bytes = static_cast<size_t>(batch) * v.n_q * D * 4;
    unsigned char* sp = static_cast<unsigned char*>(staging);
    uint16_t* dK = reinterpret_cast<uint16_t*>(sp);
    uint16_t* dV = reinterpret_cast<uint16_t*>(sp + kv);
    uint16_t* dQ = reinterpret_cast<uint16_t*>(sp + 2 * kv);
    float* dO = reinterpret_cast<float*>(sp + 2 * kv + q);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(dK, K_new_host, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return WUSHKV_ECUDA;
    if (cudaMemcpyAsync(dV, V_new_host, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return WUSHKV_ECUDA;
    if (cudaMemcpyAsync(dQ, Q_host, q_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return WUSHKV_ECUDA;
    int r = wushkv_append(cache, batch, slot, seq_len, cu_new, batch, 1, dK, dV, stream);
    if (r != WUSHKV_OK) return r;
    r = wushkv_decode_attn(cache, batch, slot, seq_len, max_seq_len, dQ, dO, workspace, workspace_bytes, stream);
    if (r != WUSHKV_OK) return r;
    if (cudaMemcpyAsync(O_host, dO, o_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return WUSHKV_ECUDA;
    return WUSHKV_OK;
}
