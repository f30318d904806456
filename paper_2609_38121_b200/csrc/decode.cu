// Decode attention over the packed cache (Algorithm 2 lines 3 and 5; Eq. 2; Eq. 3; Section 4.4).
//
// Three launches on the caller's stream:
//   1. decode_prep_kernel   q' = T_K^{-T} q per query head (Algorithm 2 line 3), written as mma
//                           B-fragments: for the quantized positions a 16-bit fixed-point copy of q' split
//                           into two signed bytes per channel (the operand of the integer mma), for the
//                           bf16 windows a bf16 value + rounding remainder.  Block (0,0) also writes the
//                           work plan: the prefix sums of work units per sequence.
//   2. decode_main_kernel   ONE wave of CTAs; every WARP owns an equal, contiguous slice of the
//                           flattened list of work units (sequence, KV head, unit), a unit being a
//                           64-token packed page or up to 8 tokens of the bf16 sink / recent windows.
//                           A warp streams its units into shared memory with bulk async copies (mbarrier
//                           ring).  Scores: the packed key codes become unsigned bytes with one AND per four
//                           codes and go through mma.sync.m16n8k32 (u8 x s8, exact 32-bit sums); values:
//                           code words become fp16 A-fragments with one AND per two codes and go through
//                           mma.sync.m16n8k16 with fp32 accumulation.  The affine part of Eq. 6 is factored
//                           out of the contractions:
//                               q'.k_hat = Delta_k (q'.c_k) + x_min_k sum(q'),
//                               o        = sum_s (p_s Delta_v,s) c_v,s + (sum_s p_s x_min_v,s) 1.
//                           Window units use ldmatrix + bf16 mma on the staged rows and fold into the
//                           same accumulators.  Softmax is online (running max / sum) per warp; a warp
//                           writes one partial (max, sum, o) per (sequence, KV head) it touched.
//   3. decode_combine_kernel merges the partials of each (sequence, query head) into O.
//
// No kernel waits on another CTA.  The only waits are on a warp's own copy barriers, bounded by an
// iteration limit after which the kernel records WUSHKV_DEV_COPY_TIMEOUT and drains.
//
// Data that an earlier kernel of the same step may still be writing while a later one is already
// resident (programmatic dependent launch: sequence lengths, plan, query fragments, partials) is read
// with ld.global.cg or plain loads after griddepcontrol.wait, never through the read-only path.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cuda_fp8.h>

#include <algorithm>
#include <cstdlib>

#include "host_common.h"
#include "prologue.cuh"
#include "layout.cuh"

namespace wushkv {

constexpr unsigned FULL = 0xffffffffu;
constexpr int PART_STRIDE = 132;          // floats per partial: [0]=max (log2 domain) [1]=sum [4..131]=o
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LO_SCALE = 2048.f;        // a "remainder" column of a window unit carries (x - rounded(x)) * 2^11
constexpr float Q_MAX = 32512.f;          // largest magnitude of the 16-bit fixed-point query (127 * 256: both digits fit a signed byte)
// Exponentials are taken against (running reference - LOG2_PV): every probability, and with it l, z and
// o of a partial, carries the common factor 2^LOG2_PV, which cancels in the final ratio and keeps
// fp16(p Delta_v) out of the subnormals.  The reference is only raised (and the state rescaled) when
// a unit's maximum exceeds it by more than MAX_SLACK, so p <= 2^(LOG2_PV + MAX_SLACK) and
// p Delta_v stays finite in fp16 for Delta_v < 2^(16 - LOG2_PV - MAX_SLACK) = 1024.
constexpr float LOG2_PV = 3.f;
constexpr float MAX_SLACK = 3.f;
// Warps per CTA of the main kernel.  ONE CTA per SM (16 warps, or 12 where registers or the larger 4-bit records
// limit it) instead of several CTAs of 4: the hardware warp scheduler serves the warps of an older CTA first, so with
// several CTAs per SM equal slices finished up to 15 us apart.
__host__ __device__ constexpr int main_warps(int bits, int mode) { return (bits == 2 && mode == 0) ? 16 : 12; }
constexpr int WIN_TOKENS = 8;             // window tokens per work unit
constexpr int WIN_ROW = 272;              // padded bytes per staged bf16 row (conflict-free ldmatrix)
constexpr int WIN_V_OFF = WIN_TOKENS * WIN_ROW;

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream is still running; it must call pdl_wait() before it
// touches anything the predecessor writes.  Without the attribute both calls are no-ops.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct DecodeParams {
    CacheView c;
    int batch;
    const int* slot;
    const int* seq_len;
    const unsigned short* Q;
    float* O;
    uint4* qfrag;        // [batch*n_kv][256]: s8 B fragments of the 4 k-steps, 2 x 32 uint4 per digit set (MODE 0: one set
                         // whose columns alternate high / low digit; MODE 1: high-digit set, low-digit set)
    uint4* qwfrag;       // [batch*n_kv][2][128]: bf16 B fragments for the windows (MODE 1: value set, remainder set)
    float* qscal;        // [batch][n_q][2]: score multiplier (log2 domain, > 0), x_min multiplier divided by it
    long long* plan;     // [batch+1]: exclusive prefix of work units per sequence (per KV head)
    float* part;         // [n_warps + batch*n_kv][G][PART_STRIDE]
    int n_warps;         // warps of the main kernel
    int wait_limit;      // poll limit of the device-side barrier waits (0: default, about a second)
    long long drop_unit; // testing aid: flattened index of a unit whose copy is never issued (-1: none)
    int q_early;         // 1: Q was final before the kernel ahead of the preparation kernel started
    int stream_pages;    // 1: the packed pages of a step cannot stay in L2 anyway: copy them with an evict-first hint
    Prologue pro;        // pro.rope != nullptr: Q holds projected queries, normalised and rotated by the preparation kernel
};

// shift of the code field used by k-step / channel block idx (0..7) inside its 16-bit lane, after
// the optional whole-word shift: the fp16 value of the masked field is code * 2^(field_shift - 24)
template <int BITS>
__host__ __device__ constexpr int field_shift(int idx) {
    return BITS != 4 ? (idx < 5 ? 2 * idx : 2 * (idx - 5)) : 4 * (idx & 1);     // 3 bits: its 2-bit plane
}
// bf16x2 bit pattern of (2^e, 2^e)
__host__ __device__ constexpr unsigned bf16x2_pow2(int e) {
    return (static_cast<unsigned>(e + 127) << 7) | (static_cast<unsigned>(e + 127) << 23);
}

// How one sequence decomposes into work units (identical for all of its KV heads).
struct SeqInfo {
    int slot;
    int q_lo, q_hi;          // positions read from the packed codes: [q_lo, q_hi)
    int first_page, qp;      // packed pages covering them
    int n_sink, recent_lo;   // window tokens: positions [0, n_sink) and [recent_lo, S)
    int n_win;               // window tokens
    int U;                   // qp + ceil(n_win / WIN_TOKENS)
};

__device__ __forceinline__ SeqInfo seq_info(const CacheView& c, int S, int slot) {
    SeqInfo si;
    si.slot = slot;
    if (S <= 0 || slot < 0 || slot >= c.n_slots) {
        si.q_lo = si.q_hi = 0; si.first_page = si.qp = 0; si.n_sink = si.recent_lo = si.n_win = si.U = 0;
        return si;
    }
    const int nq = n_quantized(S - c.lag, c.s_sink, c.s_keep, c.s_flush);
    si.q_lo = c.s_sink; si.q_hi = c.s_sink + nq;
    si.first_page = si.q_lo / PAGE_TOKENS;
    si.qp = nq > 0 ? (si.q_hi - 1) / PAGE_TOKENS - si.first_page + 1 : 0;
    si.n_sink = min(S, c.s_sink);
    si.recent_lo = c.s_sink + nq;
    si.n_win = si.n_sink + max(0, S - si.recent_lo);
    si.U = si.qp + (si.n_win + WIN_TOKENS - 1) / WIN_TOKENS;
    return si;
}

// ------------------------------------------------------------------------------------------------
// 1. query preparation
// ------------------------------------------------------------------------------------------------
constexpr int PREP_THREADS = 512;                   // 16 warps share the 128 rows of T_K^{-T}
constexpr int PREP_ROWS = D / (PREP_THREADS / 32);   // rows per warp
template <int BITS, int MODE>
__global__ void __launch_bounds__(PREP_THREADS) decode_prep_kernel(DecodeParams P) {
    __shared__ float q_s[8][D];
    __shared__ float red_abs[8][4];
    __shared__ int red_isum[8][4];
    __shared__ long long scan_s[4];
    const int h = blockIdx.x, b = blockIdx.y, G = P.c.G;
    const int i = threadIdx.x, lane = i & 31, warp = i >> 5;
    // Normally everything this kernel reads may come from the kernel ahead of it.  In the fused step
    // (q_early) that kernel is the single-token append, which started only after all earlier work had
    // finished: Q is final already and only the lengths (for the work plan) have to wait for it, so the
    // transform of the queries runs beside the append.  The main kernel reads the lengths and stages
    // pages as soon as it starts, so the plan CTA holds its launch signal back until the append is done.
    const bool plan_cta = h == 0 && b == 0;
    if (!P.q_early) pdl_wait();
    if (!(P.q_early && plan_cta)) pdl_launch_dependents();   // the main kernel may start staging pages while this one runs

    for (int k = i; k < G * D; k += PREP_THREADS)
        q_s[k >> 7][k & (D - 1)] = bf16_bits_to_float(P.Q[(static_cast<long long>(b) * P.c.n_q + h * G) * D + k]);
    __syncthreads();
    if (P.pro.rope) {                     // projected queries: Norm and RoPE at the newest position (Algorithm 2 lines 1-2)
        if (warp < G) {
            const int S = __ldcg(P.seq_len + b);
            float4* qv = reinterpret_cast<float4*>(&q_s[warp][0]) + lane;
            const float4 v = *qv;
            float x[4] = {v.x, v.y, v.z, v.w};
            norm_rope_warp(x, lane, P.pro, h * G + warp, prologue_position(P.pro, max(S - 1, 0), P.c.dev_status, lane == 0 && S > P.pro.n_pos));
            *qv = make_float4(x[0], x[1], x[2], x[3]);
        }
        __syncthreads();
    }
    // q'[g][i] = sum_j T_invT[h][i][j] q[g][j].  Each of the 16 warps takes 8 rows, all of their loads in
    // flight together; a row is one coalesced 512-byte read (lane L holds columns 4L..4L+3); rows are
    // handled 32/GP at a time so that the GP x rows partial sums fit a 32-value transposing butterfly
    // (GP = 4 or 8 head slots).
    __shared__ float qp_s[8][D];
    {
        constexpr int GP = MODE == 0 ? 4 : 8;           // MODE 0 serves G <= 4, MODE 1 serves G <= 8
        constexpr int rows_per = 32 / GP;
        const float4* Tbase = reinterpret_cast<const float4*>(P.c.T_K_invT + (static_cast<long long>(h) * D + warp * PREP_ROWS) * D) + lane;
        float4 qv[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) qv[g] = g < G ? *reinterpret_cast<const float4*>(&q_s[g][4 * lane]) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r0 = 0; r0 < PREP_ROWS; r0 += rows_per) {
            float part[32];
#pragma unroll
            for (int k = 0; k < 32; ++k) part[k] = 0.f;
#pragma unroll
            for (int rr = 0; rr < 32; ++rr) {            // slot k = rr * GP + g for rr < rows_per
                if (rr < rows_per) {
                    const float4 t = __ldg(Tbase + (r0 + rr) * (D / 4));
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (g < GP && rr * GP + g < 32)
                            part[(rr * GP + g) & 31] = fmaf(t.x, qv[g].x, fmaf(t.y, qv[g].y, fmaf(t.z, qv[g].z, t.w * qv[g].w)));
                }
            }
            const float tot = warp_transpose_reduce(part, lane);
            const int rr = lane / GP, g = lane % GP;
            if (g < G) qp_s[g][warp * PREP_ROWS + r0 + rr] = tot;
        }
    }
    __syncthreads();
    if (plan_cta) {                       // work plan: exclusive prefix of units per sequence
        if (P.q_early) { pdl_wait(); pdl_launch_dependents(); }     // the lengths come from the append
        long long carry = 0;
        for (int base = 0; base < P.batch; base += 128) {
            const int bb = base + i;
            long long u = 0;
            if (i < 128 && bb < P.batch) {
                const int slot = __ldg(P.slot + bb);
                if (slot < 0 || slot >= P.c.n_slots) atomicOr(P.c.dev_status, WUSHKV_DEV_BAD_SLOT);
                u = seq_info(P.c, __ldcg(P.seq_len + bb), slot).U;
            }
            long long incl = u;
            for (int o = 1; o < 32; o <<= 1) {
                const long long v = __shfl_up_sync(FULL, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31 && warp < 4) scan_s[warp] = incl;
            __syncthreads();
            long long before = 0;
            for (int w = 0; w < warp && w < 4; ++w) before += scan_s[w];
            if (i < 128 && bb < P.batch) P.plan[bb + 1] = carry + before + incl;
            carry += scan_s[0] + scan_s[1] + scan_s[2] + scan_s[3];
            __syncthreads();
        }
        if (i == 0) P.plan[0] = 0;
    }
    if (i >= 128) return;                 // the fragment stage has one thread per channel
    float acc[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) acc[g] = g < G ? qp_s[g][i] : 0.f;
    const float k2 = P.c.sm_scale * LOG2E;
    // ---- 16-bit fixed point of q' per head: q'[ch] ~ lam * qi[ch], |qi| <= Q_MAX, qi = 256 hi + lo with both
    // digits signed bytes.  The scores of the quantized positions use exactly this rounded query
    // (code part and x_min part alike), so they are the scores of a slightly perturbed query, the same
    // for every position.
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < G) {
            float ab = fabsf(acc[g]);
            for (int o = 16; o > 0; o >>= 1) ab = fmaxf(ab, __shfl_xor_sync(FULL, ab, o));
            if (lane == 0) red_abs[g][warp] = ab;
        }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");       // the four remaining warps only
    int qi[8];
    float lam[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        qi[g] = 0; lam[g] = 1.f;
        if (g < G) {
            const float amax = fmaxf(fmaxf(red_abs[g][0], red_abs[g][1]), fmaxf(red_abs[g][2], red_abs[g][3]));
            if (amax > 0.f && amax < 3e38f) {
                lam[g] = amax * (1.f / Q_MAX);
                qi[g] = max(-static_cast<int>(Q_MAX), min(static_cast<int>(Q_MAX), __float2int_rn(acc[g] * (Q_MAX / amax))));
            }
            int sm = qi[g];
            for (int o = 16; o > 0; o >>= 1) sm += __shfl_xor_sync(FULL, sm, o);
            if (lane == 0) red_isum[g][warp] = sm;
        }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (i < G) {
        const int sum = red_isum[i][0] + red_isum[i][1] + red_isum[i][2] + red_isum[i][3];
        constexpr float FS = BITS != 4 ? 4.f : 16.f;      // the integer score carries this factor (see the main kernel)
        float* qs = P.qscal + (static_cast<long long>(b) * P.c.n_q + h * G + i) * 2;
        qs[0] = k2 * lam[i] * (1.f / FS);                 // score (log2 domain) = qs[0] * (Delta_k * sum_int + x_min_k * qs[1])
        qs[1] = FS * static_cast<float>(sum);
    }
    // ---- B fragments of the integer mma (m16n8k32, B = 32 channels x 8 columns of signed bytes).  Channel i sits in
    // k-step s = i >> 5 at k index 16 hh + 4 t + bb, i.e. register hh, lane 4 n + t, byte bb of column n.
    // MODE 0: column n holds head n >> 1, high digit (n even) or low digit (n odd).  MODE 1: column n holds
    // head n; the high digits form the first fragment set, the low digits the second.
    const int s = i >> 5, hh = (i >> 4) & 1, bb = 2 * ((i >> 3) & 1) + (i & 1), t = (i >> 1) & 3;
    const long long bh = static_cast<long long>(b) * P.c.n_kv + h;
    signed char* frag = reinterpret_cast<signed char*>(P.qfrag + bh * 256);
#pragma unroll
    for (int n = 0; n < 8; ++n) {
        const int head = (MODE == 0) ? (n >> 1) : n;
        const int v = head < G ? qi[head] : 0;
        const int hi = (v + 128) >> 8, lo = v - 256 * hi;          // hi in [-127, 127], lo in [-128, 127]
        const int off = (((s >> 1) * 32 + 4 * n + t) * 16) + ((s & 1) * 2 + hh) * 4 + bb;
        if (MODE == 0) {
            frag[off] = static_cast<signed char>((n & 1) ? lo : hi);
        } else {
            frag[off] = static_cast<signed char>(hi);
            frag[1024 + off] = static_cast<signed char>(lo);
        }
    }
    // ---- bf16 B fragments for the windows (mma.m16n8k16).  Element (k-step s16, register r, lane 4n+t, half hf) is
    // channel 16 s16 + 8 r + 2 t + hf of mma column n.  MODE 0: column n holds head n>>1, its rounded value (n even)
    // or the rounding remainder (n odd).  MODE 1: column n holds head n; a second copy holds the remainders.
    const int s16 = i >> 4, r16 = i & 15, r = r16 >> 3, tw = (r16 & 7) >> 1, hf = r16 & 1;
    unsigned short* wfrag = reinterpret_cast<unsigned short*>(P.qwfrag + bh * 256);
#pragma unroll
    for (int n = 0; n < 8; ++n) {
        const int head = (MODE == 0) ? (n >> 1) : n;
        float wval = 0.f, wrem = 0.f;
        if (head < G) {
            const float y = acc[head] * k2;
            const float yh = __bfloat162float(__float2bfloat16_rn(y));
            wrem = y - yh;
            wval = (MODE == 0 && (n & 1)) ? wrem : y;
        }
        const int idx = ((((s16 >> 1) * 32 + 4 * n + tw) * 4 + (s16 & 1) * 2 + r) << 1) + hf;
        wfrag[idx] = __bfloat16_as_ushort(__float2bfloat16_rn(wval));
        if (MODE == 1) wfrag[1024 + idx] = __bfloat16_as_ushort(__float2bfloat16_rn(wrem));
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(2000u) : "memory");      // may sleep up to ~2 us in hardware
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the limit (about a second of sleeping polls).
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, int limit) {
    for (int it = 0; it < limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ void bulk_copy_g2s(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// The same copy for data that is read once per step (packed pages): evict-first in L2, so that the
// stream does not push out what the step's other kernels re-read (transforms, fragments, partials).
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_copy_g2s_stream(unsigned dst, const void* src, unsigned bytes, unsigned bar, unsigned long long pol) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ uint2 lds64(unsigned addr) {
    uint2 v;
    asm("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds128(unsigned addr) {
    uint4 v;
    asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void ldmatrix_x4(unsigned addr, unsigned& a, unsigned& b, unsigned& c, unsigned& d) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned addr, unsigned& a, unsigned& b, unsigned& c, unsigned& d) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// first MMA of a chain: D = A B (no accumulator registers to initialise)
__device__ __forceinline__ void mma_f16_zero(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
// integer mma: A = 16 x 32 unsigned bytes (codes), B = 32 x 8 signed bytes (query digits), exact 32-bit sums
__device__ __forceinline__ void mma_u8s8(int (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8s8_zero(int (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned movmatrix_trans(unsigned a) {
    unsigned d;
    asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ unsigned pack_h2(float lo, float hi) {      // lo -> bits 0..15, hi -> bits 16..31, saturating
    unsigned d;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ unsigned pack_bf2(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ unsigned mul_bf2(unsigned a, unsigned b) {
    unsigned d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float ex2(float x) {      // 2^x, -inf -> 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float2 h2f2(unsigned u) {     // both halves of an fp16x2 register as floats
    __half2 h;
    *reinterpret_cast<unsigned*>(&h) = u;
    return __half22float2(h);
}
__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Field idx (0..7) of a code word as an fp16x2 A-fragment register.  `w` is the raw word, `ws` the
// same word shifted right so that the upper fields fall into the low bits of each 16-bit lane.
template <int BITS>
__device__ __forceinline__ unsigned field(unsigned w, unsigned ws, int idx) {
    if (BITS != 4) {
        constexpr unsigned M0 = 0x00030003u;
        return idx < 5 ? (w & (M0 << (2 * idx))) : (ws & (M0 << (2 * (idx - 5))));
    } else {
        constexpr unsigned M0 = 0x000F000Fu;
        return idx < 2 ? (w & (M0 << (4 * idx))) : (ws & (M0 << (4 * (idx - 2))));
    }
}
template <int BITS> __device__ __forceinline__ unsigned pre_shift(unsigned w) { return BITS != 4 ? (w >> 10) : (w >> 8); }

// Per-warp running softmax state of one (sequence, KV head).  MODE 0: one head per thread (head t,
// value and rounding-remainder columns).  MODE 1: two heads per thread (2t, 2t+1).
// o[i][.] accumulates channel block i in units of 2^(field_shift(i) - 24); l, z and o carry the
// common factor 2^LOG2_PV.  m is the reference of the partial, not necessarily its exact maximum.
template <int MODE>
struct WarpState {
    static constexpr int NH = MODE == 0 ? 1 : 2;
    float m[NH], mr[NH], l[NH], z[NH];
    float o[8][4];
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int k = 0; k < NH; ++k) { m[k] = -INFINITY; mr[k] = 0.f; l[k] = 0.f; z[k] = 0.f; }
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    }
    // Make the running reference cover this unit's maxima to within MAX_SLACK.  mx holds each lane's
    // maximum over its own tokens; the warp-wide reduction is only needed when some lane is past the
    // slack, which after the first unit of a slice is rare.  mr is what the exponentials subtract.
    __device__ __forceinline__ void raise_max(float (&mx)[NH]) {
        bool grew = false;
#pragma unroll
        for (int k = 0; k < NH; ++k) grew |= mx[k] > m[k] + MAX_SLACK;      // reference -inf: any finite score
        if (__any_sync(FULL, grew)) {
            float scl[NH];
#pragma unroll
            for (int k = 0; k < NH; ++k) {
                mx[k] = fmaxf(mx[k], __shfl_xor_sync(FULL, mx[k], 4));       // over the 8 token rows of the fragment
                mx[k] = fmaxf(mx[k], __shfl_xor_sync(FULL, mx[k], 8));
                mx[k] = fmaxf(mx[k], __shfl_xor_sync(FULL, mx[k], 16));
                const float mnew = fmaxf(m[k], mx[k]);
                const float ref = (mnew == -INFINITY) ? 0.f : mnew;          // all masked so far: any finite reference works
                scl[k] = ex2(m[k] - ref);                                    // old reference -inf: state is all zero, factor 0
                l[k] *= scl[k]; z[k] *= scl[k];
                m[k] = mnew;
                mr[k] = ref - LOG2_PV;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                o[i][0] *= scl[0]; o[i][2] *= scl[0];
                o[i][1] *= scl[NH - 1]; o[i][3] *= scl[NH - 1];
            }
        }
    }
};

// Writes this warp's partial (max, sum, o[128]) of every head of one (sequence, KV head) to global memory.
template <int BITS, int MODE>
__device__ __forceinline__ void store_partial(const WarpState<MODE>& st, float* dst0, int lane, int G) {
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
            float* dst = dst0 + head * PART_STRIDE;
            if (g == 0) { dst[0] = st.m[k]; dst[1] = l; }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float osc = exp2f(static_cast<float>(24 - field_shift<BITS>(i)));
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

// One window unit: up to 8 bf16 tokens staged at shared-memory address rec (key rows, then value rows at
// WIN_V_OFF, WIN_ROW bytes apart); wsrc points at the (sequence, KV head)'s bf16 query fragments.
template <int BITS, int MODE>
__device__ __forceinline__ void window_unit(WarpState<MODE>& st, unsigned rec, int n_valid, const uint4* wsrc, int lane) {
    constexpr int NH = WarpState<MODE>::NH;
    const int g = lane >> 2;
    const int r_eff = (lane & 7) < n_valid ? (lane & 7) : 0;      // rows beyond the valid ones alias row 0
    const int mat = lane >> 3;
    const unsigned frag_off = r_eff * WIN_ROW + ((mat >> 1) * 16 + (mat & 1) * 8) * 2;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int pass = 0; pass < (MODE == 0 ? 1 : 2); ++pass) {
#pragma unroll
        for (int s2 = 0; s2 < 4; ++s2) {
            const uint4 bq = __ldcg(wsrc + pass * 128 + s2 * 32 + lane);
            unsigned k0, k1, k2, k3;                      // (step 2s2: ch lo, ch hi), (step 2s2+1: ch lo, ch hi)
            ldmatrix_x4(rec + frag_off + s2 * 64, k0, k1, k2, k3);
            mma_bf16(acc, k0, k0, k1, k1, bq.x, bq.y);    // token rows 8..15 alias rows 0..7
            mma_bf16(acc, k2, k2, k3, k3, bq.z, bq.w);
        }
    }
    const bool ok = g < n_valid;
    float sc[NH], mx[NH];
    if (MODE == 0) sc[0] = ok ? acc[0] + acc[1] : -INFINITY;
    else { sc[0] = ok ? acc[0] : -INFINITY; sc[NH - 1] = ok ? acc[1] : -INFINITY; }
#pragma unroll
    for (int k = 0; k < NH; ++k) mx[k] = sc[k];
    st.raise_max(mx);
    float p[NH];
#pragma unroll
    for (int k = 0; k < NH; ++k) { p[k] = ex2(sc[k] - st.mr[k]); st.l[k] += p[k]; }
#pragma unroll
    for (int pass = 0; pass < (MODE == 0 ? 1 : 2); ++pass) {
        unsigned pr;                                      // this token's probabilities in the score-fragment layout
        if (MODE == 0) pr = pack_bf2(p[0], (p[0] - bf16_round(p[0])) * LO_SCALE);   // value column, remainder column
        else if (pass == 0) pr = pack_bf2(p[0], p[NH - 1]);
        else pr = pack_bf2(p[0] - bf16_round(p[0]), p[NH - 1] - bf16_round(p[NH - 1]));
        const unsigned b01 = movmatrix_trans(pr);         // tokens 2t, 2t+1 of column g; tokens 8..15 get zero
#pragma unroll
        for (int i2 = 0; i2 < 4; ++i2) {
            unsigned v0, v1, v2, v3;                      // (block 2i2: ch lo, ch hi), (block 2i2+1: ch lo, ch hi)
            ldmatrix_x4_trans(rec + WIN_V_OFF + frag_off + i2 * 64, v0, v1, v2, v3);
            // fold the block's accumulator unit in: p * v * 2^(shift - 24)
            mma_bf16(st.o[2 * i2], v0, v1, v0, v1, mul_bf2(b01, bf16x2_pow2(field_shift<BITS>(2 * i2) - 24)), 0u);
            mma_bf16(st.o[2 * i2 + 1], v2, v3, v2, v3, mul_bf2(b01, bf16x2_pow2(field_shift<BITS>(2 * i2 + 1) - 24)), 0u);
        }
    }
}

// One (sequence, KV head) stretch of a warp's slice, kept in shared memory.  Units [u0, u1) of the
// head's unit list: units below qp are packed pages (page index first_page + u), the rest are window
// units of WIN_TOKENS tokens.
struct Segment {
    int b, h, slot, u0, u1, qp, first_page, q_lo, q_hi, n_win, n_sink, recent_lo;
};
constexpr int MAX_SEGMENTS = 6;           // per warp and round; more segments take further rounds

// ------------------------------------------------------------------------------------------------
// main kernel
// ------------------------------------------------------------------------------------------------
#ifndef WUSHKV_ABL
#define WUSHKV_ABL 0        // timing experiments only: 1 no value contraction, 2 no key contraction, 8 no page copies, 16 per-warp time stamps
#endif
#if WUSHKV_ABL & 16
__device__ unsigned long long g_timeline[8192 * 4];
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define TL(slot) do { if (lane == 0) g_timeline[((blockIdx.x * 16 + warp) & 8191) * 4 + (slot)] = gtime(); } while (0)
#else
#define TL(slot) do { } while (0)
#endif

template <int BITS, int MODE, int STAGES>
__global__ void __launch_bounds__(main_warps(BITS, MODE) * 32, 1) decode_main_kernel(DecodeParams P) {
    constexpr int MAIN_WARPS = main_warps(BITS, MODE);
    constexpr int REC = record_bytes(BITS);
    constexpr int CB = code_block_bytes(BITS);
    constexpr int NH = WarpState<MODE>::NH;
    static_assert(2 * WIN_TOKENS * WIN_ROW <= REC, "a window unit must fit in one stage");
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + MAIN_WARPS * STAGES * REC);
    Segment* seg_all = reinterpret_cast<Segment*>(smem + MAIN_WARPS * STAGES * REC + MAIN_WARPS * STAGES * 8);
    const CacheView& c = P.c;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = c.G;
    Segment* segs = seg_all + warp * MAX_SEGMENTS;
    TL(0);

    // ---- work plan: prefix sums of units per sequence.  Recomputed here from the inputs (into the still
    // unused staging area) so that nothing the preparation kernel writes is needed before the first copies.
    __shared__ long long scan_s[MAIN_WARPS];
    long long* plan_s = reinterpret_cast<long long*>(smem);
    const bool local_plan = (static_cast<size_t>(P.batch) + 1) * sizeof(long long) <= static_cast<size_t>(MAIN_WARPS) * STAGES * REC;
    if (local_plan) {
        long long carry = 0;
        for (int base = 0; base < P.batch; base += MAIN_WARPS * 32) {
            const int bb = base + threadIdx.x;
            long long incl = 0;
            if (bb < P.batch) incl = seq_info(c, __ldcg(P.seq_len + bb), __ldg(P.slot + bb)).U;
            for (int o = 1; o < 32; o <<= 1) {
                const long long v = __shfl_up_sync(FULL, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31) scan_s[warp] = incl;
            __syncthreads();
            long long before = 0, all = 0;
            for (int w = 0; w < MAIN_WARPS; ++w) { if (w < warp) before += scan_s[w]; all += scan_s[w]; }
            if (bb < P.batch) plan_s[bb + 1] = carry + before + incl;
            carry += all;
            __syncthreads();
        }
        if (threadIdx.x == 0) plan_s[0] = 0;
        __syncthreads();
    } else {
        pdl_wait();
    }
    const long long* plan = local_plan ? plan_s : P.plan;

    // ---- this warp's slice of the flattened unit list
    const long long total = plan[P.batch] * c.n_kv;
    const long long wg = static_cast<long long>(blockIdx.x) * MAIN_WARPS + warp;
    long long L = total > 0 ? wg * total / P.n_warps : 0;
    const long long L1 = total > 0 ? (wg + 1) * total / P.n_warps : 0;

    // position of the slice start: sequence b, head h, unit u
    int sb = 0, sh = 0, su = 0;
    if (L < L1) {
        int lo = 0, hi = P.batch;           // largest b with n_kv * plan[b] <= L
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (plan[mid] * c.n_kv <= L) lo = mid; else hi = mid;
        }
        sb = lo;
        const long long U = max(plan[lo + 1] - plan[lo], 1LL);
        const long long rem = L - plan[lo] * c.n_kv;
        sh = static_cast<int>(rem / U);
        su = static_cast<int>(rem % U);
    }
    __syncthreads();                        // the staging area stops being plan scratch here
    pdl_launch_dependents();
    if (L >= L1) return;

    // ---- barriers
    const unsigned bar0 = smem_u32(bars + warp * STAGES);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const unsigned stage0 = smem_u32(smem + warp * STAGES * REC);
    const long long page_row_bytes = static_cast<long long>(c.n_kv) * REC;
    const unsigned long long stream_policy = l2_evict_first_policy();

    if (WUSHKV_ABL & 8) { for (int k = lane; k < STAGES * REC / 4; k += 32) reinterpret_cast<unsigned*>(smem + warp * STAGES * REC)[k] = 0u; __syncwarp(); }
    unsigned qf[4][2];                  // integer B fragments of the four k-steps (MODE 1: the high digits)
    unsigned qfl[MODE == 1 ? 4 : 1][2]; // MODE 1: the low digits
    float fmul[NH], gadd[NH];
    WarpState<MODE> st;
    int stage = 0;                      // ring position of the next unit to consume (and to refill)
    unsigned phase_bits = 0;            // parity of each stage's next completion
    unsigned bad_bits = 0;              // lane 0: stages whose unit could not be fetched
    bool timed_out = false;
    const int wait_limit = P.wait_limit > 0 ? P.wait_limit : (1 << 19);      // polls that may sleep ~2 us each: about a second

    while (L < L1 && !timed_out) {
        // ================= round set-up: list the next segments of the slice =====================
        int n_seg = 0, round_units = 0;
        while (n_seg < MAX_SEGMENTS && L < L1) {
            const SeqInfo si = seq_info(c, __ldcg(P.seq_len + sb), __ldg(P.slot + sb));
            if (si.U > 0) {
                const int u1 = static_cast<int>(min(static_cast<long long>(si.U), su + (L1 - L)));
                if (lane == 0) {
                    Segment sg;
                    sg.b = sb; sg.h = sh; sg.slot = si.slot; sg.u0 = su; sg.u1 = u1; sg.qp = si.qp; sg.first_page = si.first_page;
                    sg.q_lo = si.q_lo; sg.q_hi = si.q_hi; sg.n_win = si.n_win; sg.n_sink = si.n_sink; sg.recent_lo = si.recent_lo;
                    segs[n_seg] = sg;
                }
                ++n_seg;
                round_units += u1 - su;
                L += u1 - su;
                su = u1;
            }
            if (si.U == 0 || su >= si.U) {              // next head, or next sequence
                su = 0;
                if (si.U == 0 || ++sh >= c.n_kv) { sh = 0; ++sb; }
                if (sb >= P.batch) break;
            }
        }
        __syncwarp();

        // ================= producer: stages the units of this round, in order =====================
        const long long round_L0 = L - round_units;      // flattened index of the round's first unit
        int p_seg = -1, p_u = 0, p_u1 = 0, p_qp = 0, p_head_off = 0, issued = 0;
        const int* p_ptab = nullptr;
        auto issue_next = [&](const int s) {            // whole warp; stages the round's next unit into ring slot s
            if (p_u == p_u1) {                          // next segment
                ++p_seg;
                const Segment& sg = segs[p_seg];
                p_u = sg.u0; p_u1 = sg.u1; p_qp = sg.qp; p_head_off = sg.h * REC;
                p_ptab = c.page_table + static_cast<long long>(sg.slot) * c.max_pages + sg.first_page;
                if (sg.first_page + sg.qp > c.max_pages) {      // the page table cannot hold this length
                    if (lane == 0) atomicOr(c.dev_status, WUSHKV_DEV_PAGE_TABLE_FULL);
                    p_qp = min(p_qp, max(c.max_pages - sg.first_page, 0));   // pages beyond it are treated as window-less gaps below
                }
            }
            const unsigned bar = bar0 + 8 * s, dst = stage0 + s * REC;
            const Segment& sg = segs[p_seg];
            if (p_u < sg.qp) {                          // a packed page: one bulk copy
                if (lane == 0) {
                    const int page = (p_u < p_qp) ? __ldg(p_ptab + p_u) : -1;
                    if (static_cast<unsigned>(page) >= static_cast<unsigned long long>(c.n_pages)) {
                        if (p_u < p_qp) atomicOr(c.dev_status, WUSHKV_DEV_BAD_PAGE_ID);
                        bad_bits |= 1u << s;
                        mbar_arrive(bar);
                    } else if (WUSHKV_ABL & 8) {        // timing experiment: no copy, the stage keeps its (zeroed) content
                        bad_bits &= ~(1u << s);
                        mbar_arrive(bar);
                    } else {
                        bad_bits &= ~(1u << s);
                        mbar_expect_tx(bar, REC);
                        if (P.drop_unit >= 0 && P.drop_unit == round_L0 + issued) {
                            // testing aid: the copy is announced but never issued, so the wait for it runs into its limit
                        } else if (P.stream_pages) bulk_copy_g2s_stream(dst, c.pages + page * page_row_bytes + p_head_off, REC, bar, stream_policy);
                        else bulk_copy_g2s(dst, c.pages + page * page_row_bytes + p_head_off, REC, bar);
                    }
                }
            } else {                                    // up to 8 window tokens: one 256-byte row copy per lane
                const int w0 = (p_u - sg.qp) * WIN_TOKENS;
                const int n_valid = min(WIN_TOKENS, sg.n_win - w0);
                if (lane == 0) { bad_bits &= ~(1u << s); mbar_expect_tx(bar, n_valid * 2 * D * 2); }
                __syncwarp();
                const int r = lane & 7, which = lane >> 3;      // lanes 0-7: key rows, 8-15: value rows
                if (lane < 16 && r < n_valid) {
                    const int w = w0 + r;
                    const long long plane = (static_cast<long long>(sg.slot) * c.n_kv + sg.h) * 2 + which;
                    const unsigned short* src;
                    if (w < sg.n_sink) src = c.sink_kv + (plane * c.s_sink + w) * D;
                    else src = c.ring_kv + (plane * c.ring_cap + (sg.recent_lo + (w - sg.n_sink)) % c.ring_cap) * D;
                    bulk_copy_g2s(dst + which * WIN_V_OFF + r * WIN_ROW, src, D * 2, bar);
                }
            }
            ++p_u;
            ++issued;
        };
        for (int k = 0; k < STAGES && k < round_units; ++k) issue_next((stage + k) % STAGES);
        TL(1);

        // ================= consumer ==============================================================
        pdl_wait();                                     // query fragments come from the preparation kernel
        for (int cs = 0; cs < n_seg && !timed_out; ++cs) {
            const Segment& sg = segs[cs];               // rarely used fields are re-read from shared memory
            const long long bh = static_cast<long long>(sg.b) * c.n_kv + sg.h;
            const int u1 = sg.u1, qp = sg.qp, q_lo = sg.q_lo, q_hi = sg.q_hi;
            int pos0 = (sg.first_page + sg.u0) * PAGE_TOKENS;
            {   // query fragments and per-head scalars of this (sequence, KV head)
                const uint4* src = P.qfrag + bh * 256;
#pragma unroll
                for (int s2 = 0; s2 < 2; ++s2) {
                    const uint4 v = __ldcg(src + s2 * 32 + lane);
                    qf[2 * s2][0] = v.x; qf[2 * s2][1] = v.y; qf[2 * s2 + 1][0] = v.z; qf[2 * s2 + 1][1] = v.w;
                    if (MODE == 1) {
                        const uint4 w = __ldcg(src + 64 + s2 * 32 + lane);
                        qfl[2 * s2][0] = w.x; qfl[2 * s2][1] = w.y; qfl[2 * s2 + 1][0] = w.z; qfl[2 * s2 + 1][1] = w.w;
                    }
                }
#pragma unroll
                for (int k = 0; k < NH; ++k) {
                    const int head = MODE == 0 ? t : 2 * t + k;
                    fmul[k] = 1.f; gadd[k] = 0.f;             // unused head slots stay finite
                    if (head < G) {
                        const float2 v = __ldcg(reinterpret_cast<const float2*>(P.qscal + (static_cast<long long>(sg.b) * c.n_q + sg.h * G + head) * 2));
                        fmul[k] = v.x; gadd[k] = v.y;
                    }
                }
                st.reset();
            }
            for (int u = sg.u0; u < u1; ++u, pos0 += PAGE_TOKENS) {
                const int s = stage;
                // a phase that one lane saw complete is complete for all: keep the decision warp-uniform
                if (!__any_sync(FULL, mbar_wait_bounded(bar0 + 8 * s, (phase_bits >> s) & 1u, wait_limit))) { timed_out = true; break; }
                phase_bits ^= 1u << s;
#if WUSHKV_ABL & 16
                if (lane == 0 && g_timeline[((blockIdx.x * 16 + warp) & 8191) * 4 + 2] == 0) g_timeline[((blockIdx.x * 16 + warp) & 8191) * 4 + 2] = gtime();
#endif
                const unsigned rec = stage0 + s * REC;
                if (u >= qp) {
                    // ======================= window unit: up to 8 bf16 tokens ==========================
                    const int w0 = (u - qp) * WIN_TOKENS;
                    window_unit<BITS, MODE>(st, rec, min(WIN_TOKENS, sg.n_win - w0),
                                            P.qwfrag + (static_cast<long long>(sg.b) * c.n_kv + sg.h) * 256, lane);
                } else if (!__any_sync(FULL, (bad_bits >> s) & 1u)) {
                    // ======================= packed page: 64 quantized tokens ==========================
                    const bool full_page = (pos0 >= q_lo) && (pos0 + PAGE_TOKENS <= q_hi);
                    float sc[4][2 * NH];          // [block][row g: heads..., row g+8: heads...]
                    unsigned vmeta[4][2];         // fp16x2 (Delta_v, x_min_v) of rows g, g+8
#pragma unroll
                    for (int bi = 0; bi < 4; ++bi) {
                        // The four k-steps of a block take one field of every code byte each.  Fields at an even
                        // position come out of the mask as the code itself, fields at an odd position as the code
                        // times FS (4 at 2 bits, 16 at 4 bits): the two kinds are summed separately (X, Y) and
                        // joined as FS * X + Y, which is FS times the exact integer dot product.
                        constexpr int FS = BITS != 4 ? 4 : 16;
                        unsigned a[4][4];             // [k-step][A register]
                        if (BITS != 4) {
                            const uint4 kw = lds128(rec + bi * CB + 16 * lane);      // (row g, ch half 0), (g+8, 0), (g, 1), (g+8, 1)
                            const unsigned sx = kw.x >> 4, sy = kw.y >> 4, sz = kw.z >> 4, sw = kw.w >> 4;
                            a[0][0] = kw.x & 0x03030303u; a[0][1] = kw.y & 0x03030303u; a[0][2] = kw.z & 0x03030303u; a[0][3] = kw.w & 0x03030303u;
                            a[1][0] = kw.x & 0x0C0C0C0Cu; a[1][1] = kw.y & 0x0C0C0C0Cu; a[1][2] = kw.z & 0x0C0C0C0Cu; a[1][3] = kw.w & 0x0C0C0C0Cu;
                            a[2][0] = sx & 0x03030303u;   a[2][1] = sy & 0x03030303u;   a[2][2] = sz & 0x03030303u;   a[2][3] = sw & 0x03030303u;
                            a[3][0] = sx & 0x0C0C0C0Cu;   a[3][1] = sy & 0x0C0C0C0Cu;   a[3][2] = sz & 0x0C0C0C0Cu;   a[3][3] = sw & 0x0C0C0C0Cu;
                        } else {
                            const uint4 ka = lds128(rec + bi * CB + 16 * lane);          // k-steps 0 (low nibbles), 1 (high nibbles)
                            const uint4 kb = lds128(rec + bi * CB + 512 + 16 * lane);    // k-steps 2, 3
                            a[0][0] = ka.x & 0x0F0F0F0Fu; a[0][1] = ka.y & 0x0F0F0F0Fu; a[0][2] = ka.z & 0x0F0F0F0Fu; a[0][3] = ka.w & 0x0F0F0F0Fu;
                            a[1][0] = ka.x & 0xF0F0F0F0u; a[1][1] = ka.y & 0xF0F0F0F0u; a[1][2] = ka.z & 0xF0F0F0F0u; a[1][3] = ka.w & 0xF0F0F0F0u;
                            a[2][0] = kb.x & 0x0F0F0F0Fu; a[2][1] = kb.y & 0x0F0F0F0Fu; a[2][2] = kb.z & 0x0F0F0F0Fu; a[2][3] = kb.w & 0x0F0F0F0Fu;
                            a[3][0] = kb.x & 0xF0F0F0F0u; a[3][1] = kb.y & 0xF0F0F0F0u; a[3][2] = kb.z & 0xF0F0F0F0u; a[3][3] = kb.w & 0xF0F0F0F0u;
                        }
                        int dot[4];                   // MODE 0: (row g, row g+8) x (high, low digit) joined below; MODE 1: rows x heads 2t, 2t+1
                        if (WUSHKV_ABL & 2) { dot[0] = a[0][0] & 1; dot[1] = a[0][1] & 1; dot[2] = a[0][2] & 1; dot[3] = a[0][3] & 1; } else
                        {
                            int X[4], Y[4];
                            mma_u8s8_zero(X, a[0][0], a[0][1], a[0][2], a[0][3], qf[0][0], qf[0][1]);
                            mma_u8s8_zero(Y, a[1][0], a[1][1], a[1][2], a[1][3], qf[1][0], qf[1][1]);
                            mma_u8s8(X, a[2][0], a[2][1], a[2][2], a[2][3], qf[2][0], qf[2][1]);
                            mma_u8s8(Y, a[3][0], a[3][1], a[3][2], a[3][3], qf[3][0], qf[3][1]);
#pragma unroll
                            for (int e = 0; e < 4; ++e) dot[e] = X[e] * FS + Y[e];
                        }
                        unsigned ah[4][4];            // 3 bits: A registers of the 1-bit plane (codes' high bits), one shift + mask each
                        if (BITS == 3 && !(WUSHKV_ABL & 2)) {
                            const uint2 kh = lds64(rec + k_hi_offset(3) + bi * 256 + 8 * lane);      // words of token rows g, g+8
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                ah[ks][0] = (kh.x >> (2 * ks)) & 0x01010101u;     ah[ks][1] = (kh.y >> (2 * ks)) & 0x01010101u;
                                ah[ks][2] = (kh.x >> (2 * ks + 1)) & 0x01010101u; ah[ks][3] = (kh.y >> (2 * ks + 1)) & 0x01010101u;
                            }
                            int Z[4];
                            mma_u8s8_zero(Z, ah[0][0], ah[0][1], ah[0][2], ah[0][3], qf[0][0], qf[0][1]);
#pragma unroll
                            for (int ks = 1; ks < 4; ++ks) mma_u8s8(Z, ah[ks][0], ah[ks][1], ah[ks][2], ah[ks][3], qf[ks][0], qf[ks][1]);
#pragma unroll
                            for (int e = 0; e < 4; ++e) dot[e] += 4 * FS * Z[e];       // code = low plane + 4 x high bit
                        }
                        if (MODE == 1 && !(WUSHKV_ABL & 2)) {              // second fragment set: the low digits of the eight heads
                            int X[4], Y[4];
                            mma_u8s8_zero(X, a[0][0], a[0][1], a[0][2], a[0][3], qfl[0][0], qfl[0][1]);
                            mma_u8s8_zero(Y, a[1][0], a[1][1], a[1][2], a[1][3], qfl[1][0], qfl[1][1]);
                            mma_u8s8(X, a[2][0], a[2][1], a[2][2], a[2][3], qfl[2][0], qfl[2][1]);
                            mma_u8s8(Y, a[3][0], a[3][1], a[3][2], a[3][3], qfl[3][0], qfl[3][1]);
                            if (BITS == 3) {
                                int Z[4];
                                mma_u8s8_zero(Z, ah[0][0], ah[0][1], ah[0][2], ah[0][3], qfl[0][0], qfl[0][1]);
#pragma unroll
                                for (int ks = 1; ks < 4; ++ks) mma_u8s8(Z, ah[ks][0], ah[ks][1], ah[ks][2], ah[ks][3], qfl[ks][0], qfl[ks][1]);
#pragma unroll
                                for (int e = 0; e < 4; ++e) Y[e] += 4 * FS * Z[e];
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) dot[e] = dot[e] * 256 + (X[e] * FS + Y[e]);
                        }
                        const uint4 mt = lds128(rec + meta_offset(BITS) + 128 * bi + 16 * g);   // rows g (x,y) and g+8 (z,w)
                        const float2 km_a = h2f2(mt.x), km_b = h2f2(mt.z);
                        const float kd0 = km_a.x, km0 = km_a.y, kd1 = km_b.x, km1 = km_b.y;
                        vmeta[bi][0] = mt.y; vmeta[bi][1] = mt.w;
                        if (MODE == 0) {
                            const float d0 = static_cast<float>(dot[0] * 256 + dot[1]), d1 = static_cast<float>(dot[2] * 256 + dot[3]);
                            sc[bi][0] = fmaf(km0, gadd[0], d0 * kd0);
                            sc[bi][NH] = fmaf(km1, gadd[0], d1 * kd1);
                        } else {
                            sc[bi][0] = fmaf(km0, gadd[0], static_cast<float>(dot[0]) * kd0);
                            sc[bi][NH - 1] = fmaf(km0, gadd[NH - 1], static_cast<float>(dot[1]) * kd0);
                            sc[bi][NH] = fmaf(km1, gadd[0], static_cast<float>(dot[2]) * kd1);
                            sc[bi][2 * NH - 1] = fmaf(km1, gadd[NH - 1], static_cast<float>(dot[3]) * kd1);
                        }
                    }
                    if (!full_page) {             // first / last page of the quantized range: mask the tokens outside it
#pragma unroll
                        for (int bi = 0; bi < 4; ++bi) {
                            const int p0 = pos0 + bi * 16 + g, p1 = p0 + 8;
                            if (p0 < q_lo || p0 >= q_hi) {
                                vmeta[bi][0] = 0u;
#pragma unroll
                                for (int k = 0; k < NH; ++k) sc[bi][k] = -INFINITY;
                            }
                            if (p1 < q_lo || p1 >= q_hi) {
                                vmeta[bi][1] = 0u;
#pragma unroll
                                for (int k = 0; k < NH; ++k) sc[bi][NH + k] = -INFINITY;
                            }
                        }
                    }
                    // ---------------- running maximum of the page, rescale if it grew
                    float mx[NH];
#pragma unroll
                    for (int k = 0; k < NH; ++k) {
                        const float v = fmaxf(fmaxf(fmaxf(sc[0][k], sc[0][NH + k]), fmaxf(sc[1][k], sc[1][NH + k])),
                                              fmaxf(fmaxf(sc[2][k], sc[2][NH + k]), fmaxf(sc[3][k], sc[3][NH + k])));
                        mx[k] = v * fmul[k];          // scores are kept divided by the head's multiplier (> 0)
                    }
                    st.raise_max(mx);
                    // ---------------- probabilities, value reduction
#pragma unroll
                    for (int bi = 0; bi < 4; ++bi) {
                        const float2 vm_a = h2f2(vmeta[bi][0]), vm_b = h2f2(vmeta[bi][1]);
                        const float vd0 = vm_a.x, vn0 = vm_a.y, vd1 = vm_b.x, vn1 = vm_b.y;
                        unsigned r0, r1;
                        if (MODE == 0) {
                            const float p0 = ex2(fmaf(sc[bi][0], fmul[0], -st.mr[0])), p1 = ex2(fmaf(sc[bi][NH], fmul[0], -st.mr[0]));
                            st.l[0] += p0 + p1;
                            st.z[0] = fmaf(p0, vn0, fmaf(p1, vn1, st.z[0]));
                            r0 = pack_h2(p0 * vd0, 0.f);
                            r1 = pack_h2(p1 * vd1, 0.f);
                        } else {
                            const float p00 = ex2(fmaf(sc[bi][0], fmul[0], -st.mr[0])), p01 = ex2(fmaf(sc[bi][NH - 1], fmul[NH - 1], -st.mr[NH - 1]));
                            const float p10 = ex2(fmaf(sc[bi][NH], fmul[0], -st.mr[0])), p11 = ex2(fmaf(sc[bi][2 * NH - 1], fmul[NH - 1], -st.mr[NH - 1]));
                            st.l[0] += p00 + p10; st.l[NH - 1] += p01 + p11;
                            st.z[0] = fmaf(p00, vn0, fmaf(p10, vn1, st.z[0]));
                            st.z[NH - 1] = fmaf(p01, vn0, fmaf(p11, vn1, st.z[NH - 1]));
                            r0 = pack_h2(p00 * vd0, p01 * vd0);
                            r1 = pack_h2(p10 * vd1, p11 * vd1);
                        }
                        const unsigned b01 = movmatrix_trans(r0), b23 = movmatrix_trans(r1);
                        if (WUSHKV_ABL & 1) { st.o[bi][0] += __uint_as_float(b01 ^ b23); } else
                        if (BITS != 4) {
                            const uint4 vw = lds128(rec + v_codes_offset(BITS) + bi * CB + 16 * lane);
                            const unsigned sx = pre_shift<2>(vw.x), sy = pre_shift<2>(vw.y), sz = pre_shift<2>(vw.z), sw = pre_shift<2>(vw.w);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                mma_f16(st.o[i], field<2>(vw.x, sx, i), field<2>(vw.y, sy, i), field<2>(vw.z, sz, i), field<2>(vw.w, sw, i), b01, b23);
                            if (BITS == 3) {
                                // 1-bit plane: words of token halves ps = 0, 1; one of five shifts of a word puts the bit of
                                // (row half, channel block i) two bits above the low plane's field of block i, so that it reads
                                // as 4 x (high bit) in that field's unit and lands in the same accumulator
                                const uint2 vh = lds64(rec + v_hi_offset(3) + bi * 256 + 8 * lane);
                                const unsigned xv[5] = {vh.x, vh.x << 1, vh.x >> 9, vh.x >> 10, vh.x << 6};
                                const unsigned yv[5] = {vh.y, vh.y << 1, vh.y >> 9, vh.y >> 10, vh.y << 6};
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const unsigned m = 0x00010001u << v1_target(i);
                                    const int r0 = i < 5 ? 0 : 2, r1 = i < 5 ? 1 : (i < 7 ? 3 : 4);
                                    mma_f16(st.o[i], xv[r0] & m, xv[r1] & m, yv[r0] & m, yv[r1] & m, b01, b23);
                                }
                            }
                        } else {
                            const uint4 va = lds128(rec + v_codes_offset(4) + bi * CB + 16 * lane);         // tokens 2t,2t+1
                            const uint4 vb = lds128(rec + v_codes_offset(4) + bi * CB + 512 + 16 * lane);   // tokens 2t+8,2t+9
                            const unsigned a0s = pre_shift<4>(va.x), a1s = pre_shift<4>(va.y), a2s = pre_shift<4>(va.z), a3s = pre_shift<4>(va.w);
                            const unsigned b0s = pre_shift<4>(vb.x), b1s = pre_shift<4>(vb.y), b2s = pre_shift<4>(vb.z), b3s = pre_shift<4>(vb.w);
#pragma unroll
                            for (int k = 0; k < 4; ++k)     // channel blocks 0..3: words (rsel, j=0)
                                mma_f16(st.o[k], field<4>(va.x, a0s, k), field<4>(va.z, a2s, k), field<4>(vb.x, b0s, k), field<4>(vb.z, b2s, k), b01, b23);
#pragma unroll
                            for (int k = 0; k < 4; ++k)     // channel blocks 4..7: words (rsel, j=1)
                                mma_f16(st.o[4 + k], field<4>(va.y, a1s, k), field<4>(va.w, a3s, k), field<4>(vb.y, b1s, k), field<4>(vb.w, b3s, k), b01, b23);
                        }
                    }
                }
                __syncwarp();
                if (issued < round_units) issue_next(s);         // refill the stage just consumed
                stage = (stage + 1 == STAGES) ? 0 : stage + 1;
            }
            store_partial<BITS, MODE>(st, P.part + (wg + static_cast<long long>(sg.b) * c.n_kv + sg.h) * G * PART_STRIDE, lane, G);
        }
        __syncwarp();
    }
    TL(3);
    if (timed_out) {
        if (lane == 0) atomicOr(c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
        // Copies of this warp's other stages may still be in flight: wait for each (bounded; a stage with nothing
        // pending simply runs the limit out) before the CTA's shared memory can be released.
        const int drain_limit = min(wait_limit, 1 << 9);
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_wait_bounded(bar0 + 8 * s, (phase_bits >> s) & 1u, drain_limit);
    }
}

// ------------------------------------------------------------------------------------------------
// 3. combine
// ------------------------------------------------------------------------------------------------
// One CTA per (sequence, query head): up to 8 thread groups of one thread per channel, each merging a
// contiguous share of the head's partials.  The partials sit in L2, so the cost is load latency: a
// group issues the loads of COMBINE_BATCH partials together before it merges them.
constexpr int COMBINE_BATCH = 8;        // loads in flight per thread
template <int MAX_GROUPS, int GS>      // GS: log2 of the warps per slice (compile-time copy of slice_shift)
__global__ void __launch_bounds__(128 * MAX_GROUPS) decode_combine_kernel(DecodeParams P) {
    __shared__ float red_m[MAX_GROUPS], red_l[MAX_GROUPS], red_o[MAX_GROUPS][D];
    const CacheView& c = P.c;
    const int j = blockIdx.x, b = blockIdx.y, ch = threadIdx.x, grp = threadIdx.y, n_grp = blockDim.y;
    pdl_wait();                                         // partials and the plan come from the earlier kernels
    pdl_launch_dependents();                            // a programmatically launched successor waits for us itself
    float* out = P.O + (static_cast<long long>(b) * c.n_q + j) * D;
    const long long U = P.plan[b + 1] - P.plan[b];
    const long long total = P.plan[P.batch] * c.n_kv;
    if (U <= 0 || total <= 0) { if (grp == 0) out[ch] = 0.f; return; }
    const int h = j / c.G, head = j % c.G;
    const long long La = P.plan[b] * c.n_kv + static_cast<long long>(h) * U, Lb = La + U;      // units [La, Lb)
    // The unit list is cut into ns equal slices, slice i = [floor(i total / ns), floor((i+1) total / ns)); a
    // slice belongs to one warp (slice_shift 0) or to the four warps of a CTA (slice_shift 2), and every
    // warp of a slice that meets [La, Lb) wrote a partial, at slot (slice + bh) * warps_per_slice + warp.
    constexpr int gs = GS, group_mask = (1 << gs) - 1;
    const long long ns = static_cast<long long>(P.n_warps) >> gs;
    const long long s_first = ((La + 1) * ns - 1) / total, s_last = (Lb * ns - 1) / total;   // owners of La and Lb-1
    const long long bh = static_cast<long long>(b) * c.n_kv + h;
    const long long stride = static_cast<long long>(c.G) * PART_STRIDE;
    const int n = static_cast<int>(s_last - s_first + 1) << gs;
    // thread group grp merges the contiguous share [k0, k1) of the n partials
    const int share = (n + n_grp - 1) / n_grp;
    const int k0 = min(grp * share, n), k1 = min(k0 + share, n);
    const float* base = P.part + ((((s_first + bh) << gs) + k0) * c.G + head) * PART_STRIDE;
    // slice bounds advance by q = total / ns with a carry of r = total % ns (no division in the loop)
    const long long q = total / ns, r = total % ns;
    const long long sl0 = s_first + (k0 >> gs);
    long long lo_w = sl0 * total / ns, rem = (sl0 * total) % ns;
    long long hi_w = lo_w + q;
    rem += r;
    if (rem >= ns) { rem -= ns; ++hi_w; }
    float m = -INFINITY, l = 0.f, o = 0.f;
    for (int s0 = k0; s0 < k1; s0 += COMBINE_BATCH) {
        float pm[COMBINE_BATCH], pl[COMBINE_BATCH], po[COMBINE_BATCH];
#pragma unroll
        for (int k = 0; k < COMBINE_BATCH; ++k) {
            pm[k] = -INFINITY; pl[k] = 0.f; po[k] = 0.f;
            if (s0 + k < k1) {
                const bool wrote = max(lo_w, La) < min(hi_w, Lb);     // a slice that misses the range wrote nothing
                if (((s0 + k + 1) & group_mask) == 0) {               // next partial belongs to the next slice
                    lo_w = hi_w;
                    hi_w = lo_w + q;
                    rem += r;
                    if (rem >= ns) { rem -= ns; ++hi_w; }
                }
                if (wrote) {
                    const float* p = base + (s0 - k0 + k) * stride;
                    pm[k] = __ldcg(p); pl[k] = __ldcg(p + 1); po[k] = __ldcg(p + 4 + ch);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < COMBINE_BATCH; ++k) {
            if (pm[k] == -INFINITY) continue;
            const float mn = fmaxf(m, pm[k]);
            const float sa = exp2f(m - mn), sb = exp2f(pm[k] - mn);   // m = -inf on the first partial: sa = 0
            l = l * sa + pl[k] * sb;
            o = o * sa + po[k] * sb;
            m = mn;
        }
    }
    if (MAX_GROUPS > 1 && n_grp > 1) {                  // merge the groups' states, in group order
        if (ch == 0) { red_m[grp] = m; red_l[grp] = l; }
        red_o[grp][ch] = o;
        __syncthreads();
        if (grp != 0) return;
        for (int k = 1; k < n_grp; ++k) {
            const float pm = red_m[k];
            if (pm == -INFINITY) continue;
            const float mn = fmaxf(m, pm);
            const float sa = exp2f(m - mn), sb = exp2f(pm - mn);
            l = l * sa + red_l[k] * sb;
            o = o * sa + red_o[k][ch] * sb;
            m = mn;
        }
    }
    out[ch] = l > 0.f ? o / l : 0.f;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct DecodePlan {
    int n_ctas, n_warps;
    size_t off_qfrag, off_qwfrag, off_qscal, off_plan, off_part, total;
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool make_plan(const CacheView& c, int batch, int max_seq_len, DecodePlan& pl) {
    if (batch <= 0 || max_seq_len <= 0) return false;
    const long long pages_max = (static_cast<long long>(max_seq_len) + PAGE_TOKENS - 1) / PAGE_TOKENS + 1;
    const long long win_max = std::min<long long>(max_seq_len, c.s_sink + c.s_keep + c.s_flush - 1 + c.lag);
    const long long units_max = (pages_max + (win_max + WIN_TOKENS - 1) / WIN_TOKENS + 1) * batch * c.n_kv;
    const int warps = main_warps(c.bits, c.G <= 4 ? 0 : 1);
    long long ctas = knobs().decode_ctas;
    if (ctas <= 0) {
        // one CTA per SM; small problems take fewer, so that every warp still gets about two units
        ctas = std::min<long long>(sm_count(), (units_max + 2 * warps - 1) / (2 * warps));
    }
    ctas = std::max<long long>(1, std::min<long long>(ctas, 1 << 20));
    pl.n_ctas = static_cast<int>(ctas);
    pl.n_warps = pl.n_ctas * warps;
    const size_t bh = static_cast<size_t>(batch) * c.n_kv;
    size_t off = 0;
    pl.off_qfrag = off;  off = align_up(off + bh * 256 * sizeof(uint4), 256);
    pl.off_qwfrag = off; off = align_up(off + bh * 256 * sizeof(uint4), 256);
    pl.off_qscal = off;  off = align_up(off + static_cast<size_t>(batch) * c.n_q * 2 * sizeof(float), 256);
    pl.off_plan = off;   off = align_up(off + (static_cast<size_t>(batch) + 1) * sizeof(long long), 256);
    pl.off_part = off;   off = align_up(off + (pl.n_warps + bh) * c.G * PART_STRIDE * sizeof(float), 256);
    pl.total = off;
    return true;
}

static cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;

template <int BITS, int MODE>
static int launch_decode(const DecodeParams& P, int n_ctas, cudaStream_t st) {
    constexpr int MAIN_WARPS = main_warps(BITS, MODE);
#ifndef WUSHKV_STAGES_2BIT
#define WUSHKV_STAGES_2BIT 2
#endif
    constexpr int STAGES = (BITS == 2 && MODE == 0) ? WUSHKV_STAGES_2BIT : 2;      // per-warp ring depth
    constexpr size_t SMEM = static_cast<size_t>(MAIN_WARPS) * STAGES * record_bytes(BITS) + MAIN_WARPS * STAGES * 8 +
                            MAIN_WARPS * MAX_SEGMENTS * sizeof(Segment);
    cudaLaunchAttribute pdl_attr[1];
    pdl_attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl_attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st;
    cfg.attrs = pdl_attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(P.c.n_kv, P.batch);
    cfg.blockDim = dim3(PREP_THREADS);
    cfg.dynamicSmemBytes = 0;
    if (cudaLaunchKernelEx(&cfg, decode_prep_kernel<BITS, MODE>, P) != cudaSuccess) return WUSHKV_ECUDA;
    if (!opt_in_dynamic_smem(reinterpret_cast<const void*>(decode_main_kernel<BITS, MODE, STAGES>), static_cast<int>(SMEM))) return WUSHKV_ECUDA;
    if (g_prof_start) cudaEventRecord(g_prof_start, st);
    cfg.gridDim = dim3(n_ctas);
    cfg.blockDim = dim3(MAIN_WARPS * 32);
    cfg.dynamicSmemBytes = SMEM;
    if (cudaLaunchKernelEx(&cfg, decode_main_kernel<BITS, MODE, STAGES>, P) != cudaSuccess) return WUSHKV_ECUDA;
    if (g_prof_stop) cudaEventRecord(g_prof_stop, st);
    // Partials per (sequence, KV head) are about n_warps / (batch n_kv).  Short lists go to one thread
    // group per CTA (a few rounds of COMBINE_BATCH loads); a long list (few sequences, long context)
    // is shared by 8 groups.
    const long long per_head = P.n_warps / (static_cast<long long>(P.batch) * P.c.n_kv) + 2;
    cfg.gridDim = dim3(P.c.n_q, P.batch);
    cfg.dynamicSmemBytes = 0;
    if (per_head <= 4 * COMBINE_BATCH) {
        cfg.blockDim = dim3(128, 1);
        if (cudaLaunchKernelEx(&cfg, decode_combine_kernel<1, 0>, P) != cudaSuccess) return WUSHKV_ECUDA;
    } else {
        cfg.blockDim = dim3(128, 8);
        if (cudaLaunchKernelEx(&cfg, decode_combine_kernel<8, 0>, P) != cudaSuccess) return WUSHKV_ECUDA;
    }
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

static int decode_attn_impl(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                            int32_t max_seq_len, const uint16_t* Q, float* O,
                            void* workspace, size_t workspace_bytes, void* stream, int q_early,
                            const wushkv_prologue* prologue = nullptr) {
    DecodeParams P;
    P.q_early = q_early;
    const int rc = make_view(cache, P.c);
    if (rc != WUSHKV_OK) return rc;
    if (!slot || !seq_len || !Q || !O || !workspace || !aligned(Q, 16) || !aligned(O, 16) || !aligned(workspace, 256)) return WUSHKV_EINVAL;
    DecodePlan pl;
    if (!make_plan(P.c, batch, max_seq_len, pl)) return WUSHKV_EINVAL;
    if (batch > 65535) return WUSHKV_EINVAL;
    if (workspace_bytes < pl.total) return WUSHKV_ECAPACITY;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    P.batch = batch; P.slot = slot; P.seq_len = seq_len; P.Q = Q; P.O = O;
    P.qfrag = reinterpret_cast<uint4*>(ws + pl.off_qfrag);
    P.qwfrag = reinterpret_cast<uint4*>(ws + pl.off_qwfrag);
    P.qscal = reinterpret_cast<float*>(ws + pl.off_qscal);
    P.plan = reinterpret_cast<long long*>(ws + pl.off_plan);
    P.part = reinterpret_cast<float*>(ws + pl.off_part);
    P.n_warps = pl.n_warps;
    P.wait_limit = static_cast<int>(std::min<long long>(std::max<long long>(knobs().wait_limit, 0), 1 << 30));
    P.drop_unit = knobs().drop_copy_unit;
    P.pro = Prologue{nullptr, 0, 0, nullptr, 0.f};
    if (prologue && !make_prologue(prologue, prologue->q_norm_weight, P.pro)) return WUSHKV_EINVAL;
    {   // upper bound of the packed bytes one step reads against the L2 size
        static int l2_bytes[64] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return WUSHKV_ECUDA;
        int l2 = (dev >= 0 && dev < 64) ? l2_bytes[dev] : 0;
        if (l2 == 0) {
            if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess) return WUSHKV_ECUDA;
            if (dev >= 0 && dev < 64) l2_bytes[dev] = l2;
        }
        const double step_bytes = static_cast<double>(batch) * P.c.n_kv * ((max_seq_len + PAGE_TOKENS - 1) / PAGE_TOKENS) *
                                  record_bytes(P.c.bits);
        P.stream_pages = step_bytes > static_cast<double>(l2) ? 1 : 0;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool mode0 = P.c.G <= 4;
    if (P.c.bits == 2) return mode0 ? launch_decode<2, 0>(P, pl.n_ctas, st) : launch_decode<2, 1>(P, pl.n_ctas, st);
    if (P.c.bits == 3) return mode0 ? launch_decode<3, 0>(P, pl.n_ctas, st) : launch_decode<3, 1>(P, pl.n_ctas, st);
    return mode0 ? launch_decode<4, 0>(P, pl.n_ctas, st) : launch_decode<4, 1>(P, pl.n_ctas, st);
}

extern "C" int wushkv_decode_attn(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                  int32_t max_seq_len, const uint16_t* Q, float* O,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    return decode_attn_impl(cache, batch, slot, seq_len, max_seq_len, Q, O, workspace, workspace_bytes, stream, 0);
}

extern "C" int wushkv_decode_attn_projected(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                            int32_t max_seq_len, const uint16_t* Q_proj, const wushkv_prologue* prologue, float* O,
                                            void* workspace, size_t workspace_bytes, void* stream) {
    if (!prologue) return WUSHKV_EINVAL;
    // the query's position is the final length minus one: the preparation kernel waits for the kernel ahead of it
    return decode_attn_impl(cache, batch, slot, seq_len, max_seq_len, Q_proj, O, workspace, workspace_bytes, stream, 0, prologue);
}

extern "C" int wushkv_decode_step(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                                  const int32_t* cu_new, int32_t max_seq_len,
                                  const uint16_t* K_new, const uint16_t* V_new, const uint16_t* Q, float* O,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    if (batch <= 0 || !Q || !O || !workspace) return WUSHKV_EINVAL;
    // validate the decode half before anything is appended
    CacheView v;
    int r = make_view(cache, v);
    if (r != WUSHKV_OK) return r;
    DecodePlan pl;
    if (!make_plan(v, batch, max_seq_len, pl) || batch > 65535 || !aligned(Q, 16) || !aligned(O, 16) || !aligned(workspace, 256)) return WUSHKV_EINVAL;
    if (workspace_bytes < pl.total) return WUSHKV_ECAPACITY;
    r = wushkv_append(cache, batch, slot, seq_len, cu_new, batch, 1, K_new, V_new, stream);
    if (r != WUSHKV_OK) return r;
    // the single-token append kernel is now the kernel ahead of the query preparation, and it started
    // only after all earlier work in the stream: the preparation may read Q without waiting for it
    return decode_attn_impl(cache, batch, slot, seq_len, max_seq_len, Q, O, workspace, workspace_bytes, stream, 1);
}

#if WUSHKV_ABL & 16
extern "C" int wushkv_debug_timeline(unsigned long long* host_out, int clear) {
    if (cudaMemcpyFromSymbol(host_out, g_timeline, sizeof(g_timeline)) != cudaSuccess) return WUSHKV_ECUDA;
    if (clear) { void* p; cudaGetSymbolAddress(&p, g_timeline); cudaMemset(p, 0, sizeof(g_timeline)); }
    return WUSHKV_OK;
}
#endif

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

// Device-side alias of a pinned, mapped host buffer (unified addressing), or nullptr.
static void* mapped_alias(const void* host_ptr) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return nullptr;
    return aligned(a.devicePointer, 16) ? a.devicePointer : nullptr;
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
    // Pinned host buffers are visible to the device: the kernels then read the new token and the queries,
    // and write the outputs, in place over the bus, which saves four copy operations per step (about 320 KB
    // in config 1, where the copies' fixed costs dominate).  WUSHKV_HOST_IO=copy forces the staged copies.
    if (!knobs().host_io_copy) {
        void* aK = mapped_alias(K_new_host);
        void* aV = aK ? mapped_alias(V_new_host) : nullptr;
        void* aQ = aV ? mapped_alias(Q_host) : nullptr;
        void* aO = aQ ? mapped_alias(O_host) : nullptr;
        if (aO)
            return wushkv_decode_step(cache, batch, slot, seq_len, cu_new, max_seq_len, static_cast<const uint16_t*>(aK),
                                      static_cast<const uint16_t*>(aV), static_cast<const uint16_t*>(aQ), static_cast<float*>(aO),
                                      workspace, workspace_bytes, stream);
    }
    if (cudaMemcpyAsync(dK, K_new_host, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return WUSHKV_ECUDA;
    if (cudaMemcpyAsync(dV, V_new_host, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return WUSHKV_ECUDA;
    if (cudaMemcpyAsync(dQ, Q_host, q_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return WUSHKV_ECUDA;
    const int r = wushkv_decode_step(cache, batch, slot, seq_len, cu_new, max_seq_len, dK, dV, dQ, dO, workspace, workspace_bytes, stream);
    if (r != WUSHKV_OK) return r;
    if (cudaMemcpyAsync(O_host, dO, o_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return WUSHKV_ECUDA;
    return WUSHKV_OK;
}
