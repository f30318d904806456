// Decode attention over the packed cache (Algorithm 2 lines 3 and 5; Eq. 2; Eq. 3; Section 4.4).
//
// Three launches on the caller's stream:
//   1. decode_prep_kernel   q' = T_K^{-T} q per query head (Algorithm 2 line 3), written as mma
//                           B-fragments: fp16 (value + rounding remainder), pre-scaled by the power of
//                           two that each packed code field carries, for the quantized positions, and
//                           bf16 (value + remainder) for the bf16 windows.  Block (0,0) also writes the
//                           work plan: the prefix sums of work units per sequence.
//   2. decode_main_kernel   ONE wave of CTAs; every WARP owns an equal, contiguous slice of the
//                           flattened list of work units (sequence, KV head, unit), a unit being a
//                           64-token packed page or up to 8 tokens of the bf16 sink / recent windows.
//                           A warp streams its units into shared memory with bulk async copies (mbarrier
//                           ring), turns code words into fp16 A-fragments with one AND per register, and
//                           runs both contractions (q'.k and p.v) on mma.sync.m16n8k16 with fp32
//                           accumulation.  The affine part of Eq. 6 is factored out of the contractions:
//                               q'.k_hat = Delta_k (q'.c_k) + x_min_k sum(q'),
//                               o        = sum_s (p_s Delta_v,s) c_v,s + (sum_s p_s x_min_v,s) 1.
//                           Window units use ldmatrix + bf16 mma on the staged rows and fold into the
//                           same accumulators.  Softmax is online (running max / sum) per warp; a warp
//                           writes one partial (max, sum, o) per (sequence, KV head) it touched.
//  2b. decode_main_tc_kernel  opt-in alternative to 2 for G <= 4 (WUSHKV_DECODE_PATH=tc): the scores come from
//                           tcgen05.mma on e4m3 code bytes held in tensor memory; a CTA's four warps share
//                           128-token tiles.  Measured slower than 2; kept with its parity test.
//   3. decode_combine_kernel merges the partials of each (sequence, query head) into O.
//
// No kernel waits on another CTA.  The only waits are on a warp's (2b: a CTA's) own copy and MMA
// barriers, bounded by an iteration limit after which the kernel records WUSHKV_DEV_COPY_TIMEOUT and
// drains; in 2b the four warps of a CTA also meet at CTA barriers, whose outcome carries that flag.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <cuda_fp8.h>

#include <algorithm>
#include <cstdlib>

#include "host_common.h"
#include "layout.cuh"

namespace wushkv {

constexpr unsigned FULL = 0xffffffffu;
constexpr int PART_STRIDE = 132;          // floats per partial: [0]=max (log2 domain) [1]=sum [4..131]=o
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LO_SCALE = 2048.f;        // a "remainder" column carries (x - rounded(x)) * 2^11
// Exponentials are taken against (running reference - LOG2_PV): every probability, and with it l, z and
// o of a partial, carries the common factor 2^LOG2_PV, which cancels in the final ratio and keeps
// fp16(p Delta_v) out of the subnormals.  The reference is only raised (and the state rescaled) when
// a unit's maximum exceeds it by more than MAX_SLACK, so p <= 2^(LOG2_PV + MAX_SLACK) and
// p Delta_v stays finite in fp16 for Delta_v < 2^(16 - LOG2_PV - MAX_SLACK) = 1024.
constexpr float LOG2_PV = 3.f;
constexpr float MAX_SLACK = 3.f;
constexpr int MAIN_WARPS = 4;
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
    uint4* qfrag;        // [batch*n_kv][2][128]: fp16 B fragments of the 8 k-steps (MODE 1: value set, remainder set)
    uint4* qwfrag;       // [batch*n_kv][2][128]: bf16 B fragments for the windows (MODE 1: value set, remainder set)
    float* qscal;        // [batch][n_q][2]: score multiplier (log2 domain, > 0), x_min multiplier divided by it
    long long* plan;     // [batch+1]: exclusive prefix of work units per sequence (per KV head)
    float* part;         // [n_warps + batch*n_kv][G][PART_STRIDE]
    int n_warps;         // warps of the main kernel
    int q_early;         // 1: Q was final before the kernel ahead of the preparation kernel started
    unsigned char* qb8;  // [batch*n_kv][2048]: e4m3 query operand of the tensor-memory kernel (null: not used)
    float* qscal8;       // [batch][n_q][2]: the same two scalars as qscal for the e4m3 operand
    int slice_shift;     // log2 of the warps that share one slice of the unit list (0: each warp its own, 2: a CTA)
    int stream_pages;    // 1: the packed pages of a step cannot stay in L2 anyway: copy them with an evict-first hint
};

// shift of the code field used by k-step / channel block idx (0..7) inside its 16-bit lane, after
// the optional whole-word shift: the fp16 value of the masked field is code * 2^(field_shift - 24)
template <int BITS>
__host__ __device__ constexpr int field_shift(int idx) {
    return BITS == 2 ? (idx < 5 ? 2 * idx : 2 * (idx - 5)) : 4 * (idx & 1);
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

// ---- constants of the tensor-memory main kernel (section 2b) that the query preparation shares
constexpr int TC_STAGES = 4;
constexpr int TC_TMEM_COLS = 64;          // 32 columns of A (128 e4m3 per token row) and two D buffers of 16
constexpr int TC_D_COL = 32;
constexpr int QB_LBO = 128, QB_SBO = 1024, QB_BYTES = 2048;       // 16 x 128 e4m3, K-major core matrices (8 rows x 16 B)
constexpr unsigned QK8_IDESC = (1u << 4) | ((16u >> 3) << 17) | ((128u >> 4) << 24);    // D fp32, A and B e4m3 K-major, N 16, M 128

// Position k (0..127) of channel ch in the e4m3 row the tensor-memory kernel lays out for a token, and
// whether the mask that extracts it leaves the code shifted up by two bits (a factor 4).  Thread (g, t)
// of a warp owns, exactly as in the register-operand kernel, the 16 bytes of key block codes of token
// rows g and g+8 x channels {16s + 8w + 2t + hi}; it writes them with tcgen05.st.16x256b, where register
// pair j of a row lands in tensor-memory columns 8j + 2t and 8j + 2t + 1, four e4m3 bytes per column.
template <int BITS>
__host__ __device__ inline int tc_k_of_channel(int ch, bool& times4) {
    const int s = ch >> 4, r16 = ch & 15, w = r16 >> 3, tq = (r16 & 7) >> 1, hi = r16 & 1;
    if (BITS == 2) {
        const int m = s & 3, byte = 2 * hi + (s >> 2);          // mask m of word w; byte = half-word, low / high byte
        times4 = (m & 1) != 0;
        return 4 * (8 * (2 * w + (m >> 1)) + 2 * tq + (m & 1)) + byte;
    } else {
        const int hn = s & 1, byte = 2 * hi + ((s & 3) >> 1), jw = 2 * (s >> 2) + w;      // nibble hn of word jw
        times4 = false;
        return 4 * (8 * jw + 2 * tq + hn) + byte;
    }
}

// ------------------------------------------------------------------------------------------------
// 1. query preparation
// ------------------------------------------------------------------------------------------------
constexpr int PREP_THREADS = 512;                   // 16 warps share the 128 rows of T_K^{-T}
constexpr int PREP_ROWS = D / (PREP_THREADS / 32);   // rows per warp
template <int BITS, int MODE>
__global__ void __launch_bounds__(PREP_THREADS) decode_prep_kernel(DecodeParams P) {
    __shared__ float q_s[8][D];
    __shared__ float red_max[8][4];
    __shared__ float red_sum[8][4];
    __shared__ float red_abs[8][4];
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
                u = seq_info(P.c, __ldg(P.seq_len + bb), slot).U;
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
    const int s = i >> 4;
    const float pos_scale = exp2f(-static_cast<float>(field_shift<BITS>(s)));
    const float k2 = P.c.sm_scale * LOG2E;
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        if (g < G) {
            float mx = fabsf(acc[g]) * pos_scale, sm = acc[g], ab = fabsf(acc[g]);
            for (int o = 16; o > 0; o >>= 1) {
                mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
                sm += __shfl_xor_sync(FULL, sm, o);
                ab = fmaxf(ab, __shfl_xor_sync(FULL, ab, o));
            }
            if (lane == 0) { red_max[g][warp] = mx; red_sum[g][warp] = sm; red_abs[g][warp] = ab; }
        }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");       // the four remaining warps only
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
                qs[0] = k2 * 16777216.f / beta[g];            // score = qs[0] * (Delta_k * (codes . q'') + x_min_k * qs[1])
                qs[1] = sum * beta[g] * (1.f / 16777216.f);
            }
        }
    }
    // B fragments.  Element (k-step s, register r, lane 4n+t, half hf) is channel 16s + 8r + 2t + hf of
    // mma column n.  MODE 0: column n holds head n>>1, its rounded value (n even) or the rounding
    // remainder times 2^11 (n odd).  MODE 1: column n holds head n; the window set has a second copy
    // with the remainders.
    const int r16 = i & 15, r = r16 >> 3, t = (r16 & 7) >> 1, hf = r16 & 1;
    const long long bh = static_cast<long long>(b) * P.c.n_kv + h;
    unsigned short* frag = reinterpret_cast<unsigned short*>(P.qfrag + bh * 256);
    unsigned short* wfrag = reinterpret_cast<unsigned short*>(P.qwfrag + bh * 256);
#pragma unroll
    for (int n = 0; n < 8; ++n) {
        const int head = (MODE == 0) ? (n >> 1) : n;
        float val = 0.f, rem = 0.f, wval = 0.f, wrem = 0.f;
        if (head < G) {
            const float x = acc[head] * pos_scale * beta[head];
            const __half hi = __float2half_rn(x);
            rem = (x - __half2float(hi)) * LO_SCALE;
            val = (MODE == 0 && (n & 1)) ? rem : x;
            const float y = acc[head] * k2;
            const float yh = __bfloat162float(__float2bfloat16_rn(y));
            wrem = y - yh;
            wval = (MODE == 0 && (n & 1)) ? wrem : y;
        }
        const int idx = ((((s >> 1) * 32 + 4 * n + t) * 4 + (s & 1) * 2 + r) << 1) + hf;
        frag[idx] = __half_as_ushort(__float2half_rn(val));
        if (MODE == 1) frag[1024 + idx] = __half_as_ushort(__float2half_rn(rem));
        wfrag[idx] = __bfloat16_as_ushort(__float2bfloat16_rn(wval));
        if (MODE == 1) wfrag[1024 + idx] = __bfloat16_as_ushort(__float2bfloat16_rn(wrem));
    }
    // Operand of the tensor-memory kernel: each head's q' as the sum of four e4m3 terms (value, then three
    // rounding remainders), scaled by a power of two so that the largest entry sits below 2^8; row n of the
    // 16 x 128 operand is head n/2's term n%2 (n < 8) or term 2 + n%2 (n >= 8), its k order is the order
    // in which a thread of that kernel lays out a token's codes, and the image is the K-major core-matrix
    // layout the MMA reads from shared memory.
    if (MODE == 0 && P.qb8 != nullptr) {
        bool times4;
        const int k = tc_k_of_channel<BITS>(i, times4);
        unsigned char* img = P.qb8 + bh * QB_BYTES + (k >> 4) * QB_LBO + (k & 15);
#pragma unroll
        for (int head = 0; head < 4; ++head) {
            float beta8 = 1.f, r = 0.f;
            if (head < G) {
                const float mx = fmaxf(fmaxf(red_abs[head][0], red_abs[head][1]), fmaxf(red_abs[head][2], red_abs[head][3]));
                int e = 0;
                if (mx > 0.f && mx < 3e38f) frexpf(mx, &e);          // mx < 2^e
                e = max(min(e, 100), -100);
                beta8 = exp2f(static_cast<float>(8 - e));
                r = acc[head] * beta8 * (times4 ? 0.25f : 1.f);
                if (i == 0) {
                    const float sum = red_sum[head][0] + red_sum[head][1] + red_sum[head][2] + red_sum[head][3];
                    float* qs = P.qscal8 + (static_cast<long long>(b) * P.c.n_q + h * G + head) * 2;
                    qs[0] = k2 * 512.f / beta8;                   // an e4m3 code field is code * 2^-9
                    qs[1] = sum * beta8 * (1.f / 512.f);
                }
            }
#pragma unroll
            for (int term = 0; term < 4; ++term) {
                const __nv_fp8_e4m3 q8(r);                         // round to nearest, saturating
                r -= static_cast<float>(q8);
                const int n = (term < 2) ? 2 * head + term : 8 + 2 * head + (term - 2);
                img[(n >> 3) * QB_SBO + (n & 7) * 16] = q8.__x;
            }
        }
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
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity) {
    for (int it = 0; it < (1 << 19); ++it)
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
    if (BITS == 2) {
        constexpr unsigned M0 = 0x00030003u;
        return idx < 5 ? (w & (M0 << (2 * idx))) : (ws & (M0 << (2 * (idx - 5))));
    } else {
        constexpr unsigned M0 = 0x000F000Fu;
        return idx < 2 ? (w & (M0 << (4 * idx))) : (ws & (M0 << (4 * (idx - 2))));
    }
}
template <int BITS> __device__ __forceinline__ unsigned pre_shift(unsigned w) { return BITS == 2 ? (w >> 10) : (w >> 8); }

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
            const uint4 bq = __ldg(wsrc + pass * 128 + s2 * 32 + lane);
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
template <int BITS, int MODE, int STAGES>
__global__ void __launch_bounds__(MAIN_WARPS * 32, (BITS == 4 ? 3 : (MODE == 0 ? 4 : 3))) decode_main_kernel(DecodeParams P) {
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
            if (bb < P.batch) incl = seq_info(c, __ldg(P.seq_len + bb), __ldg(P.slot + bb)).U;
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

    unsigned qf[8][2];
    float fmul[NH], gadd[NH];
    WarpState<MODE> st;
    int stage = 0;                      // ring position of the next unit to consume (and to refill)
    unsigned phase_bits = 0;            // parity of each stage's next completion
    unsigned bad_bits = 0;              // lane 0: stages whose unit could not be fetched
    bool timed_out = false;

    while (L < L1 && !timed_out) {
        // ================= round set-up: list the next segments of the slice =====================
        int n_seg = 0, round_units = 0;
        while (n_seg < MAX_SEGMENTS && L < L1) {
            const SeqInfo si = seq_info(c, __ldg(P.seq_len + sb), __ldg(P.slot + sb));
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
                    } else {
                        bad_bits &= ~(1u << s);
                        mbar_expect_tx(bar, REC);
                        if (P.stream_pages) bulk_copy_g2s_stream(dst, c.pages + page * page_row_bytes + p_head_off, REC, bar, stream_policy);
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
                for (int s2 = 0; s2 < 4; ++s2) {
                    const uint4 v = __ldg(src + s2 * 32 + lane);
                    qf[2 * s2][0] = v.x; qf[2 * s2][1] = v.y; qf[2 * s2 + 1][0] = v.z; qf[2 * s2 + 1][1] = v.w;
                }
#pragma unroll
                for (int k = 0; k < NH; ++k) {
                    const int head = MODE == 0 ? t : 2 * t + k;
                    fmul[k] = 1.f; gadd[k] = 0.f;             // unused head slots stay finite
                    if (head < G) {
                        const float2 v = __ldg(reinterpret_cast<const float2*>(P.qscal + (static_cast<long long>(sg.b) * c.n_q + sg.h * G + head) * 2));
                        fmul[k] = v.x; gadd[k] = v.y;
                    }
                }
                st.reset();
            }
            for (int u = sg.u0; u < u1; ++u, pos0 += PAGE_TOKENS) {
                const int s = stage;
                // a phase that one lane saw complete is complete for all: keep the decision warp-uniform
                if (!__any_sync(FULL, mbar_wait_bounded(bar0 + 8 * s, (phase_bits >> s) & 1u))) { timed_out = true; break; }
                phase_bits ^= 1u << s;
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
                        float acc[4];                 // one chain per block; the four blocks of a page are independent
                        if (BITS == 2) {
                            const uint4 kw = lds128(rec + bi * CB + 16 * lane);
                            const unsigned sx = pre_shift<2>(kw.x), sy = pre_shift<2>(kw.y), sz = pre_shift<2>(kw.z), sw = pre_shift<2>(kw.w);
                            mma_f16_zero(acc, field<2>(kw.x, sx, 0), field<2>(kw.z, sz, 0), field<2>(kw.y, sy, 0), field<2>(kw.w, sw, 0), qf[0][0], qf[0][1]);
#pragma unroll
                            for (int ks = 1; ks < 8; ++ks)
                                mma_f16(acc, field<2>(kw.x, sx, ks), field<2>(kw.z, sz, ks), field<2>(kw.y, sy, ks), field<2>(kw.w, sw, ks),
                                        qf[ks][0], qf[ks][1]);
                        } else {
                            const uint4 ka = lds128(rec + bi * CB + 16 * lane);          // row g:   W0..W3
                            const uint4 kb = lds128(rec + bi * CB + 512 + 16 * lane);    // row g+8: W0..W3
                            const unsigned a0s = pre_shift<4>(ka.x), a1s = pre_shift<4>(ka.y), a2s = pre_shift<4>(ka.z), a3s = pre_shift<4>(ka.w);
                            const unsigned b0s = pre_shift<4>(kb.x), b1s = pre_shift<4>(kb.y), b2s = pre_shift<4>(kb.z), b3s = pre_shift<4>(kb.w);
                            mma_f16_zero(acc, field<4>(ka.x, a0s, 0), field<4>(kb.x, b0s, 0), field<4>(ka.y, a1s, 0), field<4>(kb.y, b1s, 0), qf[0][0], qf[0][1]);
#pragma unroll
                            for (int ks = 1; ks < 4; ++ks)
                                mma_f16(acc, field<4>(ka.x, a0s, ks), field<4>(kb.x, b0s, ks), field<4>(ka.y, a1s, ks), field<4>(kb.y, b1s, ks),
                                        qf[ks][0], qf[ks][1]);
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                mma_f16(acc, field<4>(ka.z, a2s, ks), field<4>(kb.z, b2s, ks), field<4>(ka.w, a3s, ks), field<4>(kb.w, b3s, ks),
                                        qf[4 + ks][0], qf[4 + ks][1]);
                        }
                        if (MODE == 1) {
                            // two heads per column pair leave no room for a remainder column: a second pass over
                            // the same A fragments with the remainder fragments (re-read per block: L1 hits)
                            float accr[4] = {0.f, 0.f, 0.f, 0.f}, accr2[4] = {0.f, 0.f, 0.f, 0.f};
                            const uint4* rsrc = P.qfrag + bh * 256 + 128 + lane;
                            if (BITS == 2) {
                                const uint4 kw = lds128(rec + bi * CB + 16 * lane);
                                const unsigned sx = pre_shift<2>(kw.x), sy = pre_shift<2>(kw.y), sz = pre_shift<2>(kw.z), sw = pre_shift<2>(kw.w);
#pragma unroll
                                for (int s2 = 0; s2 < 4; ++s2) {
                                    const uint4 rq = __ldg(rsrc + s2 * 32);
                                    mma_f16(accr, field<2>(kw.x, sx, 2 * s2), field<2>(kw.z, sz, 2 * s2), field<2>(kw.y, sy, 2 * s2), field<2>(kw.w, sw, 2 * s2), rq.x, rq.y);
                                    mma_f16(accr2, field<2>(kw.x, sx, 2 * s2 + 1), field<2>(kw.z, sz, 2 * s2 + 1), field<2>(kw.y, sy, 2 * s2 + 1), field<2>(kw.w, sw, 2 * s2 + 1), rq.z, rq.w);
                                }
                            } else {
                                const uint4 ka = lds128(rec + bi * CB + 16 * lane);
                                const uint4 kb = lds128(rec + bi * CB + 512 + 16 * lane);
                                const unsigned a0s = pre_shift<4>(ka.x), a1s = pre_shift<4>(ka.y), a2s = pre_shift<4>(ka.z), a3s = pre_shift<4>(ka.w);
                                const unsigned b0s = pre_shift<4>(kb.x), b1s = pre_shift<4>(kb.y), b2s = pre_shift<4>(kb.z), b3s = pre_shift<4>(kb.w);
#pragma unroll
                                for (int s2 = 0; s2 < 2; ++s2) {
                                    const uint4 rq = __ldg(rsrc + s2 * 32), rq2 = __ldg(rsrc + (s2 + 2) * 32);
                                    mma_f16(accr, field<4>(ka.x, a0s, 2 * s2), field<4>(kb.x, b0s, 2 * s2), field<4>(ka.y, a1s, 2 * s2), field<4>(kb.y, b1s, 2 * s2), rq.x, rq.y);
                                    mma_f16(accr, field<4>(ka.x, a0s, 2 * s2 + 1), field<4>(kb.x, b0s, 2 * s2 + 1), field<4>(ka.y, a1s, 2 * s2 + 1), field<4>(kb.y, b1s, 2 * s2 + 1), rq.z, rq.w);
                                    mma_f16(accr2, field<4>(ka.z, a2s, 2 * s2), field<4>(kb.z, b2s, 2 * s2), field<4>(ka.w, a3s, 2 * s2), field<4>(kb.w, b3s, 2 * s2), rq2.x, rq2.y);
                                    mma_f16(accr2, field<4>(ka.z, a2s, 2 * s2 + 1), field<4>(kb.z, b2s, 2 * s2 + 1), field<4>(ka.w, a3s, 2 * s2 + 1), field<4>(kb.w, b3s, 2 * s2 + 1), rq2.z, rq2.w);
                                }
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[e] = fmaf(accr[e] + accr2[e], 1.f / LO_SCALE, acc[e]);
                        }
                        const uint4 mt = lds128(rec + meta_offset(BITS) + 128 * bi + 16 * g);   // rows g (x,y) and g+8 (z,w)
                        const float2 km_a = h2f2(mt.x), km_b = h2f2(mt.z);
                        const float kd0 = km_a.x, km0 = km_a.y, kd1 = km_b.x, km1 = km_b.y;
                        vmeta[bi][0] = mt.y; vmeta[bi][1] = mt.w;
                        if (MODE == 0) {
                            const float d0 = fmaf(acc[1], 1.f / LO_SCALE, acc[0]), d1 = fmaf(acc[3], 1.f / LO_SCALE, acc[2]);
                            sc[bi][0] = fmaf(km0, gadd[0], d0 * kd0);
                            sc[bi][NH] = fmaf(km1, gadd[0], d1 * kd1);
                        } else {
                            sc[bi][0] = fmaf(km0, gadd[0], acc[0] * kd0);
                            sc[bi][NH - 1] = fmaf(km0, gadd[NH - 1], acc[1] * kd0);
                            sc[bi][NH] = fmaf(km1, gadd[0], acc[2] * kd1);
                            sc[bi][2 * NH - 1] = fmaf(km1, gadd[NH - 1], acc[3] * kd1);
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
                        if (BITS == 2) {
                            const uint4 vw = lds128(rec + v_codes_offset(2) + bi * CB + 16 * lane);
                            const unsigned sx = pre_shift<2>(vw.x), sy = pre_shift<2>(vw.y), sz = pre_shift<2>(vw.z), sw = pre_shift<2>(vw.w);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                mma_f16(st.o[i], field<2>(vw.x, sx, i), field<2>(vw.y, sy, i), field<2>(vw.z, sz, i), field<2>(vw.w, sw, i), b01, b23);
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
    if (timed_out) {
        if (lane == 0) atomicOr(c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
        // give copies that may still be in flight a bounded time to land before the CTA's memory is released
        for (int k = 0; k < 1000; ++k) __nanosleep(1000);
    }
}

// ------------------------------------------------------------------------------------------------
// 2b. main kernel with the scores on the tensor core (G <= 4)
// ------------------------------------------------------------------------------------------------
// Alternative, selected with WUSHKV_DECODE_PATH=tc; slower than the kernel above on every measured
// configuration (config 1: 135 us against 82 us), see the note where the path is chosen.
// The register-operand kernel above spends one mask per two key codes plus the MMA issue itself on the
// scores.  Here a CTA of four warps takes a contiguous slice of the unit list and walks it two units
// (128 tokens) at a time; for packed pages every thread owns one token row: it masks that row's codes
// in place into e4m3 bytes (four codes per mask: a 2-bit field inside bits 0..3 of a byte is the e4m3
// value field * 2^-9, subnormals and the first binade being linear in the bit pattern), writes the 128
// bytes to tensor memory (lane = token row) and one thread issues tcgen05.mma kind::f8f6f4 with that
// A operand against the query as four e4m3 terms per head (16 columns, shared memory).  The 128 x 16
// fp32 scores come back as 16 x 256 bit fragments, which is exactly the mma.sync accumulator layout the
// softmax / value code of the kernel above works in; values stay on mma.sync with per-warp states.
// The 16-token key block at shared address blk as e4m3 bytes in tensor memory: this lane's rows g and
// g+8, eight registers (columns 8j + 2t, 8j + 2t + 1) each, written to lanes taddr .. taddr + 15.
template <int BITS>
__device__ __forceinline__ void tc_store_key_block(unsigned blk, int lane, unsigned taddr) {
    unsigned a[16];                   // a[4j], a[4j+1]: row g; a[4j+2], a[4j+3]: row g+8
    if (BITS == 2) {
        const uint4 kw = lds128(blk + 16 * lane);                   // row g: words x, y; row g+8: words z, w
        const unsigned sx = kw.x >> 4, sy = kw.y >> 4, sz = kw.z >> 4, sw = kw.w >> 4;
        a[0] = kw.x & 0x03030303u;  a[1] = kw.x & 0x0C0C0C0Cu;  a[2] = kw.z & 0x03030303u;  a[3] = kw.z & 0x0C0C0C0Cu;
        a[4] = sx & 0x03030303u;    a[5] = sx & 0x0C0C0C0Cu;    a[6] = sz & 0x03030303u;    a[7] = sz & 0x0C0C0C0Cu;
        a[8] = kw.y & 0x03030303u;  a[9] = kw.y & 0x0C0C0C0Cu;  a[10] = kw.w & 0x03030303u; a[11] = kw.w & 0x0C0C0C0Cu;
        a[12] = sy & 0x03030303u;   a[13] = sy & 0x0C0C0C0Cu;   a[14] = sw & 0x03030303u;   a[15] = sw & 0x0C0C0C0Cu;
    } else {
        const uint4 ka = lds128(blk + 16 * lane);                   // row g:   W0..W3
        const uint4 kb = lds128(blk + 512 + 16 * lane);             // row g+8: W0..W3
        a[0] = ka.x & 0x0F0F0F0Fu;  a[1] = (ka.x >> 4) & 0x0F0F0F0Fu;  a[2] = kb.x & 0x0F0F0F0Fu;  a[3] = (kb.x >> 4) & 0x0F0F0F0Fu;
        a[4] = ka.y & 0x0F0F0F0Fu;  a[5] = (ka.y >> 4) & 0x0F0F0F0Fu;  a[6] = kb.y & 0x0F0F0F0Fu;  a[7] = (kb.y >> 4) & 0x0F0F0F0Fu;
        a[8] = ka.z & 0x0F0F0F0Fu;  a[9] = (ka.z >> 4) & 0x0F0F0F0Fu;  a[10] = kb.z & 0x0F0F0F0Fu; a[11] = (kb.z >> 4) & 0x0F0F0F0Fu;
        a[12] = ka.w & 0x0F0F0F0Fu; a[13] = (ka.w >> 4) & 0x0F0F0F0Fu; a[14] = kb.w & 0x0F0F0F0Fu; a[15] = (kb.w >> 4) & 0x0F0F0F0Fu;
    }
    asm volatile(
        "tcgen05.st.sync.aligned.16x256b.x4.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        :: "r"(taddr), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]),
           "r"(a[8]), "r"(a[9]), "r"(a[10]), "r"(a[11]), "r"(a[12]), "r"(a[13]), "r"(a[14]), "r"(a[15]) : "memory");
}

__device__ __forceinline__ unsigned long long qb_smem_desc(unsigned smem_addr) {
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((smem_addr >> 4) & 0x3FFFu);            // start address
    d |= static_cast<unsigned long long>((QB_LBO >> 4) & 0x3FFFu) << 16;         // leading (k chunk) byte offset
    d |= static_cast<unsigned long long>((QB_SBO >> 4) & 0x3FFFu) << 32;         // stride (row group) byte offset
    d |= 1ull << 46;                                                             // descriptor version of sm_100
    return d;                                                                    // no swizzle
}

template <int BITS>
__global__ void __launch_bounds__(MAIN_WARPS * 32, (BITS == 4 ? 3 : 4)) decode_main_tc_kernel(DecodeParams P) {
    constexpr int REC = record_bytes(BITS);
    constexpr int CB = code_block_bytes(BITS);
    constexpr int TILE = 2 * REC;                       // a stage holds two units
    static_assert(2 * WIN_TOKENS * WIN_ROW <= REC, "a window unit must fit in half a stage");
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* qb = smem + TC_STAGES * TILE;                                           // two operand buffers
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(qb + 2 * QB_BYTES);   // full[TC_STAGES], mma
    unsigned* misc = reinterpret_cast<unsigned*>(bars + TC_STAGES + 1);                    // [0] tensor-memory base, [1 + s] missing halves of stage s, [7] abort
    Segment* segs = reinterpret_cast<Segment*>(misc + 8);
    const CacheView& c = P.c;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = c.G;
    const int half = warp >> 1;                          // which unit of a stage this warp works on
    const int blk0 = 2 * (warp & 1);                     // its two 16-token blocks of that unit: blk0, blk0 + 1

    // ---- work plan (as in the kernel above)
    __shared__ long long scan_s[MAIN_WARPS];
    long long* plan_s = reinterpret_cast<long long*>(smem);
    const bool local_plan = (static_cast<size_t>(P.batch) + 1) * sizeof(long long) <= static_cast<size_t>(TC_STAGES) * TILE;
    if (local_plan) {
        long long carry = 0;
        for (int base = 0; base < P.batch; base += MAIN_WARPS * 32) {
            const int bb = base + tid;
            long long incl = 0;
            if (bb < P.batch) incl = seq_info(c, __ldg(P.seq_len + bb), __ldg(P.slot + bb)).U;
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
        if (tid == 0) plan_s[0] = 0;
        __syncthreads();
    } else {
        pdl_wait();
    }
    const long long* plan = local_plan ? plan_s : P.plan;

    // ---- this CTA's slice of the flattened unit list
    const long long total = plan[P.batch] * c.n_kv;
    const long long n_slices = gridDim.x;
    long long L = total > 0 ? blockIdx.x * total / n_slices : 0;
    const long long L1 = total > 0 ? (blockIdx.x + 1) * total / n_slices : 0;
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
    if (L >= L1) return;                    // the whole CTA: nothing allocated yet

    // ---- tensor memory, barriers
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(misc)), "r"(static_cast<unsigned>(TC_TMEM_COLS)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const unsigned bar0 = smem_u32(bars), mma_bar = bar0 + 8 * TC_STAGES;
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s <= TC_STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
#pragma unroll
        for (int s = 1; s < 8; ++s) misc[s] = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = misc[0];
    const unsigned my_tmem = tmem + (static_cast<unsigned>(warp * 32) << 16);     // this warp's 32 lanes: two 16-token blocks
    const unsigned stage0 = smem_u32(smem);
    const unsigned qb_addr = smem_u32(qb);
    const long long page_row_bytes = static_cast<long long>(c.n_kv) * REC;
    const unsigned my_rec_off = half * REC;

    WarpState<0> st;
    int stage = 0;                      // ring position of the tile being finished
    unsigned phase_bits = 0;            // parity of each stage's next completion
    unsigned mma_phase = 0;
    bool aborted = false;

    while (L < L1 && !aborted) {
        __syncthreads();                // every warp is done with the previous round's segments and stages
        // ================= round set-up: list the next segments of the slice =====================
        int n_seg = 0, round_tiles = 0;
        while (n_seg < MAX_SEGMENTS && L < L1) {
            const SeqInfo si = seq_info(c, __ldg(P.seq_len + sb), __ldg(P.slot + sb));
            if (si.U > 0) {
                const int u1 = static_cast<int>(min(static_cast<long long>(si.U), su + (L1 - L)));
                if (tid == 0) {
                    Segment sg;
                    sg.b = sb; sg.h = sh; sg.slot = si.slot; sg.u0 = su; sg.u1 = u1; sg.qp = si.qp; sg.first_page = si.first_page;
                    sg.q_lo = si.q_lo; sg.q_hi = si.q_hi; sg.n_win = si.n_win; sg.n_sink = si.n_sink; sg.recent_lo = si.recent_lo;
                    segs[n_seg] = sg;
                }
                ++n_seg;
                round_tiles += (u1 - su + 1) >> 1;
                L += u1 - su;
                su = u1;
            }
            if (si.U == 0 || su >= si.U) {              // next head, or next sequence
                su = 0;
                if (si.U == 0 || ++sh >= c.n_kv) { sh = 0; ++sb; }
                if (sb >= P.batch) break;
            }
        }
        __syncthreads();

        // ================= producer: stages the tiles of this round, in order =====================
        // Every warp tracks the cursor; the warp whose turn it is issues the copies (the turn rotates so
        // that no warp is always the last one at the CTA barrier).
        int p_seg = -1, p_u = 0, p_u1 = 0, p_qp = 0, p_sqp = 0, p_nwin = 0, p_head_off = 0, issued = 0;
        const int* p_ptab = nullptr;
        auto issue_tile = [&](const int s, const bool mine) {     // two units of one segment into ring slot s
            if (p_u >= p_u1) {                          // next segment
                ++p_seg;
                const Segment& sg = segs[p_seg];
                p_u = sg.u0; p_u1 = sg.u1; p_qp = p_sqp = sg.qp; p_nwin = sg.n_win; p_head_off = sg.h * REC;
                p_ptab = c.page_table + static_cast<long long>(sg.slot) * c.max_pages + sg.first_page;
                if (sg.first_page + sg.qp > c.max_pages) {      // the page table cannot hold this length
                    if (mine && lane == 0) atomicOr(c.dev_status, WUSHKV_DEV_PAGE_TABLE_FULL);
                    p_qp = min(p_qp, max(c.max_pages - sg.first_page, 0));
                }
            }
            if (mine) {
                const unsigned bar = bar0 + 8 * s, dst0 = stage0 + s * TILE;
                int page[2] = {-1, -1}, n_valid[2] = {0, 0};
                unsigned bytes = 0, missing = 0;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int uu = p_u + hf;
                    if (uu >= p_u1) continue;
                    if (uu < p_sqp) {
                        const int pg = (uu < p_qp) ? __ldg(p_ptab + uu) : -1;
                        if (static_cast<unsigned>(pg) >= static_cast<unsigned long long>(c.n_pages)) {
                            if (lane == 0 && uu < p_qp) atomicOr(c.dev_status, WUSHKV_DEV_BAD_PAGE_ID);
                            missing |= 1u << hf;
                        } else {
                            page[hf] = pg;
                            bytes += REC;
                        }
                    } else {
                        n_valid[hf] = min(WIN_TOKENS, p_nwin - (uu - p_sqp) * WIN_TOKENS);
                        bytes += n_valid[hf] * 2 * D * 2;
                    }
                }
                if (lane == 0) {
                    misc[1 + s] = missing;
                    if (bytes) mbar_expect_tx(bar, bytes); else mbar_arrive(bar);
                }
                __syncwarp();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    if (page[hf] >= 0) {
                        if (lane == 0) bulk_copy_g2s(dst0 + hf * REC, c.pages + page[hf] * page_row_bytes + p_head_off, REC, bar);
                    } else if (n_valid[hf] > 0) {       // up to 8 window tokens: one 256-byte row copy per lane
                        const Segment& sg = segs[p_seg];
                        const int w0 = (p_u + hf - p_sqp) * WIN_TOKENS;
                        const int r = lane & 7, which = lane >> 3;      // lanes 0-7: key rows, 8-15: value rows
                        if (lane < 16 && r < n_valid[hf]) {
                            const int w = w0 + r;
                            const long long plane = (static_cast<long long>(sg.slot) * c.n_kv + sg.h) * 2 + which;
                            const unsigned short* src;
                            if (w < sg.n_sink) src = c.sink_kv + (plane * c.s_sink + w) * D;
                            else src = c.ring_kv + (plane * c.ring_cap + (sg.recent_lo + (w - sg.n_sink)) % c.ring_cap) * D;
                            bulk_copy_g2s(dst0 + hf * REC + which * WIN_V_OFF + r * WIN_ROW, src, D * 2, bar);
                        }
                    }
                }
            }
            p_u += 2;
            ++issued;
        };
        for (int k = 0; k < TC_STAGES && k < round_tiles; ++k) issue_tile((stage + k) % TC_STAGES, warp == (k & 3));

        // ================= consumer ==============================================================
        // Software pipeline over the round's tiles: while the tensor core scores tile i+1, the warps run
        // softmax and values of tile i.  Per iteration: wait for the scores of tile i and pull them into
        // registers; write the key rows of tile i+1 (the A columns are free: the MMAs of tile i are done);
        // CTA barrier; one thread issues the MMAs of tile i+1 into the other D buffer and one warp refills
        // the stage of tile i-1; then everybody finishes tile i.
        pdl_wait();                                     // query operands come from the preparation kernel
        // tile being started (n_*) and tile being finished (f_*): segment fields live in registers
        int n_cs = -1, n_u = 0, n_u1 = 0, n_qp = 0, n_stage = stage;
        int f_cs = -1, f_u = 0, f_u1 = 0, f_qp = 0, f_qlo = 0, f_qhi = 0, f_page0 = 0, f_nwin = 0;
        long long f_bh = 0;
        float fmul = 1.f, gadd = 0.f;
        auto next_start_segment = [&]() {
            ++n_cs;
            const Segment& sg = segs[n_cs];
            n_u = sg.u0; n_u1 = sg.u1; n_qp = sg.qp;
            // the head group's e4m3 query operand into buffer n_cs & 1 (its last reader, two segments back, is done)
            const long long bh = static_cast<long long>(sg.b) * c.n_kv + sg.h;
            reinterpret_cast<uint4*>(qb + (n_cs & 1) * QB_BYTES)[tid] = __ldg(reinterpret_cast<const uint4*>(P.qb8) + bh * (QB_BYTES / 16) + tid);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        };
        auto next_finish_segment = [&]() {
            ++f_cs;
            const Segment& sg = segs[f_cs];
            f_u = sg.u0; f_u1 = sg.u1; f_qp = sg.qp; f_qlo = sg.q_lo; f_qhi = sg.q_hi; f_page0 = sg.first_page; f_nwin = sg.n_win;
            f_bh = static_cast<long long>(sg.b) * c.n_kv + sg.h;
            fmul = 1.f; gadd = 0.f;                     // unused head slots stay finite
            if (t < G) {
                const float2 v = __ldg(reinterpret_cast<const float2*>(P.qscal8 + (static_cast<long long>(sg.b) * c.n_q + sg.h * G + t) * 2));
                fmul = v.x; gadd = v.y;
            }
            st.reset();
        };
        // writes my key rows of the tile at n_u in ring slot n_stage; false if its data did not land
        auto start_tile = [&]() -> bool {
            const bool landed = __all_sync(FULL, mbar_wait_bounded(bar0 + 8 * n_stage, (phase_bits >> n_stage) & 1u));
            phase_bits ^= 1u << n_stage;
            const int my_u = n_u + half;
            if (my_u < n_u1 && my_u < n_qp && !((misc[1 + n_stage] >> half) & 1u)) {
                const unsigned rec = stage0 + n_stage * TILE + my_rec_off;
                tc_store_key_block<BITS>(rec + blk0 * CB, lane, my_tmem);
                tc_store_key_block<BITS>(rec + (blk0 + 1) * CB, lane, my_tmem + (16u << 16));
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            return landed;
        };
        auto issue_mmas = [&](int d_buf) {              // one thread
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const unsigned long long bdesc = qb_smem_desc(qb_addr + (n_cs & 1) * QB_BYTES);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const unsigned accumulate = ks > 0 ? 1u : 0u;
                asm volatile(
                    "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                    "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
                    ::"r"(tmem + TC_D_COL + 16u * d_buf), "r"(tmem + static_cast<unsigned>(8 * ks)),
                      "l"(bdesc + static_cast<unsigned long long>(ks * 2 * QB_LBO >> 4)), "r"(QK8_IDESC), "r"(accumulate) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mma_bar) : "memory");
        };
        // ---- first tile of the round
        {
            next_start_segment();
            const bool landed = start_tile();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (__syncthreads_or((!landed || misc[7] != 0u) ? 1 : 0)) aborted = true;
            if (!aborted && n_u < n_qp && tid == 0) issue_mmas(0);
        }
        next_finish_segment();
        for (int i = 0; i < round_tiles && !aborted; ++i) {
            const int s = stage;
            const int my_u = f_u + half;
            const bool tile_has_pages = f_u < f_qp;
            const bool my_page = my_u < f_u1 && my_u < f_qp && !((misc[1 + s] >> half) & 1u);
            const bool my_window = my_u < f_u1 && my_u >= f_qp;
            const unsigned rec = stage0 + s * TILE + my_rec_off;       // this warp's unit
            // ---- scores of tile i: the sums of the four e4m3 terms, rows g and g+8 of my two 16-token blocks
            float d[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
            bool scored = true;
            if (tile_has_pages) {
                scored = __all_sync(FULL, mbar_wait_bounded(mma_bar, mma_phase));
                mma_phase ^= 1u;
                if (!scored) misc[7] = 1u;                  // everybody leaves at the next barrier
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (my_page && scored) {
                    unsigned q0[8], q1[8];                  // columns 2t, 2t+1, 8+2t, 9+2t of rows g (0,1,4,5) and g+8 (2,3,6,7)
                    const unsigned dcol = TC_D_COL + 16u * (i & 1);
                    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                                 : "=r"(q0[0]), "=r"(q0[1]), "=r"(q0[2]), "=r"(q0[3]), "=r"(q0[4]), "=r"(q0[5]), "=r"(q0[6]), "=r"(q0[7])
                                 : "r"(my_tmem + dcol) : "memory");
                    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                                 : "=r"(q1[0]), "=r"(q1[1]), "=r"(q1[2]), "=r"(q1[3]), "=r"(q1[4]), "=r"(q1[5]), "=r"(q1[6]), "=r"(q1[7])
                                 : "r"(my_tmem + (16u << 16) + dcol) : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    d[0][0] = (__uint_as_float(q0[0]) + __uint_as_float(q0[1])) + (__uint_as_float(q0[4]) + __uint_as_float(q0[5]));
                    d[0][1] = (__uint_as_float(q0[2]) + __uint_as_float(q0[3])) + (__uint_as_float(q0[6]) + __uint_as_float(q0[7]));
                    d[1][0] = (__uint_as_float(q1[0]) + __uint_as_float(q1[1])) + (__uint_as_float(q1[4]) + __uint_as_float(q1[5]));
                    d[1][1] = (__uint_as_float(q1[2]) + __uint_as_float(q1[3])) + (__uint_as_float(q1[6]) + __uint_as_float(q1[7]));
                }
            }
            // ---- start tile i+1
            bool landed = true;
            const bool more = i + 1 < round_tiles;
            if (more) {
                n_u += 2;
                n_stage = (n_stage + 1 == TC_STAGES) ? 0 : n_stage + 1;
                if (n_u >= n_u1) next_start_segment();
                landed = start_tile();
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");     // my D reads and A writes precede the next MMAs
            if (__syncthreads_or((!landed || misc[7] != 0u) ? 1 : 0)) { aborted = true; break; }
            if (more && n_u < n_qp && tid == 0) issue_mmas((i + 1) & 1);
            // tiles i and i+1 are in use; the stage of tile i-1 is free now
            if (i >= 1 && issued < round_tiles) issue_tile((s + TC_STAGES - 1) % TC_STAGES, warp == (i & 3));
            // ---- finish tile i
            if (my_window && (warp & 1) == 0) {
                const int w0 = (my_u - f_qp) * WIN_TOKENS;
                window_unit<BITS, 0>(st, rec, min(WIN_TOKENS, f_nwin - w0), P.qwfrag + f_bh * 256, lane);
            }
            if (my_page && scored) {
                const int pos0 = (f_page0 + my_u) * PAGE_TOKENS;
                const bool full_page = (pos0 >= f_qlo) && (pos0 + PAGE_TOKENS <= f_qhi);
                float sc[2][2];               // [block][row g, row g+8], divided by the head multiplier
                unsigned vmeta[2][2];         // fp16x2 (Delta_v, x_min_v) of rows g, g+8
#pragma unroll
                for (int jb = 0; jb < 2; ++jb) {
                    const uint4 mt = lds128(rec + meta_offset(BITS) + 128 * (blk0 + jb) + 16 * g);   // rows g (x,y) and g+8 (z,w)
                    const float2 km_a = h2f2(mt.x), km_b = h2f2(mt.z);
                    vmeta[jb][0] = mt.y; vmeta[jb][1] = mt.w;
                    sc[jb][0] = fmaf(km_a.y, gadd, d[jb][0] * km_a.x);
                    sc[jb][1] = fmaf(km_b.y, gadd, d[jb][1] * km_b.x);
                }
                if (!full_page) {             // first / last page of the quantized range: mask the tokens outside it
#pragma unroll
                    for (int jb = 0; jb < 2; ++jb) {
                        const int p0 = pos0 + (blk0 + jb) * 16 + g, p1 = p0 + 8;
                        if (p0 < f_qlo || p0 >= f_qhi) { vmeta[jb][0] = 0u; sc[jb][0] = -INFINITY; }
                        if (p1 < f_qlo || p1 >= f_qhi) { vmeta[jb][1] = 0u; sc[jb][1] = -INFINITY; }
                    }
                }
                float mx[1];
                mx[0] = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])) * fmul;
                st.raise_max(mx);
#pragma unroll
                for (int jb = 0; jb < 2; ++jb) {
                    const int bi = blk0 + jb;
                    const float2 vm_a = h2f2(vmeta[jb][0]), vm_b = h2f2(vmeta[jb][1]);
                    const float p0 = ex2(fmaf(sc[jb][0], fmul, -st.mr[0])), p1 = ex2(fmaf(sc[jb][1], fmul, -st.mr[0]));
                    st.l[0] += p0 + p1;
                    st.z[0] = fmaf(p0, vm_a.y, fmaf(p1, vm_b.y, st.z[0]));
                    const unsigned b01 = movmatrix_trans(pack_h2(p0 * vm_a.x, 0.f)), b23 = movmatrix_trans(pack_h2(p1 * vm_b.x, 0.f));
                    if (BITS == 2) {
                        const uint4 vw = lds128(rec + v_codes_offset(2) + bi * CB + 16 * lane);
                        const unsigned sx = pre_shift<2>(vw.x), sy = pre_shift<2>(vw.y), sz = pre_shift<2>(vw.z), sw = pre_shift<2>(vw.w);
#pragma unroll
                        for (int i8 = 0; i8 < 8; ++i8)
                            mma_f16(st.o[i8], field<2>(vw.x, sx, i8), field<2>(vw.y, sy, i8), field<2>(vw.z, sz, i8), field<2>(vw.w, sw, i8), b01, b23);
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
            // ---- next tile to finish; a segment ends with its partial
            stage = (stage + 1 == TC_STAGES) ? 0 : stage + 1;
            f_u += 2;
            if (f_u >= f_u1) {
                store_partial<BITS, 0>(st, P.part + ((blockIdx.x + f_bh) * MAIN_WARPS + warp) * G * PART_STRIDE, lane, G);
                if (f_cs + 1 < n_seg) next_finish_segment();
            }
        }
    }
    if (aborted) {
        if (tid == 0) atomicOr(c.dev_status, WUSHKV_DEV_COPY_TIMEOUT);
        // give copies that may still be in flight a bounded time to land before the CTA's memory is released
        for (int k = 0; k < 1000; ++k) __nanosleep(1000);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(static_cast<unsigned>(TC_TMEM_COLS)) : "memory");
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
    bool tensor_scores;      // main kernel with the scores in tensor memory (G <= 4)
    size_t off_qfrag, off_qwfrag, off_qscal, off_plan, off_part, off_qb8, off_qscal8, total;
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool make_plan(const CacheView& c, int batch, int max_seq_len, DecodePlan& pl) {
    if (batch <= 0 || max_seq_len <= 0) return false;
    const long long pages_max = (static_cast<long long>(max_seq_len) + PAGE_TOKENS - 1) / PAGE_TOKENS + 1;
    const long long win_max = std::min<long long>(max_seq_len, c.s_sink + c.s_keep + c.s_flush - 1 + c.lag);
    const long long units_max = (pages_max + (win_max + WIN_TOKENS - 1) / WIN_TOKENS + 1) * batch * c.n_kv;
    // "tc" selects the kernel that computes the scores with tcgen05 (G <= 4 only).  It is kept as a measured
    // alternative, not the default: its four warps move in lockstep (two CTA barriers per 128 tokens), and
    // that costs more than the masks and MMA issues it saves.
    const char* path = std::getenv("WUSHKV_DECODE_PATH");
    pl.tensor_scores = c.G <= 4 && path && path[0] == 't';
    long long ctas = 0;
    if (const char* e = std::getenv("WUSHKV_DECODE_CTAS")) ctas = std::atoll(e);
    if (ctas <= 0) {
        // CTAs per SM: shared memory at 4 bits, registers for G > 4
        const long long per_sm = pl.tensor_scores ? (c.bits == 4 ? 3 : 4) : (c.bits == 4 ? 3 : (c.G <= 4 ? 4 : 3));
        ctas = std::min<long long>(per_sm * sm_count(), (units_max + 2 * MAIN_WARPS - 1) / (2 * MAIN_WARPS));
    }
    ctas = std::max<long long>(1, std::min<long long>(ctas, 1 << 20));
    pl.n_ctas = static_cast<int>(ctas);
    pl.n_warps = pl.n_ctas * MAIN_WARPS;
    const size_t bh = static_cast<size_t>(batch) * c.n_kv;
    size_t off = 0;
    pl.off_qfrag = off;  off = align_up(off + bh * 256 * sizeof(uint4), 256);
    pl.off_qwfrag = off; off = align_up(off + bh * 256 * sizeof(uint4), 256);
    pl.off_qscal = off;  off = align_up(off + static_cast<size_t>(batch) * c.n_q * 2 * sizeof(float), 256);
    pl.off_plan = off;   off = align_up(off + (static_cast<size_t>(batch) + 1) * sizeof(long long), 256);
    pl.off_part = off;   off = align_up(off + (pl.n_warps + bh * (pl.tensor_scores ? MAIN_WARPS : 1)) * c.G * PART_STRIDE * sizeof(float), 256);
    pl.off_qb8 = off;    off = align_up(off + (pl.tensor_scores ? bh * QB_BYTES : 0), 256);
    pl.off_qscal8 = off; off = align_up(off + (pl.tensor_scores ? static_cast<size_t>(batch) * c.n_q * 2 * sizeof(float) : 0), 256);
    pl.total = off;
    return true;
}

static cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;

template <int BITS, int MODE>
static int launch_decode(const DecodeParams& P, int n_ctas, cudaStream_t st) {
    constexpr int STAGES = 2;      // 4-bit records are twice as large: two stages keep three CTAs on an SM
    constexpr size_t SMEM = static_cast<size_t>(MAIN_WARPS) * STAGES * record_bytes(BITS) + MAIN_WARPS * STAGES * 8 +
                            MAIN_WARPS * MAX_SEGMENTS * sizeof(Segment);
    constexpr size_t SMEM_TC = static_cast<size_t>(TC_STAGES) * 2 * record_bytes(BITS) + 2 * QB_BYTES + (TC_STAGES + 1) * 8 + 32 +
                               MAX_SEGMENTS * sizeof(Segment);
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
    static bool smem_opted_in[64] = {};      // once per device and kernel instance
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return WUSHKV_ECUDA;
    if (dev < 0 || dev >= 64 || !smem_opted_in[dev]) {
        if (cudaFuncSetAttribute(decode_main_kernel<BITS, MODE, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM)) != cudaSuccess)
            return WUSHKV_ECUDA;
        if (MODE == 0 && cudaFuncSetAttribute(decode_main_tc_kernel<BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM_TC)) != cudaSuccess)
            return WUSHKV_ECUDA;
        if (dev >= 0 && dev < 64) smem_opted_in[dev] = true;
    }
    if (g_prof_start) cudaEventRecord(g_prof_start, st);
    cfg.gridDim = dim3(n_ctas);
    cfg.blockDim = dim3(MAIN_WARPS * 32);
    if (P.qb8 != nullptr) {
        cfg.dynamicSmemBytes = SMEM_TC;
        if (cudaLaunchKernelEx(&cfg, decode_main_tc_kernel<BITS>, P) != cudaSuccess) return WUSHKV_ECUDA;
    } else {
        cfg.dynamicSmemBytes = SMEM;
        if (cudaLaunchKernelEx(&cfg, decode_main_kernel<BITS, MODE, STAGES>, P) != cudaSuccess) return WUSHKV_ECUDA;
    }
    if (g_prof_stop) cudaEventRecord(g_prof_stop, st);
    // Partials per (sequence, KV head) are about n_warps / (batch n_kv).  Short lists go to one thread
    // group per CTA (a few rounds of COMBINE_BATCH loads); a long list (few sequences, long context)
    // is shared by 8 groups.
    const long long per_head = P.n_warps / (static_cast<long long>(P.batch) * P.c.n_kv) + 2;
    cfg.gridDim = dim3(P.c.n_q, P.batch);
    cfg.dynamicSmemBytes = 0;
    const bool shared_slices = P.slice_shift != 0;
    if (per_head <= 4 * COMBINE_BATCH) {
        cfg.blockDim = dim3(128, 1);
        if (cudaLaunchKernelEx(&cfg, shared_slices ? decode_combine_kernel<1, 2> : decode_combine_kernel<1, 0>, P) != cudaSuccess) return WUSHKV_ECUDA;
    } else {
        cfg.blockDim = dim3(128, 8);
        if (cudaLaunchKernelEx(&cfg, shared_slices ? decode_combine_kernel<8, 2> : decode_combine_kernel<8, 0>, P) != cudaSuccess) return WUSHKV_ECUDA;
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
                            void* workspace, size_t workspace_bytes, void* stream, int q_early) {
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
    P.qb8 = pl.tensor_scores ? ws + pl.off_qb8 : nullptr;
    P.qscal8 = pl.tensor_scores ? reinterpret_cast<float*>(ws + pl.off_qscal8) : nullptr;
    P.slice_shift = pl.tensor_scores ? 2 : 0;
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
                                  (P.c.bits == 2 ? record_bytes(2) : record_bytes(4));
        P.stream_pages = step_bytes > static_cast<double>(l2) ? 1 : 0;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool mode0 = P.c.G <= 4;
    if (P.c.bits == 2) return mode0 ? launch_decode<2, 0>(P, pl.n_ctas, st) : launch_decode<2, 1>(P, pl.n_ctas, st);
    return mode0 ? launch_decode<4, 0>(P, pl.n_ctas, st) : launch_decode<4, 1>(P, pl.n_ctas, st);
}

extern "C" int wushkv_decode_attn(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                  int32_t max_seq_len, const uint16_t* Q, float* O,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    return decode_attn_impl(cache, batch, slot, seq_len, max_seq_len, Q, O, workspace, workspace_bytes, stream, 0);
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
    const char* io = std::getenv("WUSHKV_HOST_IO");
    if (!(io && io[0] == 'c')) {
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
