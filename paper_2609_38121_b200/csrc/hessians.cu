// Attention-aware Hessians on the GPU (Appendix C, "Aggregation for WUSH-A"): for one calibration sequence and
// every key/value head h, the key and value Hessians summed over the perturbed position s,
//   H_K(h) = (2 / tau^2) sum_t sum_{g,g'} A_{gg'}(t) q_{g,t} q_{g',t}^T,
//   A_{gg'}(t) = sum_{s<=t} p_{g,t,s} p_{g',t,s} (v_s - o_{g,t})^T Gamma_{gg'} (v_s - o_{g',t}),
//   H_V(h) = 2 sum_{g,g'} (sum_t sum_{s<=t} p_{g,t,s} p_{g',t,s}) Gamma_{gg'},     Gamma_{gg'} = W_O(h,g) W_O(h,g')^T,
// which is the appendix's key / value Hessian with the sums over s and t exchanged.  Expanding the bilinear form,
//   A_{gg'}(t) = W2 - W1 . (Gamma_{gg'} o_{g',t}) - W1 . (Gamma_{g'g} o_{g,t}) + W0 o_{g,t} . (Gamma_{gg'} o_{g',t}),
//   W0 = sum_s w_s,  W1 = sum_s w_s v_s,  W2 = sum_s w_s (v_s^T Gamma_{gg'} v_s),  w_s = p_{g,t,s} p_{g',t,s},
// so one pass over the causal probabilities with attention-like reductions suffices; A_{gg'} = A_{g'g}.
//
// Five small kernels, fp32 arithmetic with float64 accumulation of the final sums (calibration is offline: clarity
// and exactness before speed; cost O(S^2 G^2 d) per head):
//   gamma_kernel      Gamma_{gg'} for all ordered pairs
//   rows_kernel       causal softmax statistics (max, 1 / sum) and head outputs o_{g,t}
//   project_kernel    u_{gg'}(t) = Gamma_{gg'} o_{g',t} and alpha_{gg'}(s) = v_s^T Gamma_{gg'} v_s
//   pairs_kernel      W0, W1, W2 per (t, pair g <= g'), then A_{gg'}(t)
//   reduce_kernel     H_K and H_V (float64, added to the caller's accumulators)
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>

#include "host_common.h"
#include "layout.cuh"

namespace wushkv {
namespace {

constexpr int HS_TILE = 32;                // cache positions per staged tile
constexpr int HS_PITCH = D + 4;            // floats per staged row

struct HessParams {
    int S, n_kv, n_q, G, d_model, n_pairs;
    float inv_tau;
    const unsigned short* Q;     // [S][n_q][D] bf16
    const unsigned short* K;     // [S][n_kv][D]
    const unsigned short* V;     // [S][n_kv][D]
    const float* W_O;            // [n_q][D][d_model]
    float* gamma;                // [n_kv][G][G][D][D]
    float* row_m;                // [S][n_q] running maximum of the logits (natural log domain)
    float* row_linv;             // [S][n_q] 1 / sum exp
    float* Oh;                   // [S][n_q][D]
    float* U;                    // [S][n_kv][G][G][D]   u_{gg'}(t) = Gamma_{gg'} o_{g',t}
    float* alpha;                // [S][n_kv][G][G]
    float* A;                    // [S][n_kv][n_pairs]   pairs g <= g' in row-major order
    float* W0;                   // [S][n_kv][n_pairs]
    double* H_K;                 // [n_kv][D][D]
    double* H_V;
};

// Gamma_{gg'}[i][j] = sum_m W_g[i][m] W_g'[j][m]; grid (D/16, D/16, n_kv*G*G), 16 x 16 threads.
__global__ void __launch_bounds__(256) gamma_kernel(HessParams P) {
    __shared__ float a_s[16][17], b_s[16][17];
    const int z = blockIdx.z, h = z / (P.G * P.G), g = (z / P.G) % P.G, gp = z % P.G;
    const float* Wa = P.W_O + static_cast<long long>(h * P.G + g) * D * P.d_model;
    const float* Wb = P.W_O + static_cast<long long>(h * P.G + gp) * D * P.d_model;
    const int tx = threadIdx.x, ty = threadIdx.y, i = blockIdx.y * 16 + ty, j = blockIdx.x * 16 + tx;
    double acc = 0.0;
    for (int m0 = 0; m0 < P.d_model; m0 += 16) {
        a_s[ty][tx] = m0 + tx < P.d_model ? Wa[static_cast<long long>(blockIdx.y * 16 + ty) * P.d_model + m0 + tx] : 0.f;
        b_s[ty][tx] = m0 + tx < P.d_model ? Wb[static_cast<long long>(blockIdx.x * 16 + ty) * P.d_model + m0 + tx] : 0.f;
        __syncthreads();
        float part = 0.f;
#pragma unroll
        for (int m = 0; m < 16; ++m) part = fmaf(a_s[ty][m], b_s[tx][m], part);
        acc += static_cast<double>(part);
        __syncthreads();
    }
    P.gamma[(static_cast<long long>(z) * D + i) * D + j] = static_cast<float>(acc);
}

// One warp per (t, query head): causal softmax statistics and o = sum_s p_s v_s.  grid (S, n_kv), G warps.
__global__ void rows_kernel(HessParams P) {
    const int t = blockIdx.x, h = blockIdx.y, g = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = h * P.G + g;
    const unsigned short* qrow = P.Q + (static_cast<long long>(t) * P.n_q + j) * D;
    float q[4];
    {
        const uint2 raw = *reinterpret_cast<const uint2*>(qrow + 4 * lane);
        q[0] = bf16_bits_to_float(raw.x & 0xffff); q[1] = bf16_bits_to_float(raw.x >> 16);
        q[2] = bf16_bits_to_float(raw.y & 0xffff); q[3] = bf16_bits_to_float(raw.y >> 16);
    }
    float m = -INFINITY, l = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s <= t; ++s) {
        const uint2 kr = __ldg(reinterpret_cast<const uint2*>(P.K + (static_cast<long long>(s) * P.n_kv + h) * D) + lane);
        float part = q[0] * bf16_bits_to_float(kr.x & 0xffff) + q[1] * bf16_bits_to_float(kr.x >> 16) +
                     q[2] * bf16_bits_to_float(kr.y & 0xffff) + q[3] * bf16_bits_to_float(kr.y >> 16);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
        const float z = part * P.inv_tau;
        const float mn = fmaxf(m, z);
        const float sc = __expf(m - mn), p = __expf(z - mn);
        const uint2 vr = __ldg(reinterpret_cast<const uint2*>(P.V + (static_cast<long long>(s) * P.n_kv + h) * D) + lane);
        l = l * sc + p;
        o[0] = o[0] * sc + p * bf16_bits_to_float(vr.x & 0xffff); o[1] = o[1] * sc + p * bf16_bits_to_float(vr.x >> 16);
        o[2] = o[2] * sc + p * bf16_bits_to_float(vr.y & 0xffff); o[3] = o[3] * sc + p * bf16_bits_to_float(vr.y >> 16);
        m = mn;
    }
    const float linv = 1.f / l;
    if (lane == 0) { P.row_m[static_cast<long long>(t) * P.n_q + j] = m; P.row_linv[static_cast<long long>(t) * P.n_q + j] = linv; }
    *reinterpret_cast<float4*>(P.Oh + (static_cast<long long>(t) * P.n_q + j) * D + 4 * lane) = make_float4(o[0] * linv, o[1] * linv, o[2] * linv, o[3] * linv);
}

// y = Gamma x for a 128-vector x held as 4 values per lane; returns y[r0 + lane] for the 32 rows r0.. in turn.
__device__ __noinline__ void gamma_matvec(const float* gam, const float (&x)[4], int lane, float (&y)[4]) {
#pragma unroll 1
    for (int blk = 0; blk < 4; ++blk) {
        float part[32];
#pragma unroll
        for (int r = 0; r < 32; ++r) {
            const float4 gr = __ldg(reinterpret_cast<const float4*>(gam + static_cast<long long>(32 * blk + r) * D) + lane);
            part[r] = fmaf(gr.x, x[0], fmaf(gr.y, x[1], fmaf(gr.z, x[2], gr.w * x[3])));
        }
        const float tot = warp_transpose_reduce(part, lane);  // lane L: y[32 blk + L]
        if (blk == 0) y[0] = tot; else if (blk == 1) y[1] = tot; else if (blk == 2) y[2] = tot; else y[3] = tot;
    }
}

// One warp per (position, ordered pair): u_{gg'}(t) = Gamma_{gg'} o_{g',t} and alpha_{gg'}(s) = v_s . Gamma_{gg'} v_s.
// grid (S, n_kv), up to 16 warps that share the G*G ordered pairs.
__global__ void project_kernel(HessParams P) {
    const int t = blockIdx.x, h = blockIdx.y, lane = threadIdx.x & 31;
    for (int w = threadIdx.x >> 5; w < P.G * P.G; w += blockDim.x >> 5) {
    const int g = w / P.G, gp = w % P.G;
    const float* gam = P.gamma + (static_cast<long long>(h * P.G + g) * P.G + gp) * D * D;
    float x[4], y[4];
    {
        const float4 o = *reinterpret_cast<const float4*>(P.Oh + (static_cast<long long>(t) * P.n_q + h * P.G + gp) * D + 4 * lane);
        x[0] = o.x; x[1] = o.y; x[2] = o.z; x[3] = o.w;
    }
    gamma_matvec(gam, x, lane, y);
    float* u = P.U + ((static_cast<long long>(t) * P.n_kv + h) * P.G * P.G + w) * D;
#pragma unroll
    for (int blk = 0; blk < 4; ++blk) u[32 * blk + lane] = y[blk];
    {
        const uint2 vr = *reinterpret_cast<const uint2*>(P.V + (static_cast<long long>(t) * P.n_kv + h) * D + 4 * lane);
        x[0] = bf16_bits_to_float(vr.x & 0xffff); x[1] = bf16_bits_to_float(vr.x >> 16);
        x[2] = bf16_bits_to_float(vr.y & 0xffff); x[3] = bf16_bits_to_float(vr.y >> 16);
    }
    gamma_matvec(gam, x, lane, y);
    // v . y: lane L holds y[32 blk + L]; the matching v entries are fetched one by one
    float dot = 0.f;
#pragma unroll
    for (int blk = 0; blk < 4; ++blk)
        dot = fmaf(y[blk], bf16_bits_to_float(P.V[(static_cast<long long>(t) * P.n_kv + h) * D + 32 * blk + lane]), dot);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    if (lane == 0) P.alpha[(static_cast<long long>(t) * P.n_kv + h) * P.G * P.G + w] = dot;
    }
}

// One CTA of 128 threads (one per channel) per (t, h): the pair sums W0, W1, W2 over s <= t, then A_{gg'}(t).
template <int G>
__global__ void __launch_bounds__(128) pairs_kernel(HessParams P) {
    constexpr int NP = G * (G + 1) / 2;
    __shared__ float k_s[HS_TILE][HS_PITCH], v_s[HS_TILE][HS_PITCH];
    __shared__ float q_s[G][D];
    __shared__ float p_s[G][HS_TILE];
    __shared__ float al_s[HS_TILE][G * G];
    __shared__ float red_s[4][3 * NP];
    const int t = blockIdx.x, h = blockIdx.y, c = threadIdx.x, lane = c & 31, warp = c >> 5;
    for (int g = 0; g < G; ++g) q_s[g][c] = bf16_bits_to_float(P.Q[(static_cast<long long>(t) * P.n_q + h * G + g) * D + c]);
    float w1[NP];
    float w0 = 0.f, w2 = 0.f;            // thread `pair` (< NP) accumulates W0 and W2 of its pair
#pragma unroll
    for (int k = 0; k < NP; ++k) w1[k] = 0.f;
    int my_g = 0, my_gp = 0;
    if (c < NP) { int k = c; while (k >= G - my_g) { k -= G - my_g; ++my_g; } my_gp = my_g + k; }
    for (int s0 = 0; s0 <= t; s0 += HS_TILE) {
        __syncthreads();
        const int n = min(HS_TILE, t + 1 - s0);
        for (int r = 0; r < HS_TILE; ++r) {
            const bool in = r < n;
            k_s[r][c] = in ? bf16_bits_to_float(P.K[(static_cast<long long>(s0 + r) * P.n_kv + h) * D + c]) : 0.f;
            v_s[r][c] = in ? bf16_bits_to_float(P.V[(static_cast<long long>(s0 + r) * P.n_kv + h) * D + c]) : 0.f;
        }
        for (int idx = c; idx < HS_TILE * G * G; idx += 128) {
            const int r = idx / (G * G);
            al_s[r][idx % (G * G)] = r < n ? P.alpha[(static_cast<long long>(s0 + r) * P.n_kv + h) * G * G + idx % (G * G)] : 0.f;
        }
        __syncthreads();
        // probabilities: warp w takes (g, s) items w, w + 4, ...
        for (int item = warp; item < G * HS_TILE; item += 4) {
            const int g = item / HS_TILE, r = item % HS_TILE;
            float part = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) part = fmaf(q_s[g][lane + 32 * e], k_s[r][lane + 32 * e], part);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
            if (lane == 0) {
                const long long row = static_cast<long long>(t) * P.n_q + h * G + g;
                p_s[g][r] = r < n ? __expf(part * P.inv_tau - P.row_m[row]) * P.row_linv[row] : 0.f;
            }
        }
        __syncthreads();
        for (int r = 0; r < n; ++r) {
            const float v = v_s[r][c];
            int k = 0;
#pragma unroll
            for (int g = 0; g < G; ++g)
#pragma unroll
                for (int gp = g; gp < G; ++gp, ++k) w1[k] = fmaf(p_s[g][r] * p_s[gp][r], v, w1[k]);
        }
        if (c < NP)
            for (int r = 0; r < n; ++r) {
                const float w = p_s[my_g][r] * p_s[my_gp][r];
                w0 += w;
                w2 = fmaf(w, al_s[r][my_g * G + my_gp], w2);
            }
    }
    // A_{gg'} = W2 - W1 . u_{gg'} - W1 . u_{g'g} + W0 (o_g . u_{gg'}): three channel-wise dot products per pair
    const float* Ubase = P.U + (static_cast<long long>(t) * P.n_kv + h) * G * G * D;
    float d1[NP], d2[NP], d3[NP];
    {
        int k = 0;
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int gp = g; gp < G; ++gp, ++k) {
                const float u_a = Ubase[(g * G + gp) * D + c], u_b = Ubase[(gp * G + g) * D + c];
                const float og = P.Oh[(static_cast<long long>(t) * P.n_q + h * G + g) * D + c];
                d1[k] = w1[k] * u_a; d2[k] = w1[k] * u_b; d3[k] = og * u_a;
            }
    }
#pragma unroll
    for (int k = 0; k < NP; ++k) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            d1[k] += __shfl_xor_sync(0xffffffffu, d1[k], off);
            d2[k] += __shfl_xor_sync(0xffffffffu, d2[k], off);
            d3[k] += __shfl_xor_sync(0xffffffffu, d3[k], off);
        }
        if (lane == 0) { red_s[warp][3 * k] = d1[k]; red_s[warp][3 * k + 1] = d2[k]; red_s[warp][3 * k + 2] = d3[k]; }
    }
    __syncthreads();
    if (c < NP) {
        float s1 = 0.f, s2 = 0.f, s3 = 0.f;
        for (int w = 0; w < 4; ++w) { s1 += red_s[w][3 * c]; s2 += red_s[w][3 * c + 1]; s3 += red_s[w][3 * c + 2]; }
        const long long o = (static_cast<long long>(t) * P.n_kv + h) * NP + c;
        P.A[o] = w2 - s1 - s2 + w0 * s3;
        P.W0[o] = w0;
    }
}

// H_K[h][i][j] += (2 / tau^2) sum_t sum_{g<=g'} A(t) sym(q_g[i] q_g'[j]);  H_V[h][i][j] += 2 sum_{g<=g'} c sym(Gamma_{gg'}[i][j]),
// c = sum_t W0(t).  grid (D/16, D/16, n_kv), 16 x 16 threads; float64 accumulation.
template <int G>
__global__ void __launch_bounds__(256) reduce_kernel(HessParams P) {
    constexpr int NP = G * (G + 1) / 2;
    __shared__ float qi_s[G][16], qj_s[G][16], a_s[NP];
    __shared__ double c_s[NP];
    const int h = blockIdx.z, tx = threadIdx.x, ty = threadIdx.y, tid = ty * 16 + tx;
    const int i = blockIdx.y * 16 + ty, j = blockIdx.x * 16 + tx;
    double hk = 0.0;
    double csum = 0.0;                   // threads < NP: their pair's sum of W0
    for (int t = 0; t < P.S; ++t) {
        __syncthreads();
        if (tid < G * 16) qi_s[tid / 16][tid % 16] = bf16_bits_to_float(P.Q[(static_cast<long long>(t) * P.n_q + h * G + tid / 16) * D + blockIdx.y * 16 + tid % 16]);
        else if (tid < 2 * G * 16) { const int u = tid - G * 16; qj_s[u / 16][u % 16] = bf16_bits_to_float(P.Q[(static_cast<long long>(t) * P.n_q + h * G + u / 16) * D + blockIdx.x * 16 + u % 16]); }
        if (tid < NP) {
            a_s[tid] = P.A[(static_cast<long long>(t) * P.n_kv + h) * NP + tid];
            csum += static_cast<double>(P.W0[(static_cast<long long>(t) * P.n_kv + h) * NP + tid]);
        }
        __syncthreads();
        float part = 0.f;
        int k = 0;
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int gp = g; gp < G; ++gp, ++k) {
                const float outer = g == gp ? qi_s[g][ty] * qj_s[g][tx] : qi_s[g][ty] * qj_s[gp][tx] + qi_s[gp][ty] * qj_s[g][tx];
                part = fmaf(a_s[k], outer, part);
            }
        hk += static_cast<double>(part);
    }
    __syncthreads();
    if (tid < NP) c_s[tid] = csum;
    __syncthreads();
    double hv = 0.0;
    {
        int k = 0;
        for (int g = 0; g < G; ++g)
            for (int gp = g; gp < G; ++gp, ++k) {
                const float* gam = P.gamma + (static_cast<long long>(h * G + g) * G + gp) * D * D;
                const float* gamT = P.gamma + (static_cast<long long>(h * G + gp) * G + g) * D * D;
                const double sym = g == gp ? static_cast<double>(gam[i * D + j]) : static_cast<double>(gam[i * D + j]) + static_cast<double>(gamT[i * D + j]);
                hv += c_s[k] * sym;
            }
    }
    const long long o = (static_cast<long long>(h) * D + i) * D + j;
    P.H_K[o] += 2.0 * static_cast<double>(P.inv_tau) * static_cast<double>(P.inv_tau) * hk;
    P.H_V[o] += 2.0 * hv;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct HessLayout { size_t gamma, row_m, row_linv, Oh, U, alpha, A, W0, total; };
HessLayout hess_layout(int n_kv, int n_q, long long S) {
    const int G = n_q / n_kv, NP = G * (G + 1) / 2;
    HessLayout L;
    size_t off = 0;
    L.gamma = off;    off = align256(off + static_cast<size_t>(n_kv) * G * G * D * D * sizeof(float));
    L.row_m = off;    off = align256(off + static_cast<size_t>(S) * n_q * sizeof(float));
    L.row_linv = off; off = align256(off + static_cast<size_t>(S) * n_q * sizeof(float));
    L.Oh = off;       off = align256(off + static_cast<size_t>(S) * n_q * D * sizeof(float));
    L.U = off;        off = align256(off + static_cast<size_t>(S) * n_kv * G * G * D * sizeof(float));
    L.alpha = off;    off = align256(off + static_cast<size_t>(S) * n_kv * G * G * sizeof(float));
    L.A = off;        off = align256(off + static_cast<size_t>(S) * n_kv * NP * sizeof(float));
    L.W0 = off;       off = align256(off + static_cast<size_t>(S) * n_kv * NP * sizeof(float));
    L.total = off;
    return L;
}

}  // namespace
}  // namespace wushkv

using namespace wushkv;

extern "C" size_t wushkv_attention_hessians_workspace_bytes(int32_t n_kv, int32_t n_q, int32_t d, int64_t n_tokens) {
    if (d != D || n_kv <= 0 || n_q <= 0 || n_q % n_kv != 0 || n_q / n_kv > 8 || n_tokens <= 0) return 0;
    return hess_layout(n_kv, n_q, n_tokens).total;
}

extern "C" int wushkv_accumulate_attention_hessians_device(int32_t n_kv, int32_t n_q, int32_t d, int32_t d_model, int64_t n_tokens,
                                                           const uint16_t* K, const uint16_t* Q, const uint16_t* V, const float* W_O,
                                                           double tau, double* H_K, double* H_V,
                                                           void* workspace, size_t workspace_bytes, void* stream) {
    if (d != D || n_kv <= 0 || n_q <= 0 || n_q % n_kv != 0 || d_model <= 0 || n_tokens <= 0 || n_tokens > (1 << 24)) return WUSHKV_EINVAL;
    const int G = n_q / n_kv;
    if (G > 8) return WUSHKV_EINVAL;          // the library's group sizes: 1..8
    if (!K || !Q || !V || !W_O || !H_K || !H_V || !workspace || !(tau > 0.0)) return WUSHKV_EINVAL;
    if (!aligned(K, 16) || !aligned(Q, 16) || !aligned(V, 16) || !aligned(W_O, 16) || !aligned(workspace, 256)) return WUSHKV_EINVAL;
    const HessLayout L = hess_layout(n_kv, n_q, n_tokens);
    if (workspace_bytes < L.total) return WUSHKV_ECAPACITY;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    HessParams P;
    P.S = static_cast<int>(n_tokens); P.n_kv = n_kv; P.n_q = n_q; P.G = G; P.d_model = d_model; P.n_pairs = G * (G + 1) / 2;
    P.inv_tau = static_cast<float>(1.0 / tau);
    P.Q = Q; P.K = K; P.V = V; P.W_O = W_O;
    P.gamma = reinterpret_cast<float*>(ws + L.gamma);
    P.row_m = reinterpret_cast<float*>(ws + L.row_m); P.row_linv = reinterpret_cast<float*>(ws + L.row_linv);
    P.Oh = reinterpret_cast<float*>(ws + L.Oh); P.U = reinterpret_cast<float*>(ws + L.U);
    P.alpha = reinterpret_cast<float*>(ws + L.alpha); P.A = reinterpret_cast<float*>(ws + L.A); P.W0 = reinterpret_cast<float*>(ws + L.W0);
    P.H_K = H_K; P.H_V = H_V;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    gamma_kernel<<<dim3(D / 16, D / 16, n_kv * G * G), dim3(16, 16), 0, st>>>(P);
    rows_kernel<<<dim3(P.S, n_kv), 32 * G, 0, st>>>(P);
    project_kernel<<<dim3(P.S, n_kv), 32 * std::min(G * G, 16), 0, st>>>(P);
    const dim3 grid_t(P.S, n_kv), grid_r(D / 16, D / 16, n_kv);
    switch (G) {
        case 1: pairs_kernel<1><<<grid_t, 128, 0, st>>>(P); reduce_kernel<1><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        case 2: pairs_kernel<2><<<grid_t, 128, 0, st>>>(P); reduce_kernel<2><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        case 3: pairs_kernel<3><<<grid_t, 128, 0, st>>>(P); reduce_kernel<3><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        case 4: pairs_kernel<4><<<grid_t, 128, 0, st>>>(P); reduce_kernel<4><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        case 5: pairs_kernel<5><<<grid_t, 128, 0, st>>>(P); reduce_kernel<5><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        case 6: pairs_kernel<6><<<grid_t, 128, 0, st>>>(P); reduce_kernel<6><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        case 7: pairs_kernel<7><<<grid_t, 128, 0, st>>>(P); reduce_kernel<7><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
        default: pairs_kernel<8><<<grid_t, 128, 0, st>>>(P); reduce_kernel<8><<<grid_r, dim3(16, 16), 0, st>>>(P); break;
    }
    return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
}
