// Calibration on the GPU (Algorithm 1): streaming Gram / Hessian accumulation over calibration sequences
// (lines 4-5, Eq. 4) and the WUSH transforms of all heads from the accumulated statistics (line 7, Eq. 1,
// Definition 1).  Same results as the host entry points wushkv_accumulate_gram / wushkv_build_transforms up to
// summation order; meant for calibration sets of millions of tokens, where the host loops take hours.
//
//   gram_kernel             X^T X of one head over a slice of tokens on tensor cores (bf16 operands are the inputs
//                           themselves, products exact, fp32 accumulation within the slice), added to the float64
//                           statistics with atomics.
//   build_transforms_kernel one CTA per head, float64 throughout: damping, Cholesky, L^T M L, two-sided Jacobi
//                           eigensolver with a round-robin ordering (64 disjoint rotations per step), canonical
//                           order / sign, T = c Had Lam^(-1/4) U^T L^T rounded to bf16, Gauss-Jordan inverse of the
//                           rounded matrix.
#include <cuda_runtime.h>

#include <cmath>

#include "host_common.h"
#include "layout.cuh"

namespace wushkv {
namespace {

constexpr int GR_TOK = 64;                 // tokens per staged tile
constexpr int GR_PITCH = D + 8;            // bf16 per staged row (272 bytes: conflict-free ldmatrix)
constexpr int GR_SLICE = 2048;             // tokens per CTA
constexpr int GR_FLUSH = 128;              // tokens whose products are summed in fp32 (8 tensor-core accumulations) before they move to float64

__device__ __forceinline__ unsigned saddr(const void* p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void ldsm4t(unsigned addr, unsigned& a, unsigned& b, unsigned& c, unsigned& d) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_acc(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// grid (token slices, n_kv + n_q head slots), 256 threads: warp w owns output rows 16w .. 16w+15 (all 128 columns).
__global__ void __launch_bounds__(256) gram_kernel(int n_kv, int n_q, long long n_tok, const unsigned short* __restrict__ K,
                                                   const unsigned short* __restrict__ Q, double* M, double* H) {
    __shared__ __align__(16) unsigned short xs[GR_TOK][GR_PITCH];
    const int hs = blockIdx.y;
    const bool is_key = hs < n_kv;
    const int head = is_key ? hs : hs - n_kv, n_heads = is_key ? n_kv : n_q, G = n_q / n_kv;
    const unsigned short* X = is_key ? K : Q;
    double* out = is_key ? M + static_cast<long long>(head) * D * D : H + static_cast<long long>(head / G) * D * D;
    const double weight = is_key ? 1.0 : 2.0;                 // H = 2 sum_g sum_t q q^T (Eq. 4)
    const long long t0 = static_cast<long long>(blockIdx.x) * GR_SLICE, t1 = min(t0 + GR_SLICE, n_tok);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    float acc[16][4];
    double dacc[16][4];
#pragma unroll
    for (int nb = 0; nb < 16; ++nb) {
        acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;
        dacc[nb][0] = dacc[nb][1] = dacc[nb][2] = dacc[nb][3] = 0.0;
    }
    for (long long base = t0; base < t1; base += GR_TOK) {
        __syncthreads();
        for (int item = tid; item < GR_TOK * 16; item += 256) {          // 16-byte pieces; rows past the end are zero
            const int r = item >> 4, piece = item & 15;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (base + r < t1) v = __ldg(reinterpret_cast<const uint4*>(X + ((base + r) * n_heads + head) * D + 8 * piece));
            *reinterpret_cast<uint4*>(&xs[r][8 * piece]) = v;
        }
        __syncthreads();
#pragma unroll
        for (int ks = 0; ks < GR_TOK / 16; ++ks) {
            // A = X^T (channel x token): registers (rows i0.., tokens lo), (rows i0+8.., lo), (rows i0.., hi), (rows i0+8.., hi)
            unsigned a0, a1, a2, a3;
            ldsm4t(saddr(&xs[16 * ks + 8 * (lane >> 4) + (lane & 7)][16 * warp + 8 * ((lane >> 3) & 1)]), a0, a1, a2, a3);
#pragma unroll
            for (int nb2 = 0; nb2 < 8; ++nb2) {
                unsigned b0, b1, b2, b3;                                 // B = X (token x channel): (tokens lo, cols), (hi, cols), (lo, cols+8), (hi, cols+8)
                ldsm4t(saddr(&xs[16 * ks + 8 * ((lane >> 3) & 1) + (lane & 7)][16 * nb2 + 8 * (lane >> 4)]), b0, b1, b2, b3);
                mma_bf16_acc(acc[2 * nb2], a0, a1, a2, a3, b0, b1);
                mma_bf16_acc(acc[2 * nb2 + 1], a0, a1, a2, a3, b2, b3);
            }
        }
        if (((base - t0) / GR_TOK) % (GR_FLUSH / GR_TOK) == GR_FLUSH / GR_TOK - 1 || base + GR_TOK >= t1) {
#pragma unroll
            for (int nb = 0; nb < 16; ++nb)
#pragma unroll
                for (int e = 0; e < 4; ++e) { dacc[nb][e] += static_cast<double>(acc[nb][e]); acc[nb][e] = 0.f; }
        }
    }
#pragma unroll
    for (int nb = 0; nb < 16; ++nb) {
        const int i0 = 16 * warp + g, j0 = 8 * nb + 2 * t;
        atomicAdd(out + i0 * D + j0, weight * dacc[nb][0]);
        atomicAdd(out + i0 * D + j0 + 1, weight * dacc[nb][1]);
        atomicAdd(out + (i0 + 8) * D + j0, weight * dacc[nb][2]);
        atomicAdd(out + (i0 + 8) * D + j0 + 1, weight * dacc[nb][3]);
    }
}

// ---- float64 helpers of the transform builder -----------------------------------------------------
__device__ __forceinline__ double round_double_to_bf16(double x) {     // nearest bf16, ties to even (values in the float range)
    unsigned long long u = static_cast<unsigned long long>(__double_as_longlong(x));
    u += ((1ull << 44) - 1ull) + ((u >> 45) & 1ull);
    u &= ~((1ull << 45) - 1ull);
    return __longlong_as_double(static_cast<long long>(u));
}

constexpr int BT_THREADS = 512;

__device__ double block_sum(double v, double* red) {
    const int tid = threadIdx.x;
    __syncthreads();
    red[tid] = v;
    __syncthreads();
    for (int s = BT_THREADS / 2; s > 0; s >>= 1) {
        if (tid < s) red[tid] += red[tid + s];
        __syncthreads();
    }
    return red[0];
}

// C = A^T B (ta) or A B, all d x d row-major in global memory
__device__ void matmul(const double* A, const double* B, double* C, bool ta) {
    for (int idx = threadIdx.x; idx < D * D; idx += BT_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        double s = 0;
        for (int k = 0; k < D; ++k) s += (ta ? A[k * D + i] : A[i * D + k]) * B[k * D + j];
        C[idx] = s;
    }
    __syncthreads();
}

// One CTA per head.  ws: 8 matrices of d x d float64 per head.
__global__ void __launch_bounds__(BT_THREADS) build_transforms_kernel(const double* Mall, const double* Hall, double gamma, float* Tall,
                                                                       float* Tinvall, double* wsall, int* status) {
    __shared__ double red[BT_THREADS];
    __shared__ double w_s[D], cs_s[D / 2], sn_s[D / 2];
    __shared__ int order_s[D], pp_s[D / 2], qq_s[D / 2], ring_s[D];
    __shared__ int fail_s, piv_s;
    const int h = blockIdx.x, tid = threadIdx.x;
    const double* Mh = Mall + static_cast<long long>(h) * D * D;
    const double* Hh = Hall + static_cast<long long>(h) * D * D;
    double* ws = wsall + static_cast<long long>(h) * 8 * D * D;
    double *Md = ws, *L = ws + D * D, *A = ws + 2 * D * D, *U = ws + 3 * D * D, *B = ws + 4 * D * D, *Tm = ws + 5 * D * D, *Aug = ws + 6 * D * D;   // Aug: d x 2d
    if (tid == 0) fail_s = 0;
    // ---- damping (Definition 1)
    const double trM = block_sum(tid < D ? Mh[tid * D + tid] : 0.0, red);
    const double trH = block_sum(tid < D ? Hh[tid * D + tid] : 0.0, red);
    for (int idx = tid; idx < D * D; idx += BT_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        Md[idx] = Mh[idx] + (i == j ? gamma * trM / D : 0.0);
        L[idx] = Hh[idx] + (i == j ? gamma * trH / D : 0.0);
    }
    __syncthreads();
    // ---- Cholesky of the damped Hessian, in place (lower triangle of L)
    for (int k = 0; k < D; ++k) {
        if (tid == 0) {
            const double piv = L[k * D + k];
            if (!(piv > 0.0)) fail_s = 1;
            L[k * D + k] = piv > 0.0 ? sqrt(piv) : 1.0;
        }
        __syncthreads();
        const double dk = L[k * D + k];
        for (int i = k + 1 + tid; i < D; i += BT_THREADS) L[i * D + k] /= dk;
        __syncthreads();
        const int n = D - k - 1;
        for (int idx = tid; idx < n * n; idx += BT_THREADS) {
            const int i = k + 1 + idx / n, j = k + 1 + idx % n;
            if (j <= i) L[i * D + j] -= L[i * D + k] * L[j * D + k];
        }
        __syncthreads();
    }
    for (int idx = tid; idx < D * D; idx += BT_THREADS) if ((idx & 127) > (idx >> 7)) L[idx] = 0.0;
    __syncthreads();
    if (fail_s) { if (tid == 0) atomicOr(status, WUSHKV_ENOTPD); return; }
    // ---- A = L^T Md L, symmetrised; U = I
    matmul(Md, L, B, false);
    matmul(L, B, A, true);
    for (int idx = tid; idx < D * D; idx += BT_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        if (j > i) { const double s = 0.5 * (A[i * D + j] + A[j * D + i]); A[i * D + j] = s; A[j * D + i] = s; }
        U[idx] = (i == j) ? 1.0 : 0.0;
    }
    if (tid < D) ring_s[tid] = tid;
    __syncthreads();
    // ---- two-sided Jacobi, round-robin ordering: 127 steps of 64 disjoint rotations per sweep
    for (int sweep = 0; sweep < 30; ++sweep) {
        double off = 0.0, dia = 0.0;
        for (int idx = tid; idx < D * D; idx += BT_THREADS) {
            const double v = A[idx];
            if ((idx >> 7) == (idx & 127)) dia += v * v; else off += v * v;
        }
        off = block_sum(off, red);
        dia = block_sum(dia, red);
        if (off <= 1e-30 * dia) break;
        for (int step = 0; step < D - 1; ++step) {
            if (tid < D / 2) {                              // pair k: players ring[k] and ring[D-1-k]
                int p = ring_s[tid], q = ring_s[D - 1 - tid];
                if (p > q) { const int x = p; p = q; q = x; }
                const double apq = A[p * D + q], app = A[p * D + p], aqq = A[q * D + q];
                double c = 1.0, s = 0.0;
                if (fabs(apq) > 1e-300) {
                    const double theta = (aqq - app) / (2.0 * apq);
                    const double tt = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                    c = 1.0 / sqrt(tt * tt + 1.0);
                    s = tt * c;
                }
                pp_s[tid] = p; qq_s[tid] = q; cs_s[tid] = c; sn_s[tid] = s;
            }
            __syncthreads();
            // columns: A <- A J, U <- U J
            for (int idx = tid; idx < D * (D / 2); idx += BT_THREADS) {
                const int r = idx >> 6, k = idx & 63;
                const int p = pp_s[k], q = qq_s[k];
                const double c = cs_s[k], s = sn_s[k];
                const double ap = A[r * D + p], aq = A[r * D + q];
                A[r * D + p] = c * ap - s * aq; A[r * D + q] = s * ap + c * aq;
                const double up = U[r * D + p], uq = U[r * D + q];
                U[r * D + p] = c * up - s * uq; U[r * D + q] = s * up + c * uq;
            }
            __syncthreads();
            // rows: A <- J^T A
            for (int idx = tid; idx < D * (D / 2); idx += BT_THREADS) {
                const int col = idx >> 6, k = idx & 63;
                const int p = pp_s[k], q = qq_s[k];
                const double c = cs_s[k], s = sn_s[k];
                const double ap = A[p * D + col], aq = A[q * D + col];
                A[p * D + col] = c * ap - s * aq; A[q * D + col] = s * ap + c * aq;
            }
            __syncthreads();
            if (tid == 0) {                                  // rotate the tournament: player ring[0] stays
                const int last = ring_s[D - 1];
                for (int k = D - 1; k > 1; --k) ring_s[k] = ring_s[k - 1];
                ring_s[1] = last;
            }
            __syncthreads();
        }
    }
    // ---- canonical form: eigenvalues ascending, largest-magnitude entry of each eigenvector positive
    if (tid < D) w_s[tid] = A[tid * D + tid];
    __syncthreads();
    if (tid < D) {
        int rank = 0;
        for (int j = 0; j < D; ++j) rank += (w_s[j] < w_s[tid]) || (w_s[j] == w_s[tid] && j < tid);
        order_s[rank] = tid;
        if (!(w_s[tid] > 0.0)) fail_s = 1;
    }
    __syncthreads();
    if (fail_s) { if (tid == 0) atomicOr(status, WUSHKV_ENOTPD); return; }
    const double sum_sqrt = block_sum(tid < D ? sqrt(w_s[tid]) : 0.0, red);
    const double c_norm = sqrt(1.0 + gamma) * sqrt(trM) / sqrt(sum_sqrt);
    if (tid < D) {                                           // sign and scale of row tid of Lam^(-1/4) U^T
        const int col = order_s[tid];
        int arg = 0;
        for (int k = 1; k < D; ++k) if (fabs(U[k * D + col]) > fabs(U[arg * D + col])) arg = k;
        red[tid] = (U[arg * D + col] < 0 ? -1.0 : 1.0) * pow(w_s[col], -0.25);
    }
    __syncthreads();
    // B = Lam^(-1/4) U^T L^T: B[i][j] = scale_i sum_k U[k][col_i] L[j][k]
    for (int idx = tid; idx < D * D; idx += BT_THREADS) {
        const int i = idx >> 7, j = idx & 127, col = order_s[i];
        double s = 0;
        for (int k = 0; k < D; ++k) s += U[k * D + col] * L[j * D + k];
        B[idx] = red[i] * s;
    }
    __syncthreads();
    // T = c Had B (normalized Sylvester Hadamard), rounded to bf16
    const double hn = c_norm / sqrt(static_cast<double>(D));
    float* To = Tall + static_cast<long long>(h) * D * D;
    for (int idx = tid; idx < D * D; idx += BT_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        double s = 0;
        for (int k = 0; k < D; ++k) s += (__popc(i & k) & 1) ? -B[k * D + j] : B[k * D + j];
        const double v = round_double_to_bf16(hn * s);
        Tm[idx] = v;
        To[idx] = static_cast<float>(v);
    }
    __syncthreads();
    // ---- inverse of the rounded T: Gauss-Jordan with partial pivoting on [T | I]
    for (int idx = tid; idx < D * 2 * D; idx += BT_THREADS) {
        const int i = idx / (2 * D), j = idx % (2 * D);
        Aug[idx] = j < D ? Tm[i * D + j] : ((j - D) == i ? 1.0 : 0.0);
    }
    __syncthreads();
    for (int col = 0; col < D; ++col) {
        if (tid == 0) {
            int piv = col;
            for (int r = col + 1; r < D; ++r) if (fabs(Aug[r * 2 * D + col]) > fabs(Aug[piv * 2 * D + col])) piv = r;
            piv_s = piv;
            if (Aug[piv * 2 * D + col] == 0.0) fail_s = 1;
        }
        __syncthreads();
        if (fail_s) { if (tid == 0) atomicOr(status, WUSHKV_ENOTPD); return; }
        const int piv = piv_s;
        if (piv != col)
            for (int j = tid; j < 2 * D; j += BT_THREADS) { const double x = Aug[piv * 2 * D + j]; Aug[piv * 2 * D + j] = Aug[col * 2 * D + j]; Aug[col * 2 * D + j] = x; }
        __syncthreads();
        const double inv = 1.0 / Aug[col * 2 * D + col];
        __syncthreads();
        for (int j = tid; j < 2 * D; j += BT_THREADS) Aug[col * 2 * D + j] *= inv;
        __syncthreads();
        if (tid < D) red[tid] = Aug[tid * 2 * D + col];      // the column being eliminated, before it changes
        __syncthreads();
        for (int idx = tid; idx < D * 2 * D; idx += BT_THREADS) {
            const int r = idx / (2 * D), j = idx % (2 * D);
            if (r != col) Aug[idx] -= red[r] * Aug[col * 2 * D + j];
        }
        __syncthreads();
    }
    float* Ti = Tinvall + static_cast<long long>(h) * D * D;
    for (int idx = tid; idx < D * D; idx += BT_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        Ti[idx] = static_cast<float>(Aug[j * 2 * D + D + i]);      // (T^-1)^T
    }
}

}  // namespace
}  // namespace wushkv

using namespace wushkv;

extern "C" int wushkv_accumulate_gram_device(int32_t n_kv, int32_t n_q, int32_t d, int64_t n_tok, const uint16_t* K, const uint16_t* Q,
                                             double* M, double* H, void* stream) {
    if (!K || !Q || !M || !H || n_kv <= 0 || n_q <= 0 || d != D || n_tok < 0 || n_q % n_kv != 0) return WUSHKV_EINVAL;
    if (!aligned(K, 16) || !aligned(Q, 16) || !aligned(M, 8) || !aligned(H, 8)) return WUSHKV_EINVAL;
    if (n_tok == 0) return WUSHKV_OK;
    const long long slices = (n_tok + GR_SLICE - 1) / GR_SLICE;
    if (slices > 0x7fffffffLL) return WUSHKV_EINVAL;
    gram_kernel<<<dim3(static_cast<unsigned>(slices), n_kv + n_q), 256, 0, static_cast<cudaStream_t>(stream)>>>(n_kv, n_q, n_tok, K, Q, M, H);
    return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
}

extern "C" size_t wushkv_build_transforms_workspace_bytes(int32_t n_heads, int32_t d) {
    if (n_heads <= 0 || d != D) return 0;
    return static_cast<size_t>(n_heads) * 8 * D * D * sizeof(double);
}

extern "C" int wushkv_build_transforms_device(int32_t n_heads, int32_t d, const double* M, const double* H, double gamma,
                                              float* T, float* T_invT, int32_t* dev_status, void* workspace, size_t workspace_bytes,
                                              void* stream) {
    if (!M || !H || !T || !T_invT || !dev_status || !workspace || n_heads <= 0 || d != D || !(gamma >= 0.0)) return WUSHKV_EINVAL;
    if (!aligned(M, 8) || !aligned(H, 8) || !aligned(workspace, 16)) return WUSHKV_EINVAL;
    if (workspace_bytes < wushkv_build_transforms_workspace_bytes(n_heads, d)) return WUSHKV_ECAPACITY;
    build_transforms_kernel<<<n_heads, BT_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(M, H, gamma, T, T_invT, static_cast<double*>(workspace), dev_status);
    return cudaGetLastError() == cudaSuccess ? WUSHKV_OK : WUSHKV_ECUDA;
}
