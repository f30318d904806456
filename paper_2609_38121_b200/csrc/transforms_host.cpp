// Host-side calibration arithmetic: Gram / Hessian accumulation (Eq. 4, Algorithm 1 lines 4-5)
// and the WUSH closed form (Section 3, Eq. 1, Definition 1).  Float64 throughout; runs once per
// model at calibration time, so clarity wins over speed here.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

#include "../../include/wushkv.h"

namespace {

inline double bf16_bits_to_double(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return static_cast<double>(f);
}

// Nearest bf16-representable value (8 significand bits, ties to even), straight from float64.
double round_to_bf16(double x) {
    if (x == 0.0 || !std::isfinite(x)) return x;
    int ex;
    std::frexp(x, &ex);                 // |x| = m * 2^ex, m in [0.5, 1)
    int e = std::max(ex - 1, -126);     // subnormal range shares one quantum
    const double quantum = std::ldexp(1.0, e - 7);
    double r = std::nearbyint(x / quantum) * quantum;   // default rounding mode: ties to even
    if (std::fabs(r) > 3.3895313892515355e38) r = std::copysign(INFINITY, r);
    return r;
}

// Lower Cholesky factor of the symmetric matrix A (d x d, row-major), in place in L.  false if not PD.
bool cholesky_lower(const std::vector<double>& A, std::vector<double>& L, int d) {
    L.assign(static_cast<size_t>(d) * d, 0.0);
    for (int j = 0; j < d; ++j) {
        double s = A[j * d + j];
        for (int k = 0; k < j; ++k) s -= L[j * d + k] * L[j * d + k];
        if (!(s > 0.0) || !std::isfinite(s)) return false;
        const double ljj = std::sqrt(s);
        L[j * d + j] = ljj;
        for (int i = j + 1; i < d; ++i) {
            double t = A[i * d + j];
            for (int k = 0; k < j; ++k) t -= L[i * d + k] * L[j * d + k];
            L[i * d + j] = t / ljj;
        }
    }
    return true;
}

// Cyclic Jacobi eigensolver for a symmetric matrix: A = V diag(w) V^T, columns of V orthonormal.
void jacobi_eigh(std::vector<double> A, int d, std::vector<double>& w, std::vector<double>& V) {
    V.assign(static_cast<size_t>(d) * d, 0.0);
    for (int i = 0; i < d; ++i) V[i * d + i] = 1.0;
    for (int sweep = 0; sweep < 60; ++sweep) {
        double off = 0.0, diag = 0.0;
        for (int i = 0; i < d; ++i) {
            diag += A[i * d + i] * A[i * d + i];
            for (int j = i + 1; j < d; ++j) off += A[i * d + j] * A[i * d + j];
        }
        if (off <= 1e-30 * diag) break;
        for (int p = 0; p < d - 1; ++p) {
            for (int q = p + 1; q < d; ++q) {
                const double apq = A[p * d + q];
                if (apq == 0.0) continue;
                const double app = A[p * d + p], aqq = A[q * d + q];
                if (std::fabs(apq) < 1e-300) continue;
                const double theta = (aqq - app) / (2.0 * apq);
                const double t = (theta >= 0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
                const double c = 1.0 / std::sqrt(t * t + 1.0), s = t * c;
                for (int k = 0; k < d; ++k) {           // columns p, q
                    const double akp = A[k * d + p], akq = A[k * d + q];
                    A[k * d + p] = c * akp - s * akq;
                    A[k * d + q] = s * akp + c * akq;
                }
                for (int k = 0; k < d; ++k) {           // rows p, q
                    const double apk = A[p * d + k], aqk = A[q * d + k];
                    A[p * d + k] = c * apk - s * aqk;
                    A[q * d + k] = s * apk + c * aqk;
                }
                for (int k = 0; k < d; ++k) {
                    const double vkp = V[k * d + p], vkq = V[k * d + q];
                    V[k * d + p] = c * vkp - s * vkq;
                    V[k * d + q] = s * vkp + c * vkq;
                }
            }
        }
    }
    w.resize(d);
    for (int i = 0; i < d; ++i) w[i] = A[i * d + i];
}

// Inverse by Gauss-Jordan elimination with partial pivoting (long double). false if singular.
bool invert(const std::vector<double>& A, std::vector<double>& Ainv, int d) {
    std::vector<long double> a(static_cast<size_t>(d) * 2 * d, 0.0L);
    for (int i = 0; i < d; ++i) {
        for (int j = 0; j < d; ++j) a[i * 2 * d + j] = A[i * d + j];
        a[i * 2 * d + d + i] = 1.0L;
    }
    for (int col = 0; col < d; ++col) {
        int piv = col;
        for (int r = col + 1; r < d; ++r)
            if (fabsl(a[r * 2 * d + col]) > fabsl(a[piv * 2 * d + col])) piv = r;
        if (a[piv * 2 * d + col] == 0.0L) return false;
        if (piv != col)
            for (int j = 0; j < 2 * d; ++j) std::swap(a[piv * 2 * d + j], a[col * 2 * d + j]);
        const long double inv = 1.0L / a[col * 2 * d + col];
        for (int j = 0; j < 2 * d; ++j) a[col * 2 * d + j] *= inv;
        for (int r = 0; r < d; ++r) {
            if (r == col) continue;
            const long double f = a[r * 2 * d + col];
            if (f == 0.0L) continue;
            for (int j = 0; j < 2 * d; ++j) a[r * 2 * d + j] -= f * a[col * 2 * d + j];
        }
    }
    Ainv.resize(static_cast<size_t>(d) * d);
    for (int i = 0; i < d; ++i)
        for (int j = 0; j < d; ++j) Ainv[i * d + j] = static_cast<double>(a[i * 2 * d + d + j]);
    return true;
}

}  // namespace

extern "C" int wushkv_accumulate_gram(int32_t n_kv, int32_t n_q, int32_t d, int64_t n_tok,
                                      const uint16_t* K, const uint16_t* Q, double* M, double* H) {
    if (!K || !Q || !M || !H || n_kv <= 0 || n_q <= 0 || d <= 0 || n_tok < 0 || n_q % n_kv != 0) return WUSHKV_EINVAL;
    const int G = n_q / n_kv;
    std::vector<double> row(d);
    for (int64_t t = 0; t < n_tok; ++t) {
        for (int h = 0; h < n_kv; ++h) {
            const uint16_t* k = K + (t * n_kv + h) * d;
            for (int i = 0; i < d; ++i) row[i] = bf16_bits_to_double(k[i]);
            double* Mh = M + static_cast<size_t>(h) * d * d;
            for (int i = 0; i < d; ++i) {
                const double ki = row[i];
                for (int j = 0; j < d; ++j) Mh[i * d + j] += ki * row[j];
            }
            double* Hh = H + static_cast<size_t>(h) * d * d;
            for (int g = 0; g < G; ++g) {
                const uint16_t* q = Q + (t * n_q + h * G + g) * d;
                for (int i = 0; i < d; ++i) row[i] = bf16_bits_to_double(q[i]);
                for (int i = 0; i < d; ++i) {
                    const double qi = 2.0 * row[i];
                    for (int j = 0; j < d; ++j) Hh[i * d + j] += qi * row[j];
                }
            }
        }
    }
    return WUSHKV_OK;
}

extern "C" int wushkv_build_transforms(int32_t n_heads, int32_t d, const double* M, const double* H, double gamma,
                                       float* T, float* T_invT) {
    if (!M || !H || !T || !T_invT || n_heads <= 0 || d <= 0 || d > 1024 || (d & (d - 1)) != 0 || !(gamma >= 0.0))
        return WUSHKV_EINVAL;
    const size_t dd = static_cast<size_t>(d) * d;
    std::vector<double> Md(dd), Hd(dd), L, A(dd), tmp(dd), w, U, B(dd), Tm(dd), Tinv;
    for (int h = 0; h < n_heads; ++h) {
        const double* Mh = M + h * dd;
        const double* Hh = H + h * dd;
        double trM = 0, trH = 0;
        for (int i = 0; i < d; ++i) { trM += Mh[i * d + i]; trH += Hh[i * d + i]; }
        for (size_t i = 0; i < dd; ++i) { Md[i] = Mh[i]; Hd[i] = Hh[i]; }
        for (int i = 0; i < d; ++i) { Md[i * d + i] += gamma * trM / d; Hd[i * d + i] += gamma * trH / d; }
        if (!cholesky_lower(Hd, L, d)) return WUSHKV_ENOTPD;
        // A = L^T Md L, symmetrised
        for (int i = 0; i < d; ++i)
            for (int j = 0; j < d; ++j) {
                double s = 0;
                for (int k = 0; k < d; ++k) s += Md[i * d + k] * L[k * d + j];
                tmp[i * d + j] = s;
            }
        for (int i = 0; i < d; ++i)
            for (int j = 0; j < d; ++j) {
                double s = 0;
                for (int k = 0; k < d; ++k) s += L[k * d + i] * tmp[k * d + j];
                A[i * d + j] = s;
            }
        for (int i = 0; i < d; ++i)
            for (int j = i + 1; j < d; ++j) A[i * d + j] = A[j * d + i] = 0.5 * (A[i * d + j] + A[j * d + i]);
        jacobi_eigh(A, d, w, U);
        // canonical form: eigenvalues ascending, largest-magnitude entry of each eigenvector positive
        std::vector<int> order(d);
        std::iota(order.begin(), order.end(), 0);
        std::sort(order.begin(), order.end(), [&](int a, int b) { return w[a] < w[b]; });
        if (!(w[order[0]] > 0.0)) return WUSHKV_ENOTPD;
        double sum_sqrt = 0;
        for (int i = 0; i < d; ++i) sum_sqrt += std::sqrt(w[i]);
        const double c = std::sqrt(1.0 + gamma) * std::sqrt(trM) / std::sqrt(sum_sqrt);
        // B = Lam^(-1/4) U^T L^T  (row i from eigenvector order[i])
        for (int i = 0; i < d; ++i) {
            const int col = order[i];
            int arg = 0;
            for (int k = 1; k < d; ++k)
                if (std::fabs(U[k * d + col]) > std::fabs(U[arg * d + col])) arg = k;
            const double sgn = U[arg * d + col] < 0 ? -1.0 : 1.0;
            const double scale = sgn * std::pow(w[col], -0.25);
            for (int j = 0; j < d; ++j) {
                double s = 0;
                for (int k = 0; k < d; ++k) s += U[k * d + col] * L[j * d + k];
                B[i * d + j] = scale * s;
            }
        }
        // T = c * Had * B with the normalized Sylvester Hadamard matrix Had[i][k] = (-1)^popcount(i & k) / sqrt(d)
        const double hn = c / std::sqrt(static_cast<double>(d));
        for (int i = 0; i < d; ++i)
            for (int j = 0; j < d; ++j) {
                double s = 0;
                for (int k = 0; k < d; ++k) s += (__builtin_popcount(i & k) & 1) ? -B[k * d + j] : B[k * d + j];
                Tm[i * d + j] = round_to_bf16(hn * s);
            }
        if (!invert(Tm, Tinv, d)) return WUSHKV_ENOTPD;
        float* To = T + h * dd;
        float* Ti = T_invT + h * dd;
        for (int i = 0; i < d; ++i)
            for (int j = 0; j < d; ++j) {
                To[i * d + j] = static_cast<float>(Tm[i * d + j]);
                Ti[i * d + j] = static_cast<float>(Tinv[j * d + i]);
            }
    }
    return WUSHKV_OK;
}
