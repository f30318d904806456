"""Float64 CPU oracle for the WUSH-KV serving hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Nothing in the product path may import it:
only the tests, the smoke check and the CPU-baseline leg of the benchmark do.
It shares no code, table or constant with the CUDA sources and never imports
the package that wraps them.

Every function cites the passage of the WUSH-KV paper it follows.  Where the
paper leaves a choice open the reading taken here is stated in the docstring.
All arithmetic is numpy float64 unless a storage precision is part of the
method's data format (bf16 transforms and windows, fp16 scale / zero).

Conventions
-----------
* ``d`` is the head dimension.  Vectors are stored as rows ``[token][channel]``;
  the paper's column convention ``k' = T k`` is ``k'_row = k_row @ T.T`` here.
* ``T`` is always the paper's ``T`` stored row-major ``[out][in]``.
* Positions are 0-based; the paper's ``S_start < s <= S_quant`` (1-based) is
  the 0-based half-open range ``[S_start, S_quant)``.

Parity pins (tests/test_oracle_*.py, tests/test_golden.py) cover every function below (the error metric
and the quantize-from-bf16 reading in test_oracle_attention.py, the QuEST quantizer in test_oracle_quest.py,
chunk attention in test_oracle_chunk_attn.py, Norm and RoPE in test_oracle_prologue.py, the attention-aware Hessians in test_oracle_hessians.py); none is "parity unpinned" against the mathematics.  What the paper itself does not fix
(quantile interpolation rule, tie rounding, storage precision of scale and
zero, the boundary used at attention time) cannot be pinned to the paper; each
such reading is listed where it is taken.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# storage-precision helpers
# --------------------------------------------------------------------------


def round_bf16(x):
    """Round float64 values to the nearest bfloat16 (8 significand bits,
    ties to even) and return them as float64.  Single rounding straight from
    float64: the value is scaled so that one bf16 ulp is 1, rounded with
    ``rint`` and scaled back.  bf16 subnormals and overflow follow IEEE rules
    for the 8-bit-exponent format."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = np.isfinite(x) & (x != 0.0)
    if np.any(nz):
        v = x[nz]
        _, ex = np.frexp(v)                  # |v| = m * 2**ex, m in [0.5, 1)
        e = ex - 1                           # |v| in [2**e, 2**(e+1))
        e = np.maximum(e, -126)              # subnormal range shares one quantum
        quantum = np.ldexp(1.0, e - 7)       # 7 fraction bits
        r = np.rint(v / quantum) * quantum
        big = np.abs(r) > 3.3895313892515355e38   # largest finite bf16
        r = np.where(big, np.sign(r) * np.inf, r)
        out[nz] = r
    out[~np.isfinite(x)] = x[~np.isfinite(x)]
    return out


def round_fp16(x):
    """Round float64 values to the nearest IEEE binary16 (ties to even),
    saturating at the largest finite half (65504) instead of overflowing,
    and return them as float64."""
    x = np.asarray(x, dtype=np.float64)
    clipped = np.clip(x, -65504.0, 65504.0)
    return clipped.astype(np.float16).astype(np.float64)


def round_fp32(x):
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


# --------------------------------------------------------------------------
# WUSH transform  (Section 3, Eq. 1, Definition 1)
# --------------------------------------------------------------------------


def hadamard(d: int) -> np.ndarray:
    """Normalized Sylvester Hadamard matrix of order ``d`` (a power of two):
    entry (i, j) = (-1)**popcount(i & j) / sqrt(d).  Section 3 asks only for
    some Hadamard matrix scaled to be orthonormal; the Sylvester one is the reading taken."""
    if d < 1 or (d & (d - 1)) != 0:
        raise ValueError("Sylvester Hadamard needs a power-of-two order")
    h = np.ones((1, 1))
    while h.shape[0] < d:
        h = np.block([[h, h], [h, -h]])
    return h / np.sqrt(d)


def wush_factors(M, H, gamma):
    """The pieces of Eq. 1: damped M and H, Cholesky factor L, the
    eigendecomposition (lam ascending, U canonicalised) and the scalar c.
    Canonical form (the paper fixes neither order nor sign): eigenvalues
    ascending; each eigenvector is signed so that its entry of largest
    magnitude is positive."""
    M = np.asarray(M, dtype=np.float64)
    H = np.asarray(H, dtype=np.float64)
    d = M.shape[0]
    eye = np.eye(d)
    Md = M + gamma * np.trace(M) / d * eye
    Hd = H + gamma * np.trace(H) / d * eye
    L = np.linalg.cholesky(Hd)               # lower, L L^T = Hd; raises if not PD
    A = L.T @ Md @ L
    A = 0.5 * (A + A.T)
    lam, U = np.linalg.eigh(A)               # ascending
    if lam[0] <= 0.0:
        raise np.linalg.LinAlgError("damped Gram matrix is not positive definite")
    idx = np.argmax(np.abs(U), axis=0)
    sgn = np.sign(U[idx, np.arange(d)])
    sgn[sgn == 0] = 1.0
    U = U * sgn
    c = np.sqrt(1.0 + gamma) * np.sqrt(np.trace(M)) / np.sqrt(np.sum(np.sqrt(lam)))
    return Md, Hd, L, lam, U, c


def wush(M, H, gamma: float = 1e-2) -> np.ndarray:
    """Wush(M, H, gamma) of Definition 1: T = c * Had * Lam^(-1/4) * U^T * L^T
    (Eq. 1), in float64, unrounded.  ``c`` uses the undamped tr(M)."""
    _, _, L, lam, U, c = wush_factors(M, H, gamma)
    d = L.shape[0]
    return c * (hadamard(d) @ (np.diag(lam ** -0.25) @ (U.T @ L.T)))


def gram_hessian(K, Q):
    """Key-side statistics of Eq. 4 / Algorithm 1 lines 4-5 for one KV head.
    K: [n_tok][d] post-RoPE keys; Q: [G][n_tok][d] post-RoPE queries of the
    group.  Returns M = sum_t k k^T and H = 2 sum_g sum_t q q^T."""
    K = np.asarray(K, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    M = K.T @ K
    H = np.zeros_like(M)
    for g in range(Q.shape[0]):
        H += Q[g].T @ Q[g]
    return M, 2.0 * H


def causal_probabilities(Q, K, tau: float):
    """Attention probabilities of one query head over one key head (Section 4.1): P[t, s] =
    softmax_s(q_t . k_s / tau) over s <= t, zero for s > t.  Q, K are [S][d] rows."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    S = Q.shape[0]
    logits = Q @ K.T / tau
    logits[np.triu_indices(S, k=1)] = -np.inf
    logits -= logits.max(axis=1, keepdims=True)
    E = np.exp(logits)
    return E / E.sum(axis=1, keepdims=True)


def attention_hessians(Q, K, V, W_O, tau: float):
    """Appendix C: the attention-aware Hessians of one key/value head over one calibration sequence, summed
    over the perturbed position s as the WUSH-A aggregation does ("Aggregation for WUSH-A").
      Q   [S][G][d_k]   queries of the G heads that read this key/value head (after Norm and RoPE)
      K   [S][d_k], V [S][d_v]
      W_O [G][d_v][d_model]   output-projection blocks
    Returns (H_K [d_k][d_k], H_V [d_v][d_v]) with H = 2 sum_s sum_t J_{t,s}^T J_{t,s}, where J_{t,s} is the derivative
    of the module output y_t with respect to a perturbation of k_s (key Jacobian) or of v_s (value Jacobian), taken
    literally from the appendix:
      key:   J = (1/tau) sum_g p_{g,t,s} W_O(g)^T (v_s - o_{g,t}) q_{g,t}^T      [d_model x d_k]
      value: J = sum_g p_{g,t,s} W_O(g)^T                                       [d_model x d_v]
    Plain loops over (s, t): for small calibration problems only."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    W_O = np.asarray(W_O, dtype=np.float64)
    S, G, dk = Q.shape
    dv = V.shape[1]
    P = [causal_probabilities(Q[:, g], K, tau) for g in range(G)]          # [G] x [t][s]
    Oh = [P[g] @ V for g in range(G)]                                      # head outputs o_{g,t}
    H_K = np.zeros((dk, dk))
    H_V = np.zeros((dv, dv))
    for s in range(S):
        for t in range(s, S):
            Jk = np.zeros((W_O.shape[2], dk))
            Jv = np.zeros((W_O.shape[2], dv))
            for g in range(G):
                Jk += P[g][t, s] * np.outer(W_O[g].T @ (V[s] - Oh[g][t]), Q[t, g]) / tau
                Jv += P[g][t, s] * W_O[g].T
            H_K += 2.0 * Jk.T @ Jk
            H_V += 2.0 * Jv.T @ Jv
    return H_K, H_V


def build_transforms(M, H, gamma: float = 1e-2):
    """Per-head transforms as the library stores them.  M, H: [n][d][d].
    Returns (T, T_invT): T = Wush(M, H, gamma) rounded to bf16 (the model runs
    in bf16, Sections 5.1 and 5.3; the paper does not state T's precision) and
    T_invT = (T^-1)^T of that ROUNDED matrix, rounded to fp32, so that the
    insertion identity of Eq. 3 holds for the stored pair."""
    M = np.asarray(M, dtype=np.float64)
    H = np.asarray(H, dtype=np.float64)
    T = np.empty_like(M)
    TinvT = np.empty_like(M)
    for h in range(M.shape[0]):
        T[h] = round_bf16(wush(M[h], H[h], gamma))
        TinvT[h] = round_fp32(np.linalg.inv(T[h]).T)
    return T, TinvT


# --------------------------------------------------------------------------
# normalisation and rotary embedding ahead of the transform  (Algorithm 2, lines 1-2)
# --------------------------------------------------------------------------
def rms_norm(x, weight=None, eps: float = 0.0):
    """Algorithm 2 lines 1-2, "Norm": headwise RMS normalisation of every row of ``x`` ([..., d]),
    x / sqrt(mean(x^2) + eps) times a per-channel weight ([d] or broadcastable; None: ones).
    The paper names the step and cites the architecture (Section 4.1: keys are cached after
    normalisation and rotation); the formula is the standard one of that architecture."""
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    y = x / np.sqrt(ms + eps)
    return y if weight is None else y * np.asarray(weight, dtype=np.float64)


def rope(x, positions, theta: float):
    """Algorithm 2 lines 1-2, "RoPE": rotate channel pair (j, j + d/2) of every row by the angle
    position * theta^(-2 j / d).  ``x`` is [n][..., d], ``positions`` [n] (absolute, 0-based).
    Reading: the paper does not say how channels are paired; the half-split pairing is the one of the
    model family it evaluates."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    half = d // 2
    j = np.arange(half, dtype=np.float64)
    ang = np.asarray(positions, dtype=np.float64).reshape((-1,) + (1,) * (x.ndim - 1)) * theta ** (-2.0 * j / d)
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, a * s + b * c], axis=-1)


def prepare_rows(x_proj, positions, theta: float, weight=None, eps: float = 0.0, normalise: bool = True):
    """Algorithm 2 lines 1-2 for projected keys or queries ([n][heads][d], bf16-valued): optional Norm,
    then RoPE, in float64, and ONE rounding to bf16 at the end (the model's activation format,
    Section 5.3).  Reading: the paper fixes no rounding points inside the two steps."""
    y = rms_norm(x_proj, weight, eps) if normalise else np.asarray(x_proj, dtype=np.float64)
    return round_bf16(rope(y, positions, theta))


def key_transform(T, k_rows):
    """Algorithm 2 line 3, key side: k' = T k for every row of ``k_rows``
    ([n][d]); float64, no intermediate rounding."""
    return np.asarray(k_rows, dtype=np.float64) @ np.asarray(T, dtype=np.float64).T


def query_compensation(T_invT, q_rows):
    """Algorithm 2 line 3, query side: q' = T^{-T} q, with the stored
    row-major T_invT = (T^-1)^T."""
    return np.asarray(q_rows, dtype=np.float64) @ np.asarray(T_invT, dtype=np.float64).T


# --------------------------------------------------------------------------
# percentile-clipped affine quantizer  (Section 5.3, Eq. 6)
# --------------------------------------------------------------------------


def quantile_abs(x, kappa: float) -> float:
    """quantile_kappa(|x_i|) over the d entries of one group (Eq. 6).
    Reading: linear interpolation between order statistics at fractional rank
    kappa*(d-1) of the ascending sort (the rule numpy and torch default to)."""
    a = np.sort(np.abs(np.asarray(x, dtype=np.float64)))
    d = a.shape[0]
    pos = kappa * (d - 1)
    lo = int(np.floor(pos))
    lo = min(max(lo, 0), d - 1)
    hi = min(lo + 1, d - 1)
    frac = pos - lo
    return float(a[lo] + frac * (a[hi] - a[lo]))


def clip_range(x, kappa: float):
    """x_min and x_max of Eq. 6: the group's extremes clipped to +-quantile."""
    x = np.asarray(x, dtype=np.float64)
    q = quantile_abs(x, kappa)
    x_min = max(float(np.min(x)), -q)
    x_max = min(float(np.max(x)), q)
    return x_min, x_max


def quantize(x, bits: int, kappa: float):
    """Eq. 6 for one token-head group ``x`` ([d]).  Returns (codes uint8 [d],
    delta, x_min) where delta and x_min are the STORED values.

    Readings (the paper fixes none of these): the step Delta and the offset
    x_min are stored in fp16 and the codes are computed with the stored
    values; the zero point is kept as x_min (= -Delta z, so that
    Q(x) = x_min + Delta*code is the same reconstruction as Eq. 6);
    round-to-nearest breaks ties to even; a group whose stored step is zero
    gets all-zero codes and reconstructs to x_min."""
    x = np.asarray(x, dtype=np.float64)
    levels = (1 << bits) - 1
    x_min, x_max = clip_range(x, kappa)
    delta = (x_max - x_min) / levels
    delta_s = float(round_fp16(delta))
    xmin_s = float(round_fp16(x_min))
    if delta_s > 0.0:
        codes = np.clip(np.rint((x - xmin_s) / delta_s), 0, levels)
    else:
        codes = np.zeros_like(x)
    return codes.astype(np.uint8), delta_s, xmin_s


def dequantize(codes, delta, x_min):
    """Reconstruction of Eq. 6: x_hat = Delta*(code - z) = x_min + Delta*code."""
    return x_min + delta * np.asarray(codes, dtype=np.float64)


def quantize_rows(X, bits: int, kappa: float):
    """``quantize`` applied to every row of X ([n][d])."""
    X = np.asarray(X, dtype=np.float64)
    n, d = X.shape
    codes = np.empty((n, d), dtype=np.uint8)
    delta = np.empty(n)
    xmin = np.empty(n)
    for i in range(n):
        codes[i], delta[i], xmin[i] = quantize(X[i], bits, kappa)
    return codes, delta, xmin


# --------------------------------------------------------------------------
# QuEST quantizer  (Section 4.3, Eq. 5; Lemma 1)
# --------------------------------------------------------------------------


def _gauss_grid_mse(alpha: float, bits: int) -> float:
    """E[(Q_alpha(z) - z)^2] for z ~ N(0, 1) and the 2^b levels evenly spaced from -alpha to +alpha with
    nearest-level rounding (the fixed-scale grid of Section 4.3), in closed form from the Gaussian
    density and distribution function."""
    import math
    n = 1 << bits
    step = 2.0 * alpha / (n - 1)
    levels = [-alpha + k * step for k in range(n)]
    edges = [-math.inf] + [0.5 * (levels[k] + levels[k + 1]) for k in range(n - 1)] + [math.inf]
    pdf = lambda t: 0.0 if math.isinf(t) else math.exp(-0.5 * t * t) / math.sqrt(2.0 * math.pi)   # noqa: E731
    cdf = lambda t: 0.5 * (1.0 + math.erf(t / math.sqrt(2.0)))                                      # noqa: E731
    tpdf = lambda t: 0.0 if math.isinf(t) else t * pdf(t)                                            # noqa: E731
    mse = 0.0
    for k in range(n):
        a, b, c = edges[k], edges[k + 1], levels[k]
        m0 = cdf(b) - cdf(a)                    # integral of the density
        m1 = pdf(a) - pdf(b)                    # integral of z * density
        m2 = m0 + tpdf(a) - tpdf(b)             # integral of z^2 * density
        mse += m2 - 2.0 * c * m1 + c * c * m0
    return mse


def quest_alpha(bits: int) -> float:
    """alpha_b of Eq. 5: the endpoint of the 2^b-level evenly spaced grid that minimises the mean squared
    error on a standard Gaussian (Section 4.3; the paper prints no value).  Golden-section search on the
    closed-form error, which is unimodal in alpha on (0, 8)."""
    lo, hi = 1e-3, 8.0
    r = (np.sqrt(5.0) - 1.0) / 2.0
    x1, x2 = hi - r * (hi - lo), lo + r * (hi - lo)
    f1, f2 = _gauss_grid_mse(x1, bits), _gauss_grid_mse(x2, bits)
    for _ in range(200):
        if f1 < f2:
            hi, x2, f2 = x2, x1, f1
            x1 = hi - r * (hi - lo)
            f1 = _gauss_grid_mse(x1, bits)
        else:
            lo, x1, f1 = x1, x2, f2
            x2 = lo + r * (hi - lo)
            f2 = _gauss_grid_mse(x2, bits)
    return float(0.5 * (lo + hi))


_QUEST_ALPHA = {}


def quest_quantize(x, bits: int):
    """Eq. 5 for one token-head group ``x`` ([d]): step Delta = 2 alpha_b (2^b - 1)^-1 d^-1/2 ||x||, bin index
    floor(x / Delta) clamped to [-2^(b-1), 2^(b-1) - 1], reconstruction at the bin centre Delta (index + 1/2);
    the zero group maps to zero.  Returns (codes uint8 [d] = index + 2^(b-1), delta, x_min) in the same
    storage format as ``quantize``: x_hat = x_min + delta * code with x_min = -delta (2^b - 1) / 2.

    Readings (storage, as for Eq. 6): the step is stored in fp16 and the bin indices are computed with the
    stored step; the stored offset is the fp16 rounding of -delta (2^b - 1) / 2."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[0]
    if bits not in _QUEST_ALPHA:
        _QUEST_ALPHA[bits] = quest_alpha(bits)
    half = 1 << (bits - 1)
    levels = (1 << bits) - 1
    rms = np.sqrt(np.sum(x * x) / d)
    delta = 2.0 * _QUEST_ALPHA[bits] / levels * rms
    delta_s = float(round_fp16(delta))
    xmin_s = float(round_fp16(-delta_s * levels / 2.0))
    if delta_s > 0.0:
        idx = np.clip(np.floor(x / delta_s), -half, half - 1)
    else:
        idx = np.full_like(x, -half)
        xmin_s = 0.0                                 # Q(0) = 0: every code reconstructs to zero
    return (idx + half).astype(np.uint8), delta_s, xmin_s


def pack_codes(codes, bits: int) -> np.ndarray:
    """Reference bit packing (storage definition only): the codes of a vector form one little-endian
    bit stream, channel i occupying stream bits [bits*i, bits*(i+1)); d*bits/8 bytes per vector
    (32 / 48 / 64 bytes at 2 / 3 / 4 bits for d = 128).  For 2 and 4 bits this is "channel i in bits
    bits*(i % per) of byte i // per", per = 8/bits.  The CUDA library is free to permute its physical
    layout; parity is checked on logical codes."""
    codes = np.asarray(codes, dtype=np.uint8)
    d = codes.shape[-1]
    assert (d * bits) % 8 == 0
    planes = ((codes[..., None] >> np.arange(bits, dtype=np.uint8)) & 1).astype(np.uint8)     # [..., d, bits], low bit first
    stream = planes.reshape(codes.shape[:-1] + (d * bits,))
    return np.packbits(stream, axis=-1, bitorder="little")


def unpack_codes(packed, bits: int) -> np.ndarray:
    packed = np.asarray(packed, dtype=np.uint8)
    stream = np.unpackbits(packed, axis=-1, bitorder="little")
    d = stream.shape[-1] // bits
    planes = stream.reshape(packed.shape[:-1] + (d, bits)).astype(np.uint16)
    return (planes << np.arange(bits, dtype=np.uint16)).sum(axis=-1).astype(np.uint8)


# --------------------------------------------------------------------------
# full-precision windows  (Section 4.4, Algorithm 2 lines 7-12)
# --------------------------------------------------------------------------


def boundary_step(S_quant: int, S: int, s_sink: int, s_keep: int, s_flush: int):
    """One pass of Algorithm 2 lines 7-8.  Returns (S_start, new S_quant);
    positions [S_start, S_quant) (0-based) are the ones quantized by lines
    9-12 of this pass."""
    S_start = max(S_quant, s_sink)
    S_new = max(S_quant, S_start + ((S - s_keep - S_start) // s_flush) * s_flush)
    return S_start, S_new


def n_quantized(S: int, s_sink: int, s_keep: int, s_flush: int) -> int:
    """Number of positions in the quantized middle region once the cache holds
    S positions: they are [s_sink, s_sink + n).  Closed form of the recurrence
    ``boundary_step`` (which does not depend on how S was reached)."""
    room = S - s_keep - s_sink
    if room < s_flush:
        return 0
    return (room // s_flush) * s_flush


# --------------------------------------------------------------------------
# cache with quantize-on-append, and decode attention
# --------------------------------------------------------------------------


class LayerCache:
    """One sequence, one attention module, in transformed coordinates
    (Algorithm 2 REQUIRE).  Every appended position is stored twice: as
    Eq. 6 codes + (Delta, x_min) and as the bf16 rounding of the same vector.
    Which copy attention reads is decided by the windows at read time.

    Reading: a position is quantized from the float transform output at the
    moment it is appended (the per-token quantizer makes the result
    independent of WHEN it is flushed; only a bf16 round trip before
    quantizing could change it, and that variant is available through
    ``quantize_from_bf16``)."""

    def __init__(self, n_kv, d, bits, kappa_k, kappa_v, T, quantize_from_bf16=False, quantizer="affine"):
        assert quantizer in ("affine", "quest")      # Eq. 6 (percentile-clipped affine) or Eq. 5 (QuEST; kappa unused)
        self.quantizer = quantizer
        self.n_kv, self.d, self.bits = n_kv, d, bits
        self.kappa_k, self.kappa_v = kappa_k, kappa_v
        self.T = np.asarray(T, dtype=np.float64)
        self.from_bf16 = quantize_from_bf16
        self.S = 0
        self.k_codes, self.v_codes = [], []      # each [n_kv][d] uint8 per position
        self.k_meta, self.v_meta = [], []        # each [n_kv][2] (delta, x_min)
        self.k_bf16, self.v_bf16 = [], []        # each [n_kv][d]

    def append(self, K_new, V_new):
        """Algorithm 2 lines 3-4 and 9-12 for a chunk.  K_new: [n][n_kv][d]
        post-Norm post-RoPE keys (bf16-valued); V_new: [n][n_kv][d] values in
        the folded basis (bf16-valued)."""
        K_new = np.asarray(K_new, dtype=np.float64)
        V_new = np.asarray(V_new, dtype=np.float64)
        for t in range(K_new.shape[0]):
            kc = np.empty((self.n_kv, self.d), np.uint8)
            vc = np.empty((self.n_kv, self.d), np.uint8)
            km = np.empty((self.n_kv, 2))
            vm = np.empty((self.n_kv, 2))
            kb = np.empty((self.n_kv, self.d))
            for h in range(self.n_kv):
                kp = key_transform(self.T[h], K_new[t, h][None, :])[0]
                kb[h] = round_bf16(kp)
                src = kb[h] if self.from_bf16 else kp
                if self.quantizer == "quest":
                    kc[h], km[h, 0], km[h, 1] = quest_quantize(src, self.bits)
                    vc[h], vm[h, 0], vm[h, 1] = quest_quantize(V_new[t, h], self.bits)
                else:
                    kc[h], km[h, 0], km[h, 1] = quantize(src, self.bits, self.kappa_k)
                    vc[h], vm[h, 0], vm[h, 1] = quantize(V_new[t, h], self.bits, self.kappa_v)
            self.k_codes.append(kc)
            self.v_codes.append(vc)
            self.k_meta.append(km)
            self.v_meta.append(vm)
            self.k_bf16.append(kb)
            self.v_bf16.append(round_bf16(V_new[t]))
            self.S += 1

    def arrays(self):
        """Stacked views: codes [S][n_kv][d], meta [S][n_kv][2], bf16 [S][n_kv][d]."""
        return (np.stack(self.k_codes), np.stack(self.k_meta), np.stack(self.v_codes),
                np.stack(self.v_meta), np.stack(self.k_bf16), np.stack(self.v_bf16))


def effective_kv(k_codes, k_meta, v_codes, v_meta, k_bf16, v_bf16, S, s_sink, s_keep,
                 s_flush, lag=0):
    """The cache as attention reads it for ONE KV head (Section 4.4): positions
    [s_sink, s_sink + n_quantized(S - lag)) come from the dequantized codes,
    every other position from the bf16 copy.  Inputs: codes [S][d], meta
    [S][2], bf16 [S][d].

    Reading: ``lag`` = 0 takes the boundary from the current length, the
    serving behaviour described in Section 5.3 (storage is updated before
    attention, windows are exactly S_sink and S_keep at S_flush = 1);
    ``lag`` = number of positions appended this step reproduces Algorithm 2
    literally (attention in line 5 precedes the boundary update in line 8)."""
    nq = n_quantized(S - lag, s_sink, s_keep, s_flush)
    K = np.array(k_bf16[:S], dtype=np.float64)
    V = np.array(v_bf16[:S], dtype=np.float64)
    lo, hi = s_sink, s_sink + nq
    if nq > 0:
        K[lo:hi] = k_meta[lo:hi, 1:2] + k_meta[lo:hi, 0:1] * k_codes[lo:hi].astype(np.float64)
        V[lo:hi] = v_meta[lo:hi, 1:2] + v_meta[lo:hi, 0:1] * v_codes[lo:hi].astype(np.float64)
    return K, V


def attention_one_query(q_comp, K_eff, V_eff, sm_scale):
    """Eq. 2 for a single query column that sees every cached position:
    p = softmax(sm_scale * K^T q), o = V p.  One global softmax, float64."""
    s = sm_scale * (K_eff @ q_comp)
    s = s - np.max(s)
    p = np.exp(s)
    p /= np.sum(p)
    return p @ V_eff


def decode_attn(q, T_invT, k_codes, k_meta, v_codes, v_meta, k_bf16, v_bf16, S,
                s_sink, s_keep, s_flush, sm_scale, lag=0):
    """Algorithm 2 lines 3 and 5 for one decode step of one sequence.
    q: [n_q][d] post-RoPE queries (not compensated); T_invT: [n_kv][d][d];
    cache arrays as returned by ``LayerCache.arrays`` ([S][n_kv][...]).
    Query head j reads KV head j // G.  Returns O [n_q][d] in the folded value
    basis (the output projection of line 6 is outside the path)."""
    q = np.asarray(q, dtype=np.float64)
    n_q, d = q.shape
    n_kv = T_invT.shape[0]
    G = n_q // n_kv
    out = np.empty((n_q, d))
    for h in range(n_kv):
        K_eff, V_eff = effective_kv(k_codes[:, h], k_meta[:, h], v_codes[:, h], v_meta[:, h],
                                    k_bf16[:, h], v_bf16[:, h], S, s_sink, s_keep, s_flush, lag)
        for g in range(G):
            j = h * G + g
            qc = query_compensation(T_invT[h], q[j][None, :])[0]
            out[j] = attention_one_query(qc, K_eff, V_eff, sm_scale)
    return out


def chunk_attn(q_chunk, T_invT, k_codes, k_meta, v_codes, v_meta, k_bf16, v_bf16, S, n_new,
               s_sink, s_keep, s_flush, sm_scale, lag=0, rows=None):
    """Algorithm 2 lines 3 and 5 for a chunk of ``n_new`` > = 1 new positions of one sequence, AFTER they
    were appended (line 4): the cache holds S positions, the chunk is positions [S - n_new, S).
    q_chunk: [n_new][n_q][d] post-RoPE queries of the chunk (not compensated).  Chunk position i attends to
    positions 0 .. S - n_new + i (causal inside the chunk).  Returns O [n_new][n_q][d].

    Which copy each position is read from (Section 4.4; Section 5.3): positions of the chunk itself are
    read from their bf16 copies (the method appends a new chunk in full precision and computes the chunk's
    attention output from those copies; the serving integration updates the storage before attention and
    still reads the current chunk's keys and values in bf16); every older position follows the window rule at
    the cache length S - lag, as in ``effective_kv``.  Readings: lag = 0 is the serving behaviour;
    lag = n_new is Algorithm 2 taken literally (the boundary is only moved in lines 7-8, after
    attention)."""
    q_chunk = np.asarray(q_chunk, dtype=np.float64)
    n_new_, n_q, d = q_chunk.shape
    assert n_new_ == n_new and 1 <= n_new <= S
    n_kv = T_invT.shape[0]
    G = n_q // n_kv
    S0 = S - n_new
    out = np.full((n_new, n_q, d), np.nan)             # ``rows``: only these chunk rows are computed (the rest stay NaN)
    for h in range(n_kv):
        K_eff, V_eff = effective_kv(k_codes[:, h], k_meta[:, h], v_codes[:, h], v_meta[:, h],
                                    k_bf16[:, h], v_bf16[:, h], S, s_sink, s_keep, s_flush, lag)
        K_eff[S0:S] = np.asarray(k_bf16[S0:S, h], dtype=np.float64)      # the chunk is read in full precision
        V_eff[S0:S] = np.asarray(v_bf16[S0:S, h], dtype=np.float64)
        for g in range(G):
            j = h * G + g
            qc = query_compensation(T_invT[h], q_chunk[:, j])            # [n_new][d]
            for i in (range(n_new) if rows is None else rows):
                n_vis = S0 + i + 1
                out[i, j] = attention_one_query(qc[i], K_eff[:n_vis], V_eff[:n_vis], sm_scale)
    return out


# --------------------------------------------------------------------------
# reconstruction-error metric  (Section 5.1)
# --------------------------------------------------------------------------


def rel_sq_err(A_hat, A) -> float:
    """Relative squared error ||A_hat - A||_F^2 / ||A||_F^2, numerator and
    denominator summed separately over everything passed in (Section 5.1)."""
    A_hat = np.asarray(A_hat, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    return float(np.sum((A_hat - A) ** 2) / np.sum(A ** 2))
