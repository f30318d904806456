"""Seeded synthetic inputs shaped like the paper's workloads.

This module only MAKES INPUTS (random draws, channel scales, RMSNorm, RoPE,
bf16 bit conversion).  It contains none of the method's arithmetic — no WUSH
construction, no quantizer, no attention — so that it can serve both the CPU
oracle and the CUDA library without coupling them.  A value transform, where a
workload needs one, is passed in by the caller as a plain matrix.

The paper evaluates on real model activations (Qwen3 models driven by text
corpora and benchmark suites, Section 5); none of that is available offline,
so these tensors stand in for them: same head counts, head dimension, RoPE
base, context lengths and batch as the named model layers, with an
outlier-channel value distribution (a few channels much larger than the rest,
which is the structure a data-adaptive transform exploits).

Recipe (all draws float32, numpy Generator PCG64):
  * streams = SeedSequence(seed).spawn(8) in the fixed order
    [K scales, Q scales, V scales, W_O, calibration, cache tokens, queries,
    lengths]; cache tokens and queries spawn one child per sequence.
  * per KV head a channel scale s_c = exp(sigma * N(0,1)), sigma = 1, and the
    n_outlier = 4 largest channels are multiplied by 8 more.
  * pre-RoPE key k_t = s_K * N(0,1); query q_t = alpha * s_Q * N(0,1) with
    alpha set per query head from a 256-token probe so that the logits
    q.k / sqrt(d) have standard deviation 2 (otherwise softmax is one-hot).
  * optional headwise RMSNorm (sqrt(d) x / |x| * gain, gain = exp(0.25 N(0,1)))
    on q and k, then RoPE with half-split pairs (j, j + d/2),
    omega_j = theta ** (-2 j / d), at the token's absolute position.
  * value v_t = T_V (s_V * N(0,1)) for a caller-supplied T_V (identity if
    none): "values already in their weight-folded basis".
  * everything is rounded to bf16 (ties to even) before it is handed out.
"""
from __future__ import annotations

import numpy as np

D_HEAD = 128
D_MODEL_OUT = 512          # columns of the synthetic output projection blocks


# ----------------------------------------------------------------- bf16 bits
def f32_to_bf16_bits(x) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round_f32(x) -> np.ndarray:
    """float32 values rounded to bf16 and widened back to float32."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# ------------------------------------------------------------------ configs
CONFIGS = {
    # name: the five workloads of the benchmark definition
    "cfg0": dict(seed=0, batch=1, n_q=8, n_kv=2, ctx=2048, theta=1e4, bits=2, s_sink=4, s_keep=64,
                 rmsnorm=False, ragged=None, prefill_chunk=0),
    "cfg1": dict(seed=1, batch=16, n_q=32, n_kv=8, ctx=32768, theta=5e5, bits=2, s_sink=4, s_keep=128,
                 rmsnorm=False, ragged=None, prefill_chunk=0),
    "cfg2": dict(seed=2, batch=64, n_q=32, n_kv=8, ctx=8192, theta=5e5, bits=4, s_sink=4, s_keep=128,
                 rmsnorm=False, ragged=(1024, 8192), prefill_chunk=0),
    "cfg3": dict(seed=3, batch=1, n_q=64, n_kv=8, ctx=131072, theta=5e5, bits=2, s_sink=4, s_keep=128,
                 rmsnorm=False, ragged=None, prefill_chunk=0),
    "cfg4": dict(seed=4, batch=8, n_q=28, n_kv=4, ctx=8192, theta=1e6, bits=2, s_sink=4, s_keep=128,
                 rmsnorm=True, ragged=None, prefill_chunk=8192),
}
PAGE_TOKENS = 64
KAPPA_K = 0.96
KAPPA_V = 0.92
GAMMA = 1e-2
N_CALIBRATION = 512


def _channel_scales(rng, n_heads, d, sigma=1.0, n_outlier=4, boost=8.0):
    s = np.exp(sigma * rng.standard_normal((n_heads, d), dtype=np.float32))
    for h in range(n_heads):
        top = np.argsort(s[h])[-n_outlier:]
        s[h, top] *= boost
    return s.astype(np.float32)


def rope(x, positions, theta):
    """Rotate rows of x ([n, heads, d]) by their absolute positions ([n]).
    Half-split pairing: channel j is paired with channel j + d/2."""
    d = x.shape[-1]
    half = d // 2
    omega = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * omega[None, :]
    c = np.cos(ang).astype(np.float32)[:, None, :]
    s = np.sin(ang).astype(np.float32)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x1 * s + x2 * c], axis=-1)


def rmsnorm(x, gain):
    """Headwise RMS normalisation sqrt(d) x / |x| times a per-channel gain."""
    d = x.shape[-1]
    nrm = np.sqrt(np.sum(x.astype(np.float64) ** 2, axis=-1, keepdims=True))
    return (x * (np.sqrt(d) / nrm).astype(np.float32)) * gain


class LayerWorkload:
    """All seeded inputs of one attention layer for one named config."""

    def __init__(self, name_or_cfg, **overrides):
        cfg = dict(CONFIGS[name_or_cfg]) if isinstance(name_or_cfg, str) else dict(name_or_cfg)
        cfg.update(overrides)
        self.cfg = cfg
        self.d = D_HEAD
        self.n_q, self.n_kv = cfg["n_q"], cfg["n_kv"]
        self.G = self.n_q // self.n_kv
        self.theta = cfg["theta"]
        self.batch = cfg["batch"]
        ss = np.random.SeedSequence(cfg["seed"]).spawn(8)
        (self._ss_ks, self._ss_qs, self._ss_vs, self._ss_wo, self._ss_cal, self._ss_tok,
         self._ss_qry, self._ss_len) = ss
        self.s_k = _channel_scales(np.random.default_rng(self._ss_ks), self.n_kv, self.d)
        self.s_q = _channel_scales(np.random.default_rng(self._ss_qs), self.n_q, self.d)
        self.s_v = _channel_scales(np.random.default_rng(self._ss_vs), self.n_kv, self.d)
        rng_wo = np.random.default_rng(self._ss_wo)
        # output-projection blocks W_O(h,g) [d][D_MODEL_OUT] and, for RMSNorm configs, the gains
        self.W_O = (rng_wo.standard_normal((self.n_kv, self.G, self.d, D_MODEL_OUT), dtype=np.float32)
                    / np.float32(np.sqrt(self.d)))
        if cfg["rmsnorm"]:
            self.gain_k = np.exp(0.25 * rng_wo.standard_normal((self.n_kv, self.d), dtype=np.float32))
            self.gain_q = np.exp(0.25 * rng_wo.standard_normal((self.n_q, self.d), dtype=np.float32))
        else:
            self.gain_k = self.gain_q = None
        self.alpha = np.ones(self.n_q, dtype=np.float32)
        self._fit_query_scale()

    # ---- raw draws -------------------------------------------------------
    def _keys(self, rng, positions):
        n = len(positions)
        k = rng.standard_normal((n, self.n_kv, self.d), dtype=np.float32) * self.s_k[None]
        if self.gain_k is not None:
            k = rmsnorm(k, self.gain_k[None])
        return bf16_round_f32(rope(k, positions, self.theta))

    def _queries(self, rng, positions):
        n = len(positions)
        q = rng.standard_normal((n, self.n_q, self.d), dtype=np.float32) * self.s_q[None]
        if self.gain_q is not None:
            q = rmsnorm(q, self.gain_q[None])
        q = q * self.alpha[None, :, None]
        return bf16_round_f32(rope(q, positions, self.theta))

    def _raw_values(self, rng, n):
        return rng.standard_normal((n, self.n_kv, self.d), dtype=np.float32) * self.s_v[None]

    def _fit_query_scale(self):
        rng = np.random.default_rng(np.random.SeedSequence(self.cfg["seed"]).spawn(9)[8])
        pos = np.arange(256)
        k = self._keys(rng, pos).astype(np.float64)
        q = self._queries(rng, pos).astype(np.float64)
        for j in range(self.n_q):
            logits = q[:, j] @ k[:, j // self.G].T / np.sqrt(self.d)
            self.alpha[j] = np.float32(2.0 / np.std(logits))

    # ---- public draws ----------------------------------------------------
    def calibration(self):
        """512 tokens at positions 0..511: K [n][n_kv][d], Q [n][n_q][d] (post-RoPE, bf16-valued
        float32) and the raw, untransformed values [n][n_kv][d] (float32)."""
        rng = np.random.default_rng(self._ss_cal)
        pos = np.arange(N_CALIBRATION)
        return self._keys(rng, pos), self._queries(rng, pos), self._raw_values(rng, N_CALIBRATION)

    def lengths(self):
        """Per-sequence context lengths (the position count AFTER the decode-step append)."""
        if self.cfg["ragged"] is None:
            return np.full(self.batch, self.cfg["ctx"], dtype=np.int64)
        lo, hi = self.cfg["ragged"]
        return np.random.default_rng(self._ss_len).integers(lo, hi + 1, size=self.batch)

    def sequence_tokens(self, b, n_tokens, T_V=None, chunk=4096, pos0=0):
        """Yield (first_position, K [n][n_kv][d], V [n][n_kv][d]) chunks of sequence ``b``;
        K post-RoPE, V = T_V(raw) per KV head, both bf16-valued float32."""
        rng = np.random.default_rng(np.random.SeedSequence(
            entropy=self._ss_tok.entropy, spawn_key=self._ss_tok.spawn_key + (int(b),)))
        done = 0
        while done < n_tokens:
            n = min(chunk, n_tokens - done)
            pos = np.arange(pos0 + done, pos0 + done + n)
            K = self._keys(rng, pos)
            V = self._raw_values(rng, n)
            if T_V is not None:
                V = np.einsum("thj,hij->thi", V, np.asarray(T_V, dtype=np.float32))
            yield pos0 + done, K, bf16_round_f32(V)
            done += n

    def chunk_queries(self, b, positions):
        """Queries of sequence ``b`` at several positions (a prefill chunk): [n][n_q][d] bf16-valued float32."""
        rng = np.random.default_rng(np.random.SeedSequence(
            entropy=self._ss_qry.entropy, spawn_key=self._ss_qry.spawn_key + (int(b), 1)))
        return self._queries(rng, np.asarray(positions))

    def projected(self, b, n_tokens):
        """Projected (pre-Norm, pre-RoPE) keys [n][n_kv][d] and queries [n][n_q][d] of sequence ``b``: the same
        channel-scaled Gaussians the other draws start from, rounded to bf16, for callers that apply
        normalisation and rotation themselves."""
        rng = np.random.default_rng(np.random.SeedSequence(
            entropy=self._ss_tok.entropy, spawn_key=self._ss_tok.spawn_key + (int(b), 2)))
        k = rng.standard_normal((n_tokens, self.n_kv, self.d), dtype=np.float32) * self.s_k[None]
        q = rng.standard_normal((n_tokens, self.n_q, self.d), dtype=np.float32) * self.s_q[None] * self.alpha[None, :, None]
        return bf16_round_f32(k), bf16_round_f32(q)

    def queries(self, b, position):
        """The decode-step query of sequence ``b`` at ``position``: [n_q][d] bf16-valued float32."""
        rng = np.random.default_rng(np.random.SeedSequence(
            entropy=self._ss_qry.entropy, spawn_key=self._ss_qry.spawn_key + (int(b),)))
        return self._queries(rng, np.array([position]))[0]
