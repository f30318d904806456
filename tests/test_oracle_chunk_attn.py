"""Pins for the oracle's chunk (prefill) attention over the mixed cache: Algorithm 2 line 5 for a chunk
of more than one position, Section 4.4, Section 5.3."""
import numpy as np
import pytest

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W


def _layer(seed, S, n_kv=2, G=2, bits=2):
    rng = np.random.default_rng(seed)
    d = 128
    K = W.bf16_round_f32(rng.standard_normal((S, n_kv, d)).astype(np.float32) * 2).astype(np.float64)
    V = W.bf16_round_f32(rng.standard_normal((S, n_kv, d)).astype(np.float32)).astype(np.float64)
    Ms, Hs = [], []
    for h in range(n_kv):
        Qc = rng.standard_normal((G, 256, d)) * np.exp(rng.standard_normal(d))
        M, H = O.gram_hessian(K[:, h], Qc)
        Ms.append(M)
        Hs.append(H)
    T, TinvT = O.build_transforms(np.stack(Ms), np.stack(Hs))
    cache = O.LayerCache(n_kv, d, bits, 0.96, 0.92, T)
    cache.append(K, V)
    return cache, T, TinvT, K, V, rng


def _queries(rng, n, n_q):
    return W.bf16_round_f32(rng.standard_normal((n, n_q, 128)).astype(np.float32)).astype(np.float64)


def test_chunk_of_one_is_decode():
    cache, T, TinvT, K, V, rng = _layer(81, 300)
    q = _queries(rng, 1, 4)
    arrs = cache.arrays()
    for lag in (0, 1):
        a = O.chunk_attn(q, TinvT, *arrs, 300, 1, 4, 64, 8, 0.09, lag=lag)
        b = O.decode_attn(q[0], TinvT, *arrs, 300, 4, 64, 8, 0.09, lag=lag)
        np.testing.assert_allclose(a[0], b, rtol=1e-12, atol=1e-14)


def test_literal_algorithm2_rows_are_decodes_of_the_truncated_cache():
    """With the boundary of Algorithm 2 taken literally (moved after attention: lag = chunk length), row i of a
    chunk is the decode of a single token on the cache truncated after it, whose boundary lags by i + 1."""
    S, n_new = 260, 37
    cache, T, TinvT, K, V, rng = _layer(82, S)
    q = _queries(rng, n_new, 4)
    arrs = cache.arrays()
    out = O.chunk_attn(q, TinvT, *arrs, S, n_new, 4, 64, 8, 0.09, lag=n_new)
    for i in (0, 1, 17, n_new - 1):
        Si = S - n_new + i + 1
        ref = O.decode_attn(q[i], TinvT, *[a[:Si] for a in arrs], Si, 4, 64, 8, 0.09, lag=i + 1)
        np.testing.assert_allclose(out[i], ref, rtol=1e-12, atol=1e-14)


def test_nothing_quantized_is_plain_causal_attention():
    """A cache shorter than the two windows: every position is read in bf16, and the chunk rows equal textbook
    causal softmax attention in the original coordinates (insertion identity of Eq. 3)."""
    S, n_new, s_sink, s_keep, s_flush = 90, 30, 16, 64, 16
    cache, T, TinvT, K, V, rng = _layer(83, S)
    assert O.n_quantized(S, s_sink, s_keep, s_flush) == 0
    q = _queries(rng, n_new, 4)
    arrs = cache.arrays()
    out = O.chunk_attn(q, TinvT, *arrs, S, n_new, s_sink, s_keep, s_flush, 0.09)
    kb, vb = arrs[4], arrs[5]
    for i in (0, 11, n_new - 1):
        n_vis = S - n_new + i + 1
        for j in range(4):
            h = j // 2
            qc = O.query_compensation(TinvT[h], q[i, j][None])[0]
            s = 0.09 * kb[:n_vis, h] @ qc
            p = np.exp(s - s.max())
            np.testing.assert_allclose(out[i, j], (p / p.sum()) @ vb[:n_vis, h], rtol=1e-12, atol=1e-14)
            # bf16(T k) instead of T k: close to attention on the untransformed keys, not identical
            s0 = 0.09 * K[:n_vis, h] @ q[i, j]
            p0 = np.exp(s0 - s0.max())
            ref0 = (p0 / p0.sum()) @ V[:n_vis, h]
            assert np.max(np.abs(out[i, j] - ref0)) <= 3e-2 * np.max(np.abs(ref0))


def test_against_library_attention_with_an_explicit_mask():
    torch = pytest.importorskip("torch")
    S, n_new, s_sink, s_keep, s_flush = 330, 130, 4, 64, 8          # the chunk is longer than the recent window
    cache, T, TinvT, K, V, rng = _layer(84, S, bits=4)
    q = _queries(rng, n_new, 4)
    kc, km, vc, vm, kb, vb = cache.arrays()
    out = O.chunk_attn(q, TinvT, kc, km, vc, vm, kb, vb, S, n_new, s_sink, s_keep, s_flush, 0.1)
    S0 = S - n_new
    mask = torch.from_numpy(np.arange(S)[None, :] <= (S0 + np.arange(n_new))[:, None])
    nq = O.n_quantized(S, s_sink, s_keep, s_flush)
    assert s_sink + nq > S0                                         # the boundary has moved into the chunk ...
    for j in range(4):
        h = j // 2
        Ke, Ve = O.effective_kv(kc[:, h], km[:, h], vc[:, h], vm[:, h], kb[:, h], vb[:, h], S, s_sink, s_keep, s_flush)
        Ke[S0:], Ve[S0:] = kb[S0:, h], vb[S0:, h]                   # ... but chunk positions are read in bf16
        qc = torch.from_numpy(O.query_compensation(TinvT[h], q[:, j]))[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(
            qc, torch.from_numpy(Ke)[None, None], torch.from_numpy(Ve)[None, None], attn_mask=mask[None, None], scale=0.1)[0, 0].numpy()
        np.testing.assert_allclose(out[:, j], ref, rtol=1e-10, atol=1e-12)


def test_chunk_positions_ignore_their_codes_and_older_ones_do_not():
    S, n_new = 400, 50
    cache, T, TinvT, K, V, rng = _layer(85, S)
    q = _queries(rng, n_new, 4)
    kc, km, vc, vm, kb, vb = cache.arrays()
    base = O.chunk_attn(q, TinvT, kc, km, vc, vm, kb, vb, S, n_new, 4, 64, 1, 0.09)
    kc2 = kc.copy()
    kc2[S - n_new:] = 3 - kc2[S - n_new:]                           # codes of the chunk: never read
    same = O.chunk_attn(q, TinvT, kc2, km, vc, vm, kb, vb, S, n_new, 4, 64, 1, 0.09)
    assert np.array_equal(same, base)
    kc3 = kc.copy()
    kc3[100:120] = 3 - kc3[100:120]                                 # codes of old, quantized positions: read
    other = O.chunk_attn(q, TinvT, kc3, km, vc, vm, kb, vb, S, n_new, 4, 64, 1, 0.09)
    assert np.max(np.abs(other - base)) > 1e-6
    # causality: a later chunk token's key and value do not reach an earlier row
    kb2, vb2 = kb.copy(), vb.copy()
    kb2[S - 1] += 1.0
    vb2[S - 1] += 1.0
    last = O.chunk_attn(q, TinvT, kc, km, vc, vm, kb2, vb2, S, n_new, 4, 64, 1, 0.09)
    assert np.array_equal(last[:-1], base[:-1]) and not np.array_equal(last[-1], base[-1])
