"""Pins for the oracle's cache windows (Section 4.4, Algorithm 2), decode attention (Eq. 2, Eq. 3)
and the qualitative claim that WUSH lowers reconstruction error against the identity transform."""
import numpy as np
import pytest

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W


# ------------------------------------------------------------------ windows
def test_boundary_recurrence_matches_closed_form():
    rng = np.random.default_rng(21)
    for _ in range(300):
        s_sink, s_keep, s_flush = int(rng.integers(0, 70)), int(rng.integers(1, 300)), int(rng.integers(1, 65))
        S, S_quant = 0, 0
        for _ in range(int(rng.integers(1, 30))):
            S += int(rng.integers(1, 200))
            start, S_quant_new = O.boundary_step(S_quant, S, s_sink, s_keep, s_flush)
            assert S_quant_new >= S_quant
            S_quant = S_quant_new
            n = O.n_quantized(S, s_sink, s_keep, s_flush)
            assert n == max(S_quant - s_sink, 0)
            assert n % s_flush == 0
            full_tail = S - s_sink - n                      # recent positions still in full precision
            if n > 0:
                assert s_keep <= full_tail <= s_keep + s_flush - 1
            else:
                assert S - s_sink < s_keep + s_flush


def test_paper_window_settings():
    # perplexity runs: 16 / 128 / 16; downstream runs: 64 / 256 / 8
    assert O.n_quantized(2048, 16, 128, 16) == 1904
    assert O.n_quantized(16 + 128 + 15, 16, 128, 16) == 0
    assert O.n_quantized(16 + 128 + 16, 16, 128, 16) == 16
    assert O.n_quantized(32768, 64, 256, 8) == 32448
    assert O.n_quantized(32768, 4, 128, 1) == 32636            # benchmark config 1


def _tiny_layer(seed, n_kv=2, G=2, S=300, bits=2, identity=False):
    rng = np.random.default_rng(seed)
    d = 128
    K = W.bf16_round_f32(rng.standard_normal((S, n_kv, d)).astype(np.float32) * 2).astype(np.float64)
    V = W.bf16_round_f32(rng.standard_normal((S, n_kv, d)).astype(np.float32)).astype(np.float64)
    if identity:
        T = np.stack([np.eye(d)] * n_kv)
        TinvT = T.copy()
    else:
        Ms, Hs = [], []
        for h in range(n_kv):
            Qc = rng.standard_normal((G, 512, d)) * np.exp(rng.standard_normal(d))
            M, H = O.gram_hessian(K[:, h] * 1.0, Qc)
            Ms.append(M)
            Hs.append(H)
        T, TinvT = O.build_transforms(np.stack(Ms), np.stack(Hs))
    cache = O.LayerCache(n_kv, d, bits, 0.96, 0.92, T)
    cache.append(K, V)
    q = W.bf16_round_f32(rng.standard_normal((n_kv * G, d)).astype(np.float32)).astype(np.float64)
    return cache, T, TinvT, K, V, q


def test_window_entries_pass_through_untouched():
    cache, T, TinvT, K, V, q = _tiny_layer(22)
    kc, km, vc, vm, kb, vb = cache.arrays()
    S, s_sink, s_keep, s_flush = 300, 4, 64, 8
    nq = O.n_quantized(S, s_sink, s_keep, s_flush)
    assert nq == 232
    for h in range(2):
        Ke, Ve = O.effective_kv(kc[:, h], km[:, h], vc[:, h], vm[:, h], kb[:, h], vb[:, h], S, s_sink, s_keep, s_flush)
        win = np.r_[0:s_sink, s_sink + nq:S]
        assert np.array_equal(Ve[win], V[win, h])                       # values: the input itself
        assert np.array_equal(Ke[win], O.round_bf16(K[win, h] @ T[h].T))  # keys: bf16 of T k
        mid = np.arange(s_sink, s_sink + nq)
        assert np.array_equal(Ve[mid], vm[mid, h, 1:2] + vm[mid, h, 0:1] * vc[mid, h])
        assert not np.array_equal(Ve[mid], V[mid, h])
        assert len(np.unique(Ve[mid[0]])) <= 4


def test_short_context_is_plain_bf16_attention():
    """While S <= S_sink + S_keep + S_flush - 1 nothing is read quantized, so decode must equal
    textbook softmax attention on the bf16 cache (checked with torch's own attention routine)."""
    torch = pytest.importorskip("torch")
    cache, T, TinvT, K, V, q = _tiny_layer(23, S=75)
    kc, km, vc, vm, kb, vb = cache.arrays()
    out = O.decode_attn(q, TinvT, kc, km, vc, vm, kb, vb, 75, 4, 64, 8, 1 / np.sqrt(128))
    for j in range(4):
        h = j // 2
        qc = torch.from_numpy(TinvT[h] @ q[j])[None, None, None, :]
        kk = torch.from_numpy(kb[:, h])[None, None]
        vv = torch.from_numpy(vb[:, h])[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(qc, kk, vv, scale=1 / np.sqrt(128))[0, 0, 0].numpy()
        np.testing.assert_allclose(out[j], ref, rtol=1e-10, atol=1e-12)
    # and because of Eq. 3 that is the untransformed attention up to the bf16 rounding of T k
    for j in range(4):
        h = j // 2
        s = (K[:, h] @ q[j]) / np.sqrt(128)
        p = np.exp(s - s.max())
        ref = (p / p.sum()) @ V[:, h]
        assert np.max(np.abs(out[j] - ref)) < 3e-2 * np.max(np.abs(ref))


def test_decode_matches_library_attention_on_effective_cache():
    torch = pytest.importorskip("torch")
    cache, T, TinvT, K, V, q = _tiny_layer(24, bits=4)
    kc, km, vc, vm, kb, vb = cache.arrays()
    out = O.decode_attn(q, TinvT, kc, km, vc, vm, kb, vb, 300, 4, 64, 1, 0.1)
    for j in range(4):
        h = j // 2
        Ke, Ve = O.effective_kv(kc[:, h], km[:, h], vc[:, h], vm[:, h], kb[:, h], vb[:, h], 300, 4, 64, 1)
        qc = torch.from_numpy(O.query_compensation(TinvT[h], q[j][None])[0])[None, None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(
            qc, torch.from_numpy(Ke)[None, None], torch.from_numpy(Ve)[None, None], scale=0.1)[0, 0, 0].numpy()
        np.testing.assert_allclose(out[j], ref, rtol=1e-10, atol=1e-12)


def test_alg2_literal_boundary_lags_by_the_appended_chunk():
    cache, T, TinvT, K, V, q = _tiny_layer(25)
    kc, km, vc, vm, kb, vb = cache.arrays()
    args = (kc[:, 0], km[:, 0], vc[:, 0], vm[:, 0], kb[:, 0], vb[:, 0])
    K0, _ = O.effective_kv(*args, 300, 4, 64, 1, lag=0)
    K1, _ = O.effective_kv(*args, 300, 4, 64, 1, lag=1)
    nq = O.n_quantized(300, 4, 64, 1)
    diff = np.nonzero(np.any(K0 != K1, axis=1))[0]
    assert diff.tolist() == [4 + nq - 1]                     # exactly the newest flushed position differs


def test_permutation_of_cached_tokens_leaves_output_unchanged():
    cache, T, TinvT, K, V, q = _tiny_layer(26)
    kc, km, vc, vm, kb, vb = cache.arrays()
    base = O.decode_attn(q, TinvT, kc, km, vc, vm, kb, vb, 300, 4, 64, 1, 0.09)
    nq = O.n_quantized(300, 4, 64, 1)
    perm = np.arange(300)
    perm[4:4 + nq] = np.random.default_rng(0).permutation(np.arange(4, 4 + nq))
    out = O.decode_attn(q, TinvT, kc[perm], km[perm], vc[perm], vm[perm], kb[perm], vb[perm], 300, 4, 64, 1, 0.09)
    np.testing.assert_allclose(out, base, rtol=1e-11, atol=1e-13)


def test_identity_transform_is_plain_quantized_attention():
    cache, T, TinvT, K, V, q = _tiny_layer(27, identity=True)
    kc, km, vc, vm, kb, vb = cache.arrays()
    out = O.decode_attn(q, TinvT, kc, km, vc, vm, kb, vb, 300, 0, 1, 1, 0.09)
    for j in range(4):
        h = j // 2
        Kq = np.stack([O.dequantize(*O.quantize(K[t, h], 2, 0.96)) for t in range(299)] + [K[299, h]])
        Vq = np.stack([O.dequantize(*O.quantize(V[t, h], 2, 0.92)) for t in range(299)] + [V[299, h]])
        s = 0.09 * Kq @ q[j]
        p = np.exp(s - s.max())
        np.testing.assert_allclose(out[j], (p / p.sum()) @ Vq, rtol=1e-11, atol=1e-13)


def test_eight_bits_without_clipping_converges_to_exact_attention():
    cache8, T, TinvT, K, V, q = _tiny_layer(28)
    rng = np.random.default_rng(28)
    c = O.LayerCache(2, 128, 8, 1.0, 1.0, T)
    c.append(K, V)
    out = O.decode_attn(q, TinvT, *c.arrays(), 300, 4, 64, 1, 0.09)
    errs = []
    for j in range(4):
        h = j // 2
        s = 0.09 * (K[:, h] @ q[j])
        p = np.exp(s - s.max())
        ref = (p / p.sum()) @ V[:, h]
        errs.append(np.max(np.abs(out[j] - ref)) / np.max(np.abs(ref)))
    assert max(errs) < 2e-2
    out2 = O.decode_attn(q, TinvT, *cache8.arrays(), 300, 4, 64, 1, 0.09)       # 2-bit is far worse
    assert np.max(np.abs(out2 - out)) > 5 * max(errs) * np.max(np.abs(out))


# ------------------------------------------------------------------ quality
@pytest.mark.parametrize("bits", [2, 4])
def test_wush_lowers_reconstruction_error_against_identity(bits):
    """Section 5.1's claim, on the synthetic outlier-channel workload: with the same quantizer, the
    WUSH key transform gives a lower relative squared error of the attention scores than no transform,
    and the (T_K, T_V) pair a lower error of the module output sum_g W_O^T o over 256 held-out queries."""
    wl = W.LayerWorkload("cfg0")
    d, n_kv, G = 128, wl.n_kv, wl.G
    Kc, Qc, Vraw = wl.calibration()
    Ms, Hs, Mv, Hv = [], [], [], []
    for h in range(n_kv):
        M, H = O.gram_hessian(Kc[:, h], np.stack([Qc[:, h * G + g] for g in range(G)]))
        Ms.append(M)
        Hs.append(H)
        Mv.append(Vraw[:, h].astype(np.float64).T @ Vraw[:, h].astype(np.float64))
        Hv.append(2 * sum(wl.W_O[h, g].astype(np.float64) @ wl.W_O[h, g].astype(np.float64).T for g in range(G)))
    T_K, T_KinvT = O.build_transforms(np.stack(Ms), np.stack(Hs), W.GAMMA)
    T_V = np.stack([O.wush(Mv[h], Hv[h], W.GAMMA) for h in range(n_kv)])
    S, nQ = 384, 256
    rng = np.random.default_rng(99)
    pos = np.arange(S)
    Keys = wl._keys(rng, pos).astype(np.float64)
    Vr = wl._raw_values(rng, S).astype(np.float64)
    Qs = wl._queries(rng, np.full(nQ, S - 1)).astype(np.float64)

    def run(use_wush):
        s_hat_all, s_ref_all, y_hat_all, y_ref_all = [], [], [], []
        for h in range(n_kv):
            TK = T_K[h] if use_wush else np.eye(d)
            TKi = T_KinvT[h] if use_wush else np.eye(d)
            TV = T_V[h] if use_wush else np.eye(d)
            Kp = Keys[:, h] @ TK.T
            Vp = Vr[:, h] @ TV.T
            Kq = np.stack([O.dequantize(*O.quantize(Kp[t], bits, W.KAPPA_K)) for t in range(S)])
            Vq = np.stack([O.dequantize(*O.quantize(Vp[t], bits, W.KAPPA_V)) for t in range(S)])
            TVinvT = np.linalg.inv(TV).T
            for g in range(G):
                Qg = Qs[:, h * G + g]
                s_ref = Keys[:, h] @ Qg.T                       # [S][nQ] pre-scaling scores
                s_hat = Kq @ (Qg @ TKi.T).T
                s_hat_all.append(s_hat.ravel())
                s_ref_all.append(s_ref.ravel())
                P = np.exp((s_ref - s_ref.max(0)) / np.sqrt(d))
                P /= P.sum(0)
                Ph = np.exp((s_hat - s_hat.max(0)) / np.sqrt(d))
                Ph /= Ph.sum(0)
                Wo = wl.W_O[h, g].astype(np.float64)
                y_ref_all.append(((P.T @ Vr[:, h]) @ Wo).ravel())
                y_hat_all.append(((Ph.T @ Vq) @ (TVinvT @ Wo)).ravel())
        # Section 5.1: numerator and denominator are each summed over every head and query first
        return (O.rel_sq_err(np.concatenate(s_hat_all), np.concatenate(s_ref_all)),
                O.rel_sq_err(np.concatenate(y_hat_all), np.concatenate(y_ref_all)))

    s_w, y_w = run(True)
    s_i, y_i = run(False)
    assert s_w < 0.5 * s_i, (s_w, s_i)
    assert y_w < y_i, (y_w, y_i)


# ------------------------------------------------------------------ error metric (Section 5.1)
def test_rel_sq_err_hand_cases_and_pooling():
    # |(3,2) - (3,4)|^2 / |(3,4)|^2 = 4 / 25
    assert O.rel_sq_err([3.0, 2.0], [3.0, 4.0]) == pytest.approx(0.16, rel=1e-15)
    assert O.rel_sq_err([[1.0, -2.0], [0.5, 0.0]], [[1.0, -2.0], [0.5, 0.0]]) == 0.0
    assert O.rel_sq_err(np.zeros(5), np.arange(1.0, 6.0)) == pytest.approx(1.0, rel=1e-15)     # predicting zero
    # numerator and denominator are pooled before the division: a small block that is 100 % off and a
    # large exact block give 1 / 101, not the mean 0.5 of the two blocks' ratios
    pooled = O.rel_sq_err(np.array([2.0, 10.0]), np.array([1.0, 10.0]))
    assert pooled == pytest.approx(1.0 / 101.0, rel=1e-15)
    assert abs(pooled - 0.5 * (O.rel_sq_err([2.0], [1.0]) + O.rel_sq_err([10.0], [10.0]))) > 0.4
    # invariant under a common scaling, not symmetric in its arguments
    rng = np.random.default_rng(5)
    A, E = rng.standard_normal((7, 9)), 0.1 * rng.standard_normal((7, 9))
    assert O.rel_sq_err(3.0 * (A + E), 3.0 * A) == pytest.approx(O.rel_sq_err(A + E, A), rel=1e-12)
    assert O.rel_sq_err(A + E, A) == pytest.approx(np.linalg.norm(E) ** 2 / np.linalg.norm(A) ** 2, rel=1e-12)
    assert O.rel_sq_err(A + E, A) != pytest.approx(O.rel_sq_err(A, A + E), rel=1e-6)


# ------------------------------------------------------------------ the other reading of "what is quantized"
def test_quantize_from_bf16_reading():
    """``LayerCache(quantize_from_bf16=True)`` quantizes the bf16 rounding of the transformed key (the
    lazy reading of Section 4.4: the full-precision entry is what gets flushed); the default quantizes
    the float transform output.  Values are never transformed, so they agree under both readings."""
    rng = np.random.default_rng(33)
    d, n_kv, S = 128, 2, 96
    K = W.bf16_round_f32(rng.standard_normal((S, n_kv, d)).astype(np.float32) * 2).astype(np.float64)
    V = W.bf16_round_f32(rng.standard_normal((S, n_kv, d)).astype(np.float32)).astype(np.float64)
    Ms, Hs = [], []
    for h in range(n_kv):
        Qc = rng.standard_normal((2, 256, d)) * np.exp(rng.standard_normal(d))
        M, H = O.gram_hessian(K[:, h], Qc)
        Ms.append(M)
        Hs.append(H)
    T, _ = O.build_transforms(np.stack(Ms), np.stack(Hs))
    eager = O.LayerCache(n_kv, d, 4, 0.96, 0.92, T)
    lazy = O.LayerCache(n_kv, d, 4, 0.96, 0.92, T, quantize_from_bf16=True)
    eager.append(K, V)
    lazy.append(K, V)
    kc_e, km_e, vc_e, vm_e, kb_e, vb_e = eager.arrays()
    kc_l, km_l, vc_l, vm_l, kb_l, vb_l = lazy.arrays()
    differing_vectors = 0
    for t in range(S):
        for h in range(n_kv):
            kp = O.key_transform(T[h], K[t, h][None])[0]
            c, dl, z = O.quantize(O.round_bf16(kp), 4, 0.96)
            assert np.array_equal(kc_l[t, h], c) and km_l[t, h, 0] == dl and km_l[t, h, 1] == z
            c2, dl2, z2 = O.quantize(kp, 4, 0.96)
            assert np.array_equal(kc_e[t, h], c2) and km_e[t, h, 0] == dl2 and km_e[t, h, 1] == z2
            differing_vectors += int(not np.array_equal(c, c2))
    assert differing_vectors >= 1                      # the bf16 round trip moves some code at 4 bits
    assert np.mean(kc_l != kc_e) < 0.05                # ... but only a small fraction of them
    assert np.array_equal(vc_l, vc_e) and np.array_equal(vm_l, vm_e)
    assert np.array_equal(kb_l, kb_e) and np.array_equal(vb_l, vb_e)     # window copies do not depend on the reading
