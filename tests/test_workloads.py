"""The seeded input generators: determinism, bf16 conversion, RoPE / RMSNorm sanity, logit scale."""
import numpy as np
import pytest

from paper_2609_38121_b200 import workloads as W


def test_bf16_bits_against_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(10000) * np.exp(4 * rng.standard_normal(10000))).astype(np.float32)
    bits = W.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    assert np.array_equal(W.bf16_bits_to_f32(bits), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_rope_is_a_rotation_and_relative():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 2, 128)).astype(np.float32)
    y = rng.standard_normal((5, 2, 128)).astype(np.float32)
    pos = np.array([0, 1, 7, 100, 4000])
    rx, ry = W.rope(x, pos, 1e4), W.rope(y, pos + 13, 1e4)
    np.testing.assert_allclose(np.linalg.norm(rx, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-5)
    assert np.array_equal(W.rope(x, np.zeros(5), 1e4), x)
    # dot products depend only on the position difference
    a = np.einsum("thd,thd->th", W.rope(x, pos, 1e4), W.rope(y, pos + 13, 1e4))
    b = np.einsum("thd,thd->th", W.rope(x, pos + 50, 1e4), W.rope(y, pos + 63, 1e4))
    np.testing.assert_allclose(a, b, rtol=2e-3, atol=2e-3)


def test_rmsnorm_unit_rms():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((4, 3, 128)).astype(np.float32) * 7
    y = W.rmsnorm(x, np.ones((1, 3, 128), np.float32))
    np.testing.assert_allclose(np.sqrt(np.mean(y.astype(np.float64) ** 2, -1)), 1.0, rtol=1e-5)


@pytest.mark.parametrize("name", ["cfg0", "cfg4"])
def test_workload_is_deterministic_and_shaped(name):
    a, b = W.LayerWorkload(name), W.LayerWorkload(name)
    Ka, Qa, Va = a.calibration()
    Kb, Qb, Vb = b.calibration()
    assert np.array_equal(Ka, Kb) and np.array_equal(Qa, Qb) and np.array_equal(Va, Vb)
    assert Ka.shape == (512, a.n_kv, 128) and Qa.shape == (512, a.n_q, 128)
    assert np.array_equal(W.bf16_round_f32(Ka), Ka)
    c1 = list(a.sequence_tokens(0, 100, chunk=64))
    c2 = list(b.sequence_tokens(0, 100, chunk=64))
    assert [c[0] for c in c1] == [0, 64] and c1[1][1].shape == (36, a.n_kv, 128)
    assert all(np.array_equal(x[1], y[1]) and np.array_equal(x[2], y[2]) for x, y in zip(c1, c2))
    assert not np.array_equal(next(a.sequence_tokens(1, 8))[1], c1[0][1][:8])
    assert np.array_equal(a.queries(0, 99), b.queries(0, 99))
    # logits have standard deviation about 2, so the softmax is neither flat nor one-hot
    k = np.concatenate([c[1] for c in c1]).astype(np.float64)
    q = a.queries(0, 99).astype(np.float64)
    logits = np.stack([k[:, j // a.G] @ q[j] for j in range(a.n_q)]) / np.sqrt(128)
    assert 0.7 < np.std(logits) < 5.0
    # outlier channels: the 4 largest channel scales dominate
    s = np.sort(a.s_k[0])
    assert s[-4] > 4 * np.median(s)


def test_ragged_lengths():
    wl = W.LayerWorkload("cfg2")
    L = wl.lengths()
    assert L.shape == (64,) and L.min() >= 1024 and L.max() <= 8192 and len(np.unique(L)) > 32
    assert np.array_equal(L, W.LayerWorkload("cfg2").lengths())
    assert np.all(W.LayerWorkload("cfg1").lengths() == 32768)
