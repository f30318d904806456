"""Pins of the oracle's Norm and RoPE (Algorithm 2 lines 1-2) against hand-worked values, closed
forms, invariants and independent formulations (complex multiplication, a library routine)."""
import math

import numpy as np
import pytest

from oracle import wushkv_oracle as O


def test_rms_norm_hand_example_and_unit_rms():
    x = np.array([[3.0, 4.0, 0.0, 0.0]])
    # mean square = 25 / 4 = 6.25 -> x / 2.5
    assert np.allclose(O.rms_norm(x), [[1.2, 1.6, 0.0, 0.0]], rtol=0, atol=1e-15)
    # with eps: 3 / sqrt(6.25 + 2.75) = 1
    assert np.allclose(O.rms_norm(x, eps=2.75), [[1.0, 4.0 / 3.0, 0.0, 0.0]], rtol=0, atol=1e-15)
    # per-channel weight multiplies after the normalisation
    assert np.allclose(O.rms_norm(x, weight=[2.0, 0.5, 1.0, 1.0]), [[2.4, 0.8, 0.0, 0.0]], rtol=0, atol=1e-15)
    rng = np.random.default_rng(0)
    y = O.rms_norm(rng.standard_normal((5, 3, 128)) * 7.0)
    assert np.allclose(np.sqrt(np.mean(y * y, axis=-1)), 1.0, atol=1e-12)
    # invariant to the input's scale when eps = 0
    z = rng.standard_normal((4, 128))
    assert np.allclose(O.rms_norm(z), O.rms_norm(37.0 * z), atol=1e-12)


def test_rms_norm_equals_the_library_routine():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(1)
    x = rng.standard_normal((6, 2, 128))
    w = np.exp(0.3 * rng.standard_normal(128))
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (128,), torch.from_numpy(w), 1e-6).numpy()
    assert np.allclose(O.rms_norm(x, w, 1e-6), ref, rtol=1e-13, atol=1e-13)


def test_rope_hand_examples():
    # d = 2: one pair, angle = position (theta^0 = 1): a quarter turn maps (a, b) to (-b, a)
    y = O.rope(np.array([[1.0, 2.0]]), [math.pi / 2], 10000.0)
    assert np.allclose(y, [[-2.0, 1.0]], atol=1e-15)
    # d = 4, theta = 16: frequencies 1 and 16^(-1/2) = 1/4; pairs (0, 2) and (1, 3); position 2
    x = np.array([[1.0, 1.0, 0.0, 0.0]])
    y = O.rope(x, [2], 16.0)
    assert np.allclose(y, [[math.cos(2.0), math.cos(0.5), math.sin(2.0), math.sin(0.5)]], atol=1e-15)
    # position 0 is the identity
    z = np.random.default_rng(2).standard_normal((1, 3, 128))
    assert np.array_equal(O.rope(z, [0], 5e5), z)


def test_rope_is_a_rotation_with_the_relative_position_property():
    rng = np.random.default_rng(3)
    q = rng.standard_normal((1, 128))
    k = rng.standard_normal((1, 128))
    theta = 5e5
    assert np.isclose(np.linalg.norm(O.rope(q, [12345], theta)), np.linalg.norm(q), rtol=1e-13)
    # <R_m q, R_n k> depends on m - n only
    a = (O.rope(q, [1000], theta) @ O.rope(k, [993], theta).T).item()
    b = (O.rope(q, [7], theta) @ k.T).item()
    c = (O.rope(q, [50007], theta) @ O.rope(k, [50000], theta).T).item()
    assert np.isclose(a, b, rtol=1e-10, atol=1e-10) and np.isclose(c, b, rtol=1e-9, atol=1e-9)
    # rotations compose additively
    assert np.allclose(O.rope(O.rope(q, [11], theta), [31], theta), O.rope(q, [42], theta), atol=1e-12)


def test_rope_equals_complex_multiplication():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((9, 2, 128))
    pos = np.array([0, 1, 2, 63, 64, 1000, 32767, 131071, 5])
    theta = 1e6
    z = x[..., :64] + 1j * x[..., 64:]
    w = np.exp(1j * pos[:, None, None] * theta ** (-np.arange(64) / 64.0))
    ref = z * w
    y = O.rope(x, pos, theta)
    assert np.allclose(y[..., :64], ref.real, atol=1e-12) and np.allclose(y[..., 64:], ref.imag, atol=1e-12)


def test_prepare_rows_composes_norm_then_rope_and_rounds_once():
    rng = np.random.default_rng(5)
    x = O.round_bf16(rng.standard_normal((4, 2, 128)) * 3.0)
    w = np.exp(0.25 * rng.standard_normal((2, 128)))
    pos = np.array([5, 6, 7, 8])
    y = O.prepare_rows(x, pos, 1e6, weight=w, eps=1e-6)
    assert np.array_equal(y, O.round_bf16(O.rope(O.rms_norm(x, w, 1e-6), pos, 1e6)))
    assert np.array_equal(y, O.round_bf16(y))                       # bf16-valued
    # the order matters (Norm first): normalising after the rotation would weight the wrong channels
    other = O.round_bf16(O.rms_norm(O.rope(x, pos, 1e6), w, 1e-6))
    assert not np.array_equal(y, other)
    # without Norm it is the plain rotation
    assert np.array_equal(O.prepare_rows(x, pos, 1e6, normalise=False), O.round_bf16(O.rope(x, pos, 1e6)))
