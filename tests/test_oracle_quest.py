"""Pins for the oracle's QuEST quantizer (Section 4.3, Eq. 5, Lemma 1)."""
import math

import numpy as np
import pytest

from oracle import wushkv_oracle as O


def _grid_mse_numeric(alpha, bits, n=400001, zmax=10.0):
    """E[(Q_alpha(z) - z)^2] by plain trapezoid integration over a fine grid: independent of the oracle's closed form."""
    z = np.linspace(-zmax, zmax, n)
    levels = np.linspace(-alpha, alpha, 1 << bits)
    q = levels[np.argmin(np.abs(z[:, None] - levels[None, :]), axis=1)]
    w = np.exp(-0.5 * z * z) / math.sqrt(2 * math.pi)
    return np.trapezoid((q - z) ** 2 * w, z)


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_alpha_is_the_gaussian_mse_minimiser_by_brute_force(bits):
    a = O.quest_alpha(bits)
    grid = a + np.linspace(-0.05, 0.05, 41)
    errs = [_grid_mse_numeric(x, bits, n=100001) for x in grid]
    assert abs(grid[int(np.argmin(errs))] - a) <= 0.0026              # within the scan's resolution
    assert _grid_mse_numeric(a, bits) == pytest.approx(O._gauss_grid_mse(a, bits), rel=1e-6)
    # far from the optimum the error is clearly larger
    assert _grid_mse_numeric(0.5 * a, bits, n=100001) > 1.2 * min(errs) and _grid_mse_numeric(2 * a, bits, n=100001) > 1.2 * min(errs)


def test_alpha_values():
    # one bit: the two levels +-alpha minimise E(|z| - alpha)^2 at alpha = E|z| = sqrt(2 / pi)
    assert O.quest_alpha(1) == pytest.approx(math.sqrt(2.0 / math.pi), abs=1e-7)
    # the classical optimal uniform quantizers of a unit Gaussian (endpoint = outermost level)
    assert O.quest_alpha(2) == pytest.approx(1.4935, abs=2e-4)
    assert O.quest_alpha(3) == pytest.approx(2.0511, abs=2e-4)
    assert O.quest_alpha(4) == pytest.approx(2.5141, abs=2e-4)
    assert O.quest_alpha(1) < O.quest_alpha(2) < O.quest_alpha(3) < O.quest_alpha(4)


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_lemma1_clip_bound(bits):
    """Lemma 1: E[(|z| - alpha_b)_+^2] <= (2^b - 1)^-2."""
    a = O.quest_alpha(bits)
    z = np.linspace(0, 12, 600001)
    w = np.exp(-0.5 * z * z) / math.sqrt(2 * math.pi)
    tail = 2 * np.trapezoid(np.maximum(z - a, 0) ** 2 * w, z)
    assert tail <= (2 ** bits - 1) ** -2
    assert tail > 0


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_levels_bin_centres_and_clipping(bits):
    rng = np.random.default_rng(70 + bits)
    d = 128
    half, levels = 1 << (bits - 1), (1 << bits) - 1
    for trial in range(30):
        x = rng.standard_normal(d) * np.exp(rng.standard_normal(d) * (trial % 3))
        codes, delta, xmin = O.quest_quantize(x, bits)
        assert codes.min() >= 0 and codes.max() <= levels
        rms = np.sqrt(np.mean(x * x))
        assert delta == pytest.approx(2 * O.quest_alpha(bits) / levels * rms, rel=2 ** -11)      # fp16 storage of the step
        assert xmin == pytest.approx(-delta * levels / 2, rel=2 ** -11)
        xhat = O.dequantize(codes, delta, xmin)
        centres = delta * (np.arange(-half, half) + 0.5)
        # reconstruction at bin centres (up to the fp16 rounding of the stored offset)
        assert np.all(np.min(np.abs(xhat[:, None] - centres[None, :]), axis=1) <= 2 ** -10 * abs(xmin) + 1e-12)
        inside = np.abs(x) <= delta * half
        assert np.all(np.abs(x[inside] - xhat[inside]) <= delta / 2 + 2 ** -10 * abs(xmin))
        # outside the grid: the endpoint with the sign of the entry, +-alpha_b * RMS
        out = ~inside
        assert np.all(np.sign(xhat[out]) == np.sign(x[out]))
        assert np.allclose(np.abs(xhat[out]), O.quest_alpha(bits) * rms, rtol=2 ** -9)
        # brute force: the code is the index of the nearest bin centre
        nearest = np.argmin(np.abs(x[:, None] - centres[None, :]), axis=1)
        assert np.array_equal(codes, nearest)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_zero_group_symmetry_and_scaling(bits):
    d, levels = 128, (1 << bits) - 1
    codes, delta, xmin = O.quest_quantize(np.zeros(d), bits)
    assert delta == 0.0 and np.all(O.dequantize(codes, delta, xmin) == 0.0)                     # Q(0) = 0
    rng = np.random.default_rng(75)
    x = rng.standard_normal(d)
    c1, d1, m1 = O.quest_quantize(x, bits)
    c2, d2, m2 = O.quest_quantize(-x, bits)
    assert d1 == d2 and m1 == m2 and np.array_equal(c2, levels - c1)                             # odd symmetry
    c3, d3, m3 = O.quest_quantize(8.0 * x, bits)
    assert np.array_equal(c3, c1) and d3 == 8.0 * d1 and m3 == 8.0 * m1                         # positive-scale equivariance
    # a permutation of the entries permutes the codes and leaves the step alone (the step depends on the norm only)
    perm = rng.permutation(d)
    c4, d4, _ = O.quest_quantize(x[perm], bits)
    assert d4 == d1 and np.array_equal(c4, c1[perm])


def test_cache_with_quest_quantizer():
    rng = np.random.default_rng(76)
    K = rng.standard_normal((10, 1, 128))
    V = rng.standard_normal((10, 1, 128))
    cache = O.LayerCache(1, 128, 3, 0.96, 0.92, np.eye(128)[None], quantizer="quest")
    cache.append(K, V)
    kc, km, vc, vm, kb, vb = cache.arrays()
    for t in range(10):
        c, dl, z = O.quest_quantize(K[t, 0], 3)
        assert np.array_equal(kc[t, 0], c) and km[t, 0, 0] == dl and km[t, 0, 1] == z
        c, dl, z = O.quest_quantize(V[t, 0], 3)
        assert np.array_equal(vc[t, 0], c) and vm[t, 0, 0] == dl and vm[t, 0, 1] == z
