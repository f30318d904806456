"""Pins for the oracle's percentile-clipped affine quantizer (Section 5.3, Eq. 6) and its packing."""
import itertools

import numpy as np
import pytest

from oracle import wushkv_oracle as O


@pytest.mark.parametrize("kappa", [0.96, 0.92, 0.5, 0.0, 1.0, 0.999])
def test_quantile_against_library_routine(kappa):
    rng = np.random.default_rng(11)
    for d in (128, 17, 2):
        x = rng.standard_normal(d) * np.exp(rng.standard_normal(d))
        assert O.quantile_abs(x, kappa) == pytest.approx(
            np.quantile(np.abs(x), kappa, method="linear"), rel=1e-13, abs=0)


def test_quantile_order_statistics_at_paper_kappas():
    """d = 128: kappa = 0.96 sits at rank 121.92 (7th / 6th largest |x|), 0.92 at rank 116.84."""
    rng = np.random.default_rng(12)
    x = rng.standard_normal(128)
    a = np.sort(np.abs(x))
    assert O.quantile_abs(x, 0.96) == pytest.approx(0.08 * a[121] + 0.92 * a[122], rel=1e-12)
    assert O.quantile_abs(x, 0.92) == pytest.approx(0.16 * a[116] + 0.84 * a[117], rel=1e-12)
    assert a[122] == np.sort(np.abs(x))[::-1][5] and a[116] == np.sort(np.abs(x))[::-1][11]


def test_clip_range_cases():
    # symmetric outlier: both ends clipped to the quantile
    x = np.concatenate([np.linspace(-1, 1, 126), [50.0, -60.0]])
    q = np.quantile(np.abs(x), 0.96)
    assert O.clip_range(x, 0.96) == (pytest.approx(-q), pytest.approx(q))
    # one-sided data: the minimum is NOT pushed below the data's own minimum
    y = np.abs(x) + 0.25
    lo, hi = O.clip_range(y, 0.96)
    assert lo == pytest.approx(y.min()) and hi == pytest.approx(np.quantile(y, 0.96))
    # kappa = 1: textbook min-max affine range
    assert O.clip_range(x, 1.0) == (pytest.approx(-60.0), pytest.approx(50.0))


@pytest.mark.parametrize("bits", [2, 4])
def test_levels_range_and_endpoints(bits):
    rng = np.random.default_rng(13)
    L = (1 << bits) - 1
    for _ in range(50):
        x = rng.standard_normal(128) * np.exp(rng.standard_normal(128))
        codes, delta, xmin = O.quantize(x, bits, 0.96)
        assert codes.dtype == np.uint8 and codes.min() >= 0 and codes.max() <= L
        xh = O.dequantize(codes, delta, xmin)
        assert len(np.unique(xh)) <= 2 ** bits
        assert codes.min() == 0 and codes.max() == L         # both ends of the grid are reached
        if bits == 2:
            assert len(np.unique(codes)) == 4                # "exactly 2^b levels" on spread-out data
        lo, hi = O.clip_range(x, 0.96)
        assert delta == pytest.approx((hi - lo) / L, rel=2 ** -10)   # fp16 storage
        assert xmin == pytest.approx(lo, rel=2 ** -10)
        # everything at or beyond the clip range lands on the end codes
        assert np.all(codes[x <= lo] == 0) and np.all(codes[x >= hi + 0.51 * delta] == L)


@pytest.mark.parametrize("bits", [2, 4])
def test_brute_force_nearest_level(bits):
    """code_i is the level of the grid {x_min + c Delta} nearest to x_i (clamping = nearest end)."""
    rng = np.random.default_rng(14)
    L = (1 << bits) - 1
    for d in (4, 6, 9):
        for _ in range(200):
            x = rng.standard_normal(d) * 3
            codes, delta, xmin = O.quantize(x, bits, 0.8)
            grid = xmin + delta * np.arange(L + 1)
            dist = np.abs(x[:, None] - grid[None, :])
            best = np.argmin(dist, axis=1)
            srt = np.sort(dist, axis=1)
            clear = (srt[:, 1] - srt[:, 0]) > 1e-9          # ignore exact ties
            assert np.array_equal(codes[clear], best[clear])


def test_exact_small_case_by_enumeration():
    """Tiny vector worked by hand: every quantity is exactly representable, so the whole of Eq. 6
    is checked including which code each value gets."""
    x = np.array([-1.5, -0.5, 0.0, 0.75, 1.5, 6.0])          # |x| sorted: 0 .5 .75 1.5 1.5 6
    # kappa = 0.8: rank 4.0 -> quantile = 1.5; range [-1.5, 1.5]; b = 2 -> Delta = 1
    codes, delta, xmin = O.quantize(x, 2, 0.8)
    assert (delta, xmin) == (1.0, -1.5)
    assert codes.tolist() == [0, 1, 2, 2, 3, 3]              # 0.0 -> 1.5 ties to even (2); 0.75 -> 2.25 -> 2
    assert O.dequantize(codes, delta, xmin).tolist() == [-1.5, -0.5, 0.5, 0.5, 1.5, 1.5]
    # all 4^3 code patterns of a 3-vector: the chosen one minimises the clipped reconstruction error
    y = np.array([0.1, 0.9, -0.6])
    c, dl, mn = O.quantize(y, 2, 1.0)
    best = min(itertools.product(range(4), repeat=3),
               key=lambda cc: np.sum((mn + dl * np.array(cc) - y) ** 2))
    assert tuple(c.tolist()) == best


@pytest.mark.parametrize("bits", [2, 4])
def test_equivariance_and_mirror(bits):
    rng = np.random.default_rng(15)
    L = (1 << bits) - 1
    x = np.round(rng.standard_normal(128) * 64) / 256.0       # coarse dyadic values
    codes, delta, xmin = O.quantize(x, bits, 0.96)
    c4, d4, m4 = O.quantize(4.0 * x, bits, 0.96)              # power-of-two scale commutes with fp16 rounding
    assert np.array_equal(c4, codes) and d4 == 4.0 * delta and m4 == 4.0 * xmin
    cm, dm, mm = O.quantize(-x, bits, 0.96)                    # sign flip mirrors the grid
    lo, hi = O.clip_range(x, 0.96)
    assert mm == O.round_fp16(-hi) and dm == delta
    # mirrored grid: code L - c, except where fp16 rounding of the two offsets moves a near-tie
    t = (x - xmin) / delta
    clear = np.abs(t - np.floor(t) - 0.5) > 0.02
    assert clear.sum() > 64 and np.array_equal(cm[clear], L - codes[clear])


def test_kappa_one_is_min_max_affine():
    rng = np.random.default_rng(16)
    x = np.round(rng.standard_normal(128) * 32) / 32.0
    for bits in (2, 4, 8):
        L = (1 << bits) - 1
        codes, delta, xmin = O.quantize(x, bits, 1.0)
        assert xmin == x.min() and delta == O.round_fp16((x.max() - x.min()) / L)
        ref = np.clip(np.rint((x - x.min()) / delta), 0, L)
        assert np.array_equal(codes, ref)
        assert np.max(np.abs(O.dequantize(codes, delta, xmin) - x)) <= 0.5 * delta * (1 + 2 ** -9) + L * delta * 2 ** -10


def test_degenerate_groups():
    for v in (0.0, 3.25, -7.0):
        codes, delta, xmin = O.quantize(np.full(128, v), 2, 0.96)
        assert delta == 0.0 and not codes.any()
        assert np.array_equal(O.dequantize(codes, delta, xmin), np.full(128, v))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_pack_roundtrip_and_layout(bits):
    rng = np.random.default_rng(17)
    codes = rng.integers(0, 1 << bits, size=(5, 3, 128), dtype=np.uint8)
    packed = O.pack_codes(codes, bits)
    assert packed.shape == (5, 3, 128 * bits // 8) and packed.dtype == np.uint8
    assert np.array_equal(O.unpack_codes(packed, bits), codes)
    one = np.zeros(128, np.uint8)
    one[:4] = [1, 2, 3, 1]
    if bits == 2:
        assert O.pack_codes(one, 2)[0] == 1 | (2 << 2) | (3 << 4) | (1 << 6)
    elif bits == 3:
        # 48 bytes per 128-channel vector; the stream 001 010 011 001 (low bit first per code) by hand:
        # bits 0..11 = 1,0,0, 0,1,0, 1,1,0, 1,0,0 -> byte 0 = 0b11010001, byte 1 low nibble = 0b0010
        one[:4] = [1, 2, 3, 1]
        p3 = O.pack_codes(one, 3)
        assert p3.shape == (48,) and p3[0] == 0b11010001 and p3[1] == 0b0010 and not p3[2:].any()
        seven = np.full(128, 7, np.uint8)
        assert np.all(O.pack_codes(seven, 3) == 0xFF)
    else:
        assert O.pack_codes(one, 4)[:2].tolist() == [1 | (2 << 4), 3 | (1 << 4)]


def test_quantize_rows_matches_single():
    rng = np.random.default_rng(18)
    X = rng.standard_normal((9, 128))
    C, D, Z = O.quantize_rows(X, 4, 0.92)
    for i in range(9):
        c, dl, z = O.quantize(X[i], 4, 0.92)
        assert np.array_equal(C[i], c) and D[i] == dl and Z[i] == z
