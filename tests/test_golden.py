"""Oracle against the text fixtures under tests/golden/: hand-worked examples of Eq. 6 and of the window
boundary of Algorithm 2 (derived without the oracle, the derivation is in each file), and a regression
record of the oracle's own outputs on a small seeded problem (written by a committed script that calls
only oracle/)."""
import importlib.util
import os

import numpy as np
import pytest

from oracle import wushkv_oracle as O

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _blocks(path):
    block = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            if not line and block:
                yield block
                block = {}
            continue
        key, val = line.split(":", 1)
        block[key.strip()] = val.split()
    if block:
        yield block


def test_eq6_worked_examples():
    n = 0
    for ex in _blocks(os.path.join(GOLDEN, "eq6_worked_examples.txt")):
        x = np.array([float(v) for v in ex["x"]])
        codes, delta, xmin = O.quantize(x, int(ex["bits"][0]), float(ex["kappa"][0]))
        assert delta == float(ex["delta"][0]) and xmin == float(ex["xmin"][0])
        assert codes.tolist() == [int(v) for v in ex["codes"]]
        assert O.dequantize(codes, delta, xmin).tolist() == [float(v) for v in ex["dequant"]]
        n += 1
    assert n == 3


def test_alg2_boundary_table():
    rows = [tuple(int(v) for v in line.split()) for line in open(os.path.join(GOLDEN, "alg2_boundary_table.txt"))
            if line.strip() and not line.startswith("#")]
    assert len(rows) >= 12
    for S, s_sink, s_keep, s_flush, n in rows:
        assert O.n_quantized(S, s_sink, s_keep, s_flush) == n
        if S <= 4096:                       # the recurrence of lines 7-8, one token at a time, lands on the same boundary
            sq = 0
            for s in range(1, S + 1):
                _, sq = O.boundary_step(sq, s, s_sink, s_keep, s_flush)
            assert max(sq - s_sink, 0) == n


def test_oracle_regression_record():
    spec = importlib.util.spec_from_file_location("make_oracle_regression", os.path.join(GOLDEN, "make_oracle_regression.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = {}
    for line in open(os.path.join(GOLDEN, "oracle_regression.txt")):
        if line.startswith("#") or "|" not in line:
            continue
        name, val = line.split("|")
        want[name.strip()] = float(val)
    got = dict(mod.summary())
    assert set(got) == set(want)
    for name, val in got.items():
        # integer-valued rows (code sums) exactly, the rest to the last few bits (BLAS summation order may differ between hosts)
        if "codes" in name:
            assert val == want[name], name
        else:
            assert val == pytest.approx(want[name], rel=1e-9, abs=1e-12), name
