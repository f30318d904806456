"""Writes tests/golden/oracle_regression.txt: outputs of the float64 oracle on a small seeded problem,
so that a later edit of the oracle's arithmetic cannot go unnoticed.  Calls only `oracle/` and numpy.

    python tests/golden/make_oracle_regression.py
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
from oracle import wushkv_oracle as O  # noqa: E402


def problem():
    """One KV head with two query heads, d = 128, 40 cached positions, sink 2 / keep 8 / flush 4, 2 bits."""
    rng = np.random.default_rng(20260938121)
    d, S, G = 128, 40, 2
    scale = np.exp(rng.standard_normal(d))
    K = O.round_bf16(rng.standard_normal((512, d)) * scale)
    Q = O.round_bf16(rng.standard_normal((G, 512, d)) * scale[::-1])
    M, H = O.gram_hessian(K, Q)
    T, T_invT = O.build_transforms(M[None], H[None], 1e-2)
    keys = O.round_bf16(rng.standard_normal((S, 1, d)) * scale)
    vals = O.round_bf16(rng.standard_normal((S, 1, d)))
    q = O.round_bf16(rng.standard_normal((G, d)) * scale[::-1] * 0.2)
    cache = O.LayerCache(1, d, 2, 0.96, 0.92, T)
    cache.append(keys, vals)
    kc, km, vc, vm, kb, vb = cache.arrays()
    out = O.decode_attn(q, T_invT, kc, km, vc, vm, kb, vb, S, 2, 8, 4, 1.0 / np.sqrt(d))
    return T, T_invT, kc, km, vc, vm, out


def summary():
    T, T_invT, kc, km, vc, vm, out = problem()
    rows = [
        ("T[0] trace", float(np.trace(T[0]))),
        ("T[0] frobenius^2", float(np.sum(T[0] ** 2))),
        ("T_invT[0][3][5]", float(T_invT[0][3][5])),
        ("k codes sum", float(kc.sum())),
        ("k codes weighted", float((kc.reshape(-1).astype(np.float64) * (np.arange(kc.size) % 97)).sum())),
        ("v codes sum", float(vc.sum())),
        ("k step sum", float(km[..., 0].sum())),
        ("k offset sum", float(km[..., 1].sum())),
        ("v step sum", float(vm[..., 0].sum())),
        ("v offset sum", float(vm[..., 1].sum())),
        ("out sum", float(out.sum())),
        ("out abs sum", float(np.abs(out).sum())),
        ("out[0][7]", float(out[0][7])),
        ("out[1][100]", float(out[1][100])),
    ]
    return rows


if __name__ == "__main__":
    with open(os.path.join(HERE, "oracle_regression.txt"), "w") as f:
        f.write("# written by tests/golden/make_oracle_regression.py from oracle/ alone; name | value (17 significant digits)\n")
        for name, val in summary():
            f.write(f"{name} | {val:.17g}\n")
    print("written")
