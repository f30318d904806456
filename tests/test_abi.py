"""CPU-side checks of the C ABI: the library loads, exports every symbol the header declares,
rejects bad arguments on the host before touching CUDA, and its host-side calibration arithmetic
(Eq. 1, Eq. 4) agrees with the float64 oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import binding as B
from paper_2609_38121_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    text = open(os.path.join(ROOT, "include", "wushkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(wushkv_[a-z_]+)\s*\(", text))
    assert declared, "no declarations found"
    assert set(B.EXPORTS) <= declared
    for name in declared:
        assert hasattr(B.lib, name), f"{name} declared in wushkv.h but not exported"


def test_struct_layout_matches_header_field_order():
    text = open(os.path.join(ROOT, "include", "wushkv.h")).read()
    body = re.search(r"typedef struct wushkv_cache \{(.*?)\} wushkv_cache;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        parts = decl.split(",")
        for p in parts:
            names.append(re.findall(r"[A-Za-z_][A-Za-z_0-9]*", p)[-1])
    assert names == [f[0] for f in B.wushkv_cache._fields_]
    assert C.sizeof(B.wushkv_cache) == 16 * 4 + 8 + 7 * 8


def test_status_strings_and_page_bytes():
    assert B.status_string(0) == "ok"
    assert "positive definite" in B.status_string(B.ENOTPD)
    assert B.page_bytes(8, 128, 2, 64) == 8 * 4608       # 64 tokens x (2 x 32 B codes + 8 B meta)
    assert B.page_bytes(8, 128, 4, 64) == 8 * 8704
    assert B.page_bytes(8, 128, 3, 64) == 8 * 6656       # 64 tokens x (2 x 48 B codes + 8 B meta)
    assert B.page_bytes(8, 64, 2, 64) == 0 and B.page_bytes(8, 128, 5, 64) == 0


def test_host_validation_rejects_bad_arguments_without_cuda():
    desc = B.wushkv_cache()                                  # all zero
    assert B.lib.wushkv_append(C.byref(desc), 1, None, None, None, 1, 1, None, None, None) == B.EINVAL
    assert B.lib.wushkv_decode_attn(C.byref(desc), 1, None, None, 64, None, None, None, 0, None) == B.EINVAL
    assert B.lib.wushkv_decode_step(C.byref(desc), 1, None, None, None, 64, None, None, None, None, None, 0, None) == B.EINVAL
    assert B.lib.wushkv_decode_step_host(C.byref(desc), 1, None, None, None, 64, None, None, None, None, None, 0, None, 0,
                                         None) != B.OK
    assert B.lib.wushkv_decode_workspace_bytes(C.byref(desc), 1, 64) == 0
    assert B.lib.wushkv_build_transforms(1, 12, None, None, 0.0, None, None) == B.EINVAL
    with pytest.raises(B.WushkvError):
        B.build_transforms(np.zeros((1, 8, 8)), np.eye(8)[None], 0.0)     # Gram of rank 0, no damping: not PD


def _canon_close(T_lib, T_ora):
    scale = np.abs(T_ora).max()
    diff = np.abs(T_lib.astype(np.float64) - T_ora)
    # both sides round the same float64 matrix to bf16; allow rare one-ulp flips where the two eigensolvers differ in the last bits
    assert diff.max() <= 2 ** -7 * scale
    assert np.mean(diff > 0) < 1e-3


def test_build_transforms_matches_oracle_on_workload_statistics():
    wl = W.LayerWorkload("cfg0")
    Kc, Qc, _ = wl.calibration()
    n_kv, G, d = wl.n_kv, wl.G, 128
    M = np.zeros((n_kv, d, d))
    H = np.zeros((n_kv, d, d))
    B.accumulate_gram(W.f32_to_bf16_bits(Kc), W.f32_to_bf16_bits(Qc), M, H)
    for h in range(n_kv):
        Mo, Ho = O.gram_hessian(Kc[:, h], np.stack([Qc[:, h * G + g] for g in range(G)]))
        np.testing.assert_allclose(M[h], Mo, rtol=1e-12, atol=1e-9 * np.abs(Mo).max())
        np.testing.assert_allclose(H[h], Ho, rtol=1e-12, atol=1e-9 * np.abs(Ho).max())
    T, TinvT = B.build_transforms(M, H, W.GAMMA)
    To, TinvTo = O.build_transforms(M, H, W.GAMMA)
    for h in range(n_kv):
        _canon_close(T[h], To[h])
        # the stored pair satisfies the insertion identity (Eq. 3) on its own
        eye = TinvT[h].astype(np.float64).T @ T[h].astype(np.float64)
        assert np.max(np.abs(eye - np.eye(d))) < 1e-4
        assert np.max(np.abs(TinvT[h] - TinvTo[h])) <= 1e-3 * np.abs(TinvTo[h]).max() or np.array_equal(T[h], To[h].astype(np.float32))
    # accumulation over two sequences equals one pass over their concatenation (Algorithm 1)
    M2 = np.zeros_like(M)
    H2 = np.zeros_like(H)
    B.accumulate_gram(W.f32_to_bf16_bits(Kc[:200]), W.f32_to_bf16_bits(Qc[:200]), M2, H2)
    B.accumulate_gram(W.f32_to_bf16_bits(Kc[200:]), W.f32_to_bf16_bits(Qc[200:]), M2, H2)
    np.testing.assert_allclose(M2, M, rtol=1e-12, atol=1e-9 * np.abs(M).max())
    np.testing.assert_allclose(H2, H, rtol=1e-12, atol=1e-9 * np.abs(H).max())


def test_build_transforms_small_orders_and_special_cases():
    rng = np.random.default_rng(0)
    for d in (2, 8, 32):
        X = rng.standard_normal((d, 4 * d)) * np.exp(rng.standard_normal(d))[:, None]
        Wt = rng.standard_normal((d, 3 * d))
        M, H = X @ X.T, 2 * Wt @ Wt.T
        T, TinvT = B.build_transforms(M[None], H[None], 1e-2)
        To, _ = O.build_transforms(M[None], H[None], 1e-2)
        _canon_close(T[0], To[0])
    T, _ = B.build_transforms(np.eye(16)[None], np.eye(16)[None], 0.25)       # M = H = I: orthogonal
    np.testing.assert_allclose(T[0].astype(np.float64) @ T[0].astype(np.float64).T, np.eye(16), atol=2e-2)
