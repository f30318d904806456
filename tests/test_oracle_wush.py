"""Pins for the oracle's WUSH construction (Section 3, Eq. 1; Appendix B, Theorem 2 and the
equalization identities).  Each check is against the mathematics or an independent library
routine, never against the oracle's own formula retyped."""
import numpy as np
import pytest
import scipy.linalg

from oracle import wushkv_oracle as O


def _spd_pair(rng, d, n=None, cond_boost=True):
    n = n or 4 * d
    s = np.exp(rng.standard_normal(d)) if cond_boost else np.ones(d)
    X = rng.standard_normal((d, n)) * s[:, None]
    W = rng.standard_normal((d, 3 * d)) * np.exp(0.5 * rng.standard_normal(d))[:, None]
    return X @ X.T, 2.0 * W @ W.T, X


def test_hadamard_entries_and_orthogonality():
    for d in (1, 2, 8, 128):
        H = O.hadamard(d)
        assert H.shape == (d, d)
        np.testing.assert_allclose(H @ H.T, np.eye(d), atol=1e-14)
        np.testing.assert_allclose(np.abs(H), 1.0 / np.sqrt(d), rtol=1e-15)
    H = O.hadamard(16) * 4.0
    for i in range(16):
        for j in range(16):
            assert H[i, j] == (-1) ** bin(i & j).count("1")
    with pytest.raises(ValueError):
        O.hadamard(12)


@pytest.mark.parametrize("d,gamma", [(8, 0.0), (16, 1e-2), (128, 1e-2)])
def test_factors_reproduce_their_definitions(d, gamma):
    rng = np.random.default_rng(d)
    M, H, _ = _spd_pair(rng, d)
    Md, Hd, L, lam, U, c = O.wush_factors(M, H, gamma)
    np.testing.assert_allclose(Md, M + gamma * np.trace(M) / d * np.eye(d), rtol=1e-15)
    assert np.allclose(L, np.tril(L))
    np.testing.assert_allclose(L @ L.T, Hd, rtol=1e-11, atol=1e-11 * np.abs(Hd).max())
    A = L.T @ Md @ L
    np.testing.assert_allclose(U @ np.diag(lam) @ U.T, A, rtol=1e-9, atol=1e-10 * np.abs(A).max())
    np.testing.assert_allclose(U.T @ U, np.eye(d), atol=1e-12)
    assert np.all(np.diff(lam) >= 0)
    # independent route to the spectrum: generalized symmetric problem  Md v = mu Hd^-1 v
    mu = scipy.linalg.eigh(Md, np.linalg.inv(Hd), eigvals_only=True)
    np.testing.assert_allclose(np.sort(mu), lam, rtol=1e-8)


@pytest.mark.parametrize("d,gamma", [(8, 0.0), (32, 1e-2), (128, 1e-2), (128, 0.0)])
def test_insertion_identity_and_inverse(d, gamma):
    """Eq. 3: (T k)^T (T^-T q) = k^T q for any invertible T."""
    rng = np.random.default_rng(100 + d)
    M, H, _ = _spd_pair(rng, d)
    T = O.wush(M, H, gamma)
    Tinv = np.linalg.inv(T)
    np.testing.assert_allclose(T @ Tinv, np.eye(d), atol=1e-9)
    k = rng.standard_normal((50, d))
    q = rng.standard_normal((50, d))
    kp = O.key_transform(T, k)
    qp = O.query_compensation(Tinv.T, q)
    ref = k @ q.T
    assert np.max(np.abs(kp @ qp.T - ref)) <= 1e-10 * np.max(np.abs(ref))
    # row/column convention: k' = T k as a column operation
    np.testing.assert_allclose(kp[3], T @ k[3], rtol=1e-12, atol=1e-12 * np.abs(kp[3]).max())
    np.testing.assert_allclose(qp[5], Tinv.T @ q[5], rtol=1e-12, atol=1e-12 * np.abs(qp[5]).max())


@pytest.mark.parametrize("d,gamma", [(16, 0.0), (128, 1e-2), (128, 0.3)])
def test_equalization_and_trace_identities(d, gamma):
    """Appendix B: T Md T^T = c^2 Had Lam^1/2 Had^T and T^-T Hd T^-1 = c^-2 Had Lam^1/2 Had^T, hence
    constant diagonals, tr(T Md T^T) = tr(Md), and the Theorem 2 trace product (sum sigma_i)^2."""
    rng = np.random.default_rng(7 + d)
    M, H, _ = _spd_pair(rng, d)
    Md, Hd, L, lam, U, c = O.wush_factors(M, H, gamma)
    T = O.wush(M, H, gamma)
    Tinv = np.linalg.inv(T)
    Had = O.hadamard(d)
    core = Had @ np.diag(np.sqrt(lam)) @ Had.T
    A = T @ Md @ T.T
    B = Tinv.T @ Hd @ Tinv
    np.testing.assert_allclose(A, c * c * core, rtol=1e-9, atol=1e-10 * np.abs(A).max())
    np.testing.assert_allclose(B, core / (c * c), rtol=1e-9, atol=1e-10 * np.abs(B).max())
    np.testing.assert_allclose(np.diag(A), np.trace(A) / d, rtol=1e-9)
    np.testing.assert_allclose(np.diag(B), np.trace(B) / d, rtol=1e-9)
    np.testing.assert_allclose(np.trace(A), (1 + gamma) * np.trace(M), rtol=1e-11)
    # sigma_i: singular values of Md^1/2 Hd^1/2, by an independent route (matrix square roots)
    sig = np.linalg.svd(scipy.linalg.sqrtm(Md).real @ scipy.linalg.sqrtm(Hd).real, compute_uv=False)
    prod = np.trace(A) * np.trace(B)
    np.testing.assert_allclose(prod, np.sum(sig) ** 2, rtol=1e-8)
    assert prod <= np.trace(Md) * np.trace(Hd) * (1 + 1e-12)       # orthogonal transforms give tr tr
    for _ in range(5):                                             # no invertible T does better
        R = rng.standard_normal((d, d)) + 3 * np.eye(d)
        Ri = np.linalg.inv(R)
        assert np.trace(R @ Md @ R.T) * np.trace(Ri.T @ Hd @ Ri) >= prod * (1 - 1e-9)


def test_norm_preservation_without_damping():
    """||T X||_F = ||X||_F at gamma = 0 (the role of the scalar c)."""
    rng = np.random.default_rng(3)
    M, H, X = _spd_pair(rng, 64)
    T = O.wush(M, H, 0.0)
    np.testing.assert_allclose(np.linalg.norm(T @ X), np.linalg.norm(X), rtol=1e-10)
    T2 = O.wush(M, H, 1e-2)                                      # "approximately so otherwise"
    assert abs(np.linalg.norm(T2 @ X) / np.linalg.norm(X) - 1.0) < 0.1


def test_scale_invariance():
    rng = np.random.default_rng(4)
    M, H, _ = _spd_pair(rng, 32)
    T = O.wush(M, H, 1e-2)
    T2 = O.wush(37.5 * M, 1e-3 * H, 1e-2)
    np.testing.assert_allclose(T2, T, rtol=1e-8, atol=1e-10 * np.abs(T).max())


def test_closed_form_special_cases():
    d = 16
    T = O.wush(np.eye(d), np.eye(d), 0.25)          # M = H = I: orthogonal, c = 1
    np.testing.assert_allclose(T @ T.T, np.eye(d), atol=1e-12)
    # M = diag(m), H = I, gamma = 0:  T = c Had P diag(m^-1/4), so T^T T = c^2 diag(m^-1/2)
    m = np.array([9.0, 1.0, 4.0, 16.0, 25.0, 0.25, 2.0, 3.0])
    T = O.wush(np.diag(m), np.eye(8), 0.0)
    c2 = np.sum(m) / np.sum(np.sqrt(m))
    np.testing.assert_allclose(T.T @ T, c2 * np.diag(m ** -0.5), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(np.abs(T), np.sqrt(c2 / 8) * np.tile(m ** -0.25, (8, 1)), rtol=1e-12)


def test_not_positive_definite_is_rejected():
    Z = np.zeros((4, 4))
    with pytest.raises(np.linalg.LinAlgError):
        O.wush(np.eye(4), Z, 0.0)
    with pytest.raises(np.linalg.LinAlgError):
        O.wush(Z + np.diag([1.0, 0, 0, 0]), np.eye(4), 0.0)


def test_gram_hessian_against_explicit_sums():
    rng = np.random.default_rng(5)
    K = rng.standard_normal((7, 6))
    Q = rng.standard_normal((3, 7, 6))
    M, H = O.gram_hessian(K, Q)
    M_ref = sum(np.outer(K[t], K[t]) for t in range(7))
    H_ref = 2 * sum(np.outer(Q[g, t], Q[g, t]) for g in range(3) for t in range(7))
    np.testing.assert_allclose(M, M_ref, rtol=1e-12)
    np.testing.assert_allclose(H, H_ref, rtol=1e-12)


def test_build_transforms_storage_and_identity():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(6)
    Ms, Hs = [], []
    for _ in range(2):
        M, H, _ = _spd_pair(rng, 128)
        Ms.append(M)
        Hs.append(H)
    T, TinvT = O.build_transforms(np.stack(Ms), np.stack(Hs), 1e-2)
    # T is bf16-representable, TinvT fp32-representable (library storage formats)
    t32 = torch.from_numpy(T.astype(np.float32))
    assert torch.equal(t32.to(torch.bfloat16).to(torch.float32), t32)
    assert np.array_equal(TinvT.astype(np.float32).astype(np.float64), TinvT)
    for h in range(2):
        exact = O.wush(Ms[h], Hs[h], 1e-2)
        assert np.max(np.abs(T[h] - exact) / np.abs(exact).max()) < 2 ** -8
        k = rng.standard_normal((20, 128))
        q = rng.standard_normal((20, 128))
        got = O.key_transform(T[h], k) @ O.query_compensation(TinvT[h], q).T
        ref = k @ q.T
        assert np.max(np.abs(got - ref)) < 1e-5 * np.max(np.abs(ref))   # fp32 storage of the inverse


def test_rounding_helpers_against_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.standard_normal(4000) * np.exp(6 * rng.standard_normal(4000)),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 65504.0, 1e-40, -3e-39, 2.0 ** -133]])
    x32 = x.astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_bf16(x32.astype(np.float64)), ref)
    y = x32[np.abs(x32) < 6e4]
    ref16 = torch.from_numpy(y).to(torch.float16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_fp16(y.astype(np.float64)), ref16)
    assert O.round_fp16(1e9) == 65504.0 and O.round_fp16(-1e9) == -65504.0
    # ties go to even: 1 + 2^-8 is halfway between bf16 neighbours 1 and 1 + 2^-7
    assert O.round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert O.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6
