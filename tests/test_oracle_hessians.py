"""Pins of the oracle's attention-aware Hessians (Appendix C) against second differences of the actual
loss, the appendix's own expanded closed forms, and special cases."""
import numpy as np

from oracle import wushkv_oracle as O


def _problem(seed, S=7, G=2, dk=5, dv=4, dm=6):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((S, G, dk))
    K = rng.standard_normal((S, dk))
    V = rng.standard_normal((S, dv))
    W = rng.standard_normal((G, dv, dm))
    return Q, K, V, W


def _module_output(Q, K, V, W, tau):
    """y_t = sum_g W_O(g)^T V^T p_{g,t}: the attention module's output, written independently of the oracle's
    helper (explicit masked softmax per row)."""
    S, G, _ = Q.shape
    Y = np.zeros((S, W.shape[2]))
    for g in range(G):
        for t in range(S):
            z = np.array([Q[t, g] @ K[s] / tau for s in range(t + 1)])
            p = np.exp(z - z.max())
            p /= p.sum()
            Y[t] += W[g].T @ (p @ V[: t + 1])
    return Y


def _second_differences(f, n, h):
    """Hessian of the scalar function f at 0 by central second differences."""
    H = np.zeros((n, n))
    e = np.eye(n) * h
    for i in range(n):
        for j in range(n):
            H[i, j] = (f(e[i] + e[j]) - f(e[i] - e[j]) - f(-e[i] + e[j]) + f(-e[i] - e[j])) / (4 * h * h)
    return H


def test_hessians_equal_second_differences_of_the_loss():
    Q, K, V, W = _problem(0)
    tau = np.sqrt(5.0)
    Y0 = _module_output(Q, K, V, W, tau)
    HK = np.zeros((5, 5))
    HV = np.zeros((4, 4))
    for s in range(Q.shape[0]):
        def loss_k(delta, s=s):
            K2 = K.copy()
            K2[s] += delta
            return np.sum((_module_output(Q, K2, V, W, tau) - Y0) ** 2)

        def loss_v(delta, s=s):
            V2 = V.copy()
            V2[s] += delta
            return np.sum((_module_output(Q, K, V2, W, tau) - Y0) ** 2)
        HK += _second_differences(loss_k, 5, 1e-3)
        HV += _second_differences(loss_v, 4, 1e-3)
    H_K, H_V = O.attention_hessians(Q, K, V, W, tau)
    # the loss is exactly quadratic in a value perturbation; in a key perturbation the fourth-order term leaves ~h^2
    assert np.allclose(H_V, HV, rtol=1e-7, atol=1e-7)
    assert np.allclose(H_K, HK, rtol=2e-4, atol=2e-5)


def test_hessians_equal_the_expanded_closed_forms():
    Q, K, V, W = _problem(1, S=6, G=3)
    tau = 2.0
    S, G, dk = Q.shape
    P = [O.causal_probabilities(Q[:, g], K, tau) for g in range(G)]
    Oh = [P[g] @ V for g in range(G)]
    Gam = [[W[g] @ W[h].T for h in range(G)] for g in range(G)]           # head-coupling matrices
    HK = np.zeros((dk, dk))
    HV = np.zeros((V.shape[1], V.shape[1]))
    for s in range(S):
        for t in range(s, S):
            for g in range(G):
                for h in range(G):
                    w = P[g][t, s] * P[h][t, s]
                    HK += 2 / tau ** 2 * w * ((V[s] - Oh[g][t]) @ Gam[g][h] @ (V[s] - Oh[h][t])) * np.outer(Q[t, g], Q[t, h])
                    HV += 2 * w * Gam[g][h]
    H_K, H_V = O.attention_hessians(Q, K, V, W, tau)
    assert np.allclose(H_K, HK, rtol=1e-12, atol=1e-12) and np.allclose(H_V, HV, rtol=1e-12, atol=1e-12)
    # symmetric positive semi-definite
    for H in (H_K, H_V):
        assert np.allclose(H, H.T, atol=1e-12) and np.linalg.eigvalsh(H).min() >= -1e-10


def test_hessian_special_cases():
    Q, K, V, W = _problem(2, S=1, G=2)
    H_K, H_V = O.attention_hessians(Q, K, V, W, 1.5)
    # one position: p = 1 and o = v, so a key perturbation changes nothing; the value Hessian is 2 (sum_g W_g)(sum_g W_g)^T
    assert np.allclose(H_K, 0.0)
    Wsum = W.sum(axis=0)
    assert np.allclose(H_V, 2 * Wsum @ Wsum.T)
    # probabilities: rows sum to one, strictly causal zeros
    P = O.causal_probabilities(np.random.default_rng(3).standard_normal((5, 4)), np.random.default_rng(4).standard_normal((5, 4)), 2.0)
    assert np.allclose(P.sum(axis=1), 1.0) and np.all(np.triu(P, 1) == 0) and P[0, 0] == 1.0
