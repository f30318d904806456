"""Attention-aware Hessians of Appendix C on the GPU (wushkv_accumulate_attention_hessians_device) against the
oracle's literal Jacobian form, on seeded calibration tensors (keys / queries after Norm and RoPE, raw values, a
slice of the synthetic output projection)."""
import numpy as np
import pytest

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = 2e-4          # of the largest entry: fp32 products and exponentials, float64 sums over tokens


def _inputs(n_q, n_kv, n_tok, d_model, seed=61):
    wl = W.LayerWorkload(dict(seed=seed, batch=1, n_q=n_q, n_kv=n_kv, ctx=0, theta=1e4, bits=2, s_sink=4, s_keep=64,
                              rmsnorm=False, ragged=None, prefill_chunk=0))
    Kc, Qc, Vraw = wl.calibration()
    K, Q, V = Kc[:n_tok], Qc[:n_tok], W.bf16_round_f32(Vraw[:n_tok])
    WO = np.ascontiguousarray(wl.W_O[:, :, :, :d_model].reshape(n_q, 128, d_model), dtype=np.float32)
    return wl, K, Q, V, WO


def _gpu(K, Q, V, WO, tau, calls=1):
    import torch
    from paper_2609_38121_b200 import binding as B
    dev = "cuda"
    bits = lambda x: torch.from_numpy(W.f32_to_bf16_bits(x).view(np.int16)).to(dev)  # noqa: E731
    n_kv = K.shape[1]
    HK = torch.zeros((n_kv, 128, 128), dtype=torch.float64, device=dev)
    HV = torch.zeros_like(HK)
    for _ in range(calls):
        B.accumulate_attention_hessians_device(bits(K), bits(Q), bits(V), torch.from_numpy(WO).to(dev), tau, HK, HV)
    torch.cuda.synchronize()
    return HK.cpu().numpy(), HV.cpu().numpy()


@pytest.mark.parametrize("n_q,n_kv,n_tok", [(8, 2, 70), (3, 1, 45), (2, 2, 33), (8, 1, 40), (7, 1, 36)])
def test_attention_hessians_match_the_oracle(n_q, n_kv, n_tok):
    wl, K, Q, V, WO = _inputs(n_q, n_kv, n_tok, 32)
    tau = float(np.sqrt(128))
    HK, HV = _gpu(K, Q, V, WO, tau)
    G = n_q // n_kv
    for h in range(n_kv):
        rk, rv = O.attention_hessians(Q[:, h * G:(h + 1) * G], K[:, h], V[:, h], WO[h * G:(h + 1) * G], tau)
        assert np.max(np.abs(HK[h] - rk)) <= TOL * np.max(np.abs(rk)), (h, np.max(np.abs(HK[h] - rk)) / np.max(np.abs(rk)))
        assert np.max(np.abs(HV[h] - rv)) <= TOL * np.max(np.abs(rv)), (h, np.max(np.abs(HV[h] - rv)) / np.max(np.abs(rv)))
        assert np.allclose(HK[h], HK[h].T, atol=1e-9 * np.max(np.abs(rk)))


def test_hessians_accumulate_over_calls_and_feed_the_transform_builder():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl, K, Q, V, WO = _inputs(8, 2, 160, 48)
    tau = float(np.sqrt(128))
    one_k, one_v = _gpu(K, Q, V, WO, tau)
    two_k, two_v = _gpu(K, Q, V, WO, tau, calls=2)
    assert np.allclose(two_k, 2 * one_k, rtol=1e-12) and np.allclose(two_v, 2 * one_v, rtol=1e-12)
    # the WUSH-A key transform: the same builder, fed the Gram matrix and the attention-aware Hessian
    M = np.stack([K[:, h].astype(np.float64).T @ K[:, h].astype(np.float64) for h in range(2)])
    T, TinvT = B.build_transforms_device(torch.from_numpy(M).cuda(), torch.from_numpy(one_k).cuda(), W.GAMMA)
    To, _ = O.build_transforms(M, one_k, W.GAMMA)
    T = T.cpu().numpy().astype(np.float64)
    # both sides round the same float64 matrix to bf16; rare one-unit flips where the eigensolvers differ in the last bits
    ulp = np.maximum(np.abs(To), 2.0 ** -120) * 2.0 ** -7
    assert np.all(np.abs(T - To) <= ulp) and np.mean(T != To) < 2e-3


def test_group_sizes_beyond_eight_are_refused():
    from paper_2609_38121_b200 import binding as B
    assert B.lib.wushkv_attention_hessians_workspace_bytes(1, 9, 128, 64) == 0
    assert B.lib.wushkv_attention_hessians_workspace_bytes(1, 8, 128, 64) > 0
