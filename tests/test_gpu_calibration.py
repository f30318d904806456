"""Calibration on the GPU (Algorithm 1 lines 4-5, 7; Eq. 4; Eq. 1) against the float64 oracle and the host calls."""
import numpy as np
import pytest

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _bits(x):
    import torch
    return torch.from_numpy(W.f32_to_bf16_bits(x).view(np.int16)).cuda()


def test_gram_accumulation_matches_the_oracle_over_several_sequences():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = W.LayerWorkload("cfg0")
    n_kv, G = wl.n_kv, wl.G
    rng = np.random.default_rng(7)
    M = torch.zeros((n_kv, 128, 128), dtype=torch.float64, device="cuda")
    H = torch.zeros_like(M)
    Mo, Ho = np.zeros((n_kv, 128, 128)), np.zeros((n_kv, 128, 128))
    for n_tok in (3000, 1, 2048, 77):                      # more than one slice, a single token, exactly one slice, a ragged tile
        pos = np.arange(n_tok)
        K = wl._keys(rng, pos)
        Q = wl._queries(rng, pos)
        B.accumulate_gram_device(_bits(K), _bits(Q), M, H)
        for h in range(n_kv):
            m, hh = O.gram_hessian(K[:, h], np.stack([Q[:, h * G + g] for g in range(G)]))
            Mo[h] += m
            Ho[h] += hh
    torch.cuda.synchronize()
    Md, Hd = M.cpu().numpy(), H.cpu().numpy()
    assert np.max(np.abs(Md - Mo)) <= 2e-6 * np.max(np.abs(Mo))
    assert np.max(np.abs(Hd - Ho)) <= 2e-6 * np.max(np.abs(Ho))
    assert np.max(np.abs(Md - Md.transpose(0, 2, 1))) <= 1e-6 * np.max(np.abs(Mo))      # symmetric up to summation order


def test_transforms_match_the_oracle_and_the_host_call():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = W.LayerWorkload("cfg1")
    Kc, Qc, _ = wl.calibration()
    n_kv, G = wl.n_kv, wl.G
    Ms, Hs = [], []
    for h in range(n_kv):
        m, hh = O.gram_hessian(Kc[:, h], np.stack([Qc[:, h * G + g] for g in range(G)]))
        Ms.append(m)
        Hs.append(hh)
    Ms, Hs = np.stack(Ms), np.stack(Hs)
    T_o, Ti_o = O.build_transforms(Ms, Hs, W.GAMMA)
    T_h, Ti_h = B.build_transforms(Ms, Hs, W.GAMMA)
    T_d, Ti_d = B.build_transforms_device(torch.from_numpy(Ms).cuda(), torch.from_numpy(Hs).cuda(), W.GAMMA)
    T_d, Ti_d = T_d.cpu().numpy().astype(np.float64), Ti_d.cpu().numpy().astype(np.float64)
    scale = np.abs(T_o).max()
    # every entry is bf16-representable; the three solvers agree except for rare one-ulp flips of the bf16 rounding
    assert np.array_equal(T_d, O.round_bf16(T_d))
    for ref in (T_o, T_h.astype(np.float64)):
        diff = np.abs(T_d - ref)
        assert diff.max() <= 2 ** -7 * scale
        assert np.mean(diff > 0) < 1e-3
    # T_invT is the inverse-transpose of the device's own rounded T: the insertion identity of Eq. 3 holds for the pair
    for h in range(n_kv):
        np.testing.assert_allclose(Ti_d[h].T @ T_d[h], np.eye(128), atol=5e-5)
    same = np.all(T_d == T_o, axis=(1, 2))
    if same.any():                                          # heads whose rounded T is identical: the inverses agree to fp32 rounding
        h = int(np.nonzero(same)[0][0])
        np.testing.assert_allclose(Ti_d[h], Ti_o[h], rtol=1e-4, atol=1e-6 * np.abs(Ti_o[h]).max())


def test_not_positive_definite_is_reported():
    import torch
    from paper_2609_38121_b200 import binding as B
    M = torch.zeros((1, 128, 128), dtype=torch.float64, device="cuda")
    H = torch.eye(128, dtype=torch.float64, device="cuda")[None].clone()
    with pytest.raises(B.WushkvError) as e:
        B.build_transforms_device(M, H, 0.0)               # Gram of rank 0 without damping
    assert e.value.status == B.ENOTPD
