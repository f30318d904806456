"""Norm and RoPE fused into the append and the query preparation (Algorithm 2 lines 1-2 ahead of line 3):
wushkv_append_projected / wushkv_decode_attn_projected against the oracle.

The fused kernels compute normalisation and rotation in fp32 and round once to bf16; the oracle does the
same in float64.  Where the float64 value sits within the fp32 path's error of a bf16 rounding boundary the
two may round differently, and one bf16 unit in one channel moves all 128 transformed channels of that
token a little.  Both sides take the rounding decision in their own precision, so the comparison is exact on
the vectors that have no such channel (the large majority) and toleranced on the others."""
import numpy as np
import pytest

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W
from tests.harness import CODE_MISMATCH_MAX, DECODE_TOL, Layer

pytestmark = pytest.mark.gpu

EPS = 1e-6
FP32_SLACK = 5e-7          # error allowed to the fp32 normalisation + rotation, relative to the magnitude of the channel pair


def _prepared(x_proj, positions, theta, weight, normalise):
    """Oracle's normalised, rotated, bf16-rounded vectors and the mask of vectors [n][heads] that hold a channel
    whose rounding the fp32 path may decide differently."""
    y = O.rms_norm(x_proj, weight, EPS) if normalise else np.asarray(x_proj, dtype=np.float64)
    r = O.rope(y, positions, theta)
    pair = np.abs(y[..., :64]) + np.abs(y[..., 64:])
    slack = FP32_SLACK * np.concatenate([pair, pair], axis=-1)
    ambiguous = np.any(O.round_bf16(r - slack) != O.round_bf16(r + slack), axis=-1)
    return O.round_bf16(r), ambiguous


def _wl(seed, batch, n_q, n_kv, bits, theta=1e6):
    return W.LayerWorkload(dict(seed=seed, batch=batch, n_q=n_q, n_kv=n_kv, ctx=0, theta=theta, bits=bits, s_sink=4,
                                s_keep=64, rmsnorm=True, ragged=None, prefill_chunk=0))


def _pair(wl, lengths, bits, normalise, weights=True):
    """(plain layer fed the oracle-prepared keys, projected layer fed the projected keys, ambiguity masks, projected queries)"""
    from paper_2609_38121_b200 import binding as B
    plain = Layer(wl, lengths, bits, 4, 64, 1, max_seq_len=max(lengths) + 64)
    fused = Layer(wl, lengths, bits, 4, 64, 1, max_seq_len=max(lengths) + 64)
    kw = wl.gain_k if weights else None
    qw = wl.gain_q if weights else None
    fused.prologue = B.Prologue(wl.theta, max(lengths) + 64, normalise=normalise, k_weight=kw, q_weight=qw, eps=EPS)
    masks, qproj = [], []
    for b, n in enumerate(lengths):
        Kp, Qp = wl.projected(b, n)
        V = plain.tokens[b][1]
        Kprep, amb = _prepared(Kp, np.arange(n), wl.theta, None if kw is None else kw[None], normalise)
        plain.tokens[b] = (Kprep.astype(np.float32), V)
        fused.tokens[b] = (Kp, V)
        masks.append(amb)
        qproj.append(Qp)
    return plain, fused, masks, qproj


def _compare_caches(plain, fused, masks, lengths, n_kv):
    """Keys: bit-identical codes / step / offset / bf16 copies on unambiguous vectors, within the usual tolerances on the
    others; values: bit-identical everywhere.  Returns (share of ambiguous vectors, code mismatch rate on them)."""
    n_amb = n_all = 0
    amb_codes = amb_diff = 0
    for b, n in enumerate(lengths):
        kb_p, vb_p = plain.gpu_window_arrays(b)
        kb_f, vb_f = fused.gpu_window_arrays(b)
        assert np.array_equal(np.isnan(kb_p), np.isnan(kb_f))
        assert np.array_equal(np.nan_to_num(vb_p), np.nan_to_num(vb_f))
        for h in range(n_kv):
            clean = ~masks[b][:, h]
            n_amb += int(np.count_nonzero(~clean))
            n_all += n
            cp, sp, zp = plain.gpu_codes(b, h, 0)
            cf, sf, zf = fused.gpu_codes(b, h, 0)
            assert np.array_equal(cp[clean], cf[clean]), f"key codes differ on an unambiguous vector (b={b} h={h})"
            assert np.array_equal(sp[clean], sf[clean]) and np.array_equal(zp[clean], zf[clean])
            live = ~np.isnan(kb_p[:, h, 0])
            assert np.array_equal(kb_p[live & clean, h], kb_f[live & clean, h])
            d = np.abs(cp[~clean].astype(np.int32) - cf[~clean].astype(np.int32))
            if d.size:
                assert d.max() <= 1
                amb_codes += d.size
                amb_diff += int(np.count_nonzero(d))
                assert np.allclose(sp[~clean], sf[~clean], rtol=2e-2)
            vp = plain.gpu_codes(b, h, 1)
            vf = fused.gpu_codes(b, h, 1)
            assert all(np.array_equal(x, y) for x, y in zip(vp, vf))
    return n_amb / max(n_all, 1), amb_diff / max(amb_codes, 1)


@pytest.mark.parametrize("bits,normalise,weights", [(2, True, True), (4, True, False), (2, False, False)])
def test_projected_append_all_paths_match_the_oracle_prepared_append(bits, normalise, weights):
    # sequence lengths chosen so that the first call takes the tensor-core chunk path (>= 128 new tokens) and the
    # second the single-token path; the third layer below takes the CUDA-core rows path
    wl = _wl(41, 3, 8, 2, bits)
    lengths = [700, 129, 260]
    plain, fused, masks, _ = _pair(wl, lengths, bits, normalise, weights)
    for L in (plain, fused):
        L.fill()                                           # chunk call, then one token per sequence
    assert plain.check_append_parity() <= CODE_MISMATCH_MAX            # the reference side equals the oracle
    share, rate = _compare_caches(plain, fused, masks, lengths, wl.n_kv)
    assert share <= 0.25, share
    assert rate <= 0.05, rate
    assert fused.cache.status() == 0 and plain.cache.status() == 0


def test_projected_append_rows_path():
    wl = _wl(43, 2, 8, 2, 2, theta=1e4)
    lengths = [57, 90]
    plain, fused, masks, _ = _pair(wl, lengths, 2, True)
    for L in (plain, fused):
        L.append_step([40, 70])                            # fewer than 128 new tokens per sequence: CUDA-core rows path
        L.append_step([17, 20])
    assert plain.check_append_parity() <= CODE_MISMATCH_MAX
    share, rate = _compare_caches(plain, fused, masks, lengths, wl.n_kv)
    assert share <= 0.25 and rate <= 0.05


@pytest.mark.parametrize("n_q,n_kv", [(8, 2), (16, 2)])
def test_projected_decode_matches_the_oracle(n_q, n_kv):
    wl = _wl(47, 3, n_q, n_kv, 2)
    lengths = [900, 130, 333]
    plain, fused, masks, qproj = _pair(wl, lengths, 2, True)
    fused.fill()
    Qp = np.stack([qproj[b][-1] for b in range(len(lengths))])                    # the query at the newest position
    got, _ = fused.decode(Qp, projected=True)
    prepared = [_prepared(Qp[b][None], [n - 1], wl.theta, wl.gain_q[None], True) for b, n in enumerate(lengths)]
    # the plain call on the oracle-prepared queries, for the exact comparison below
    plain_out, _ = fused.decode(np.stack([p[0][0] for p in prepared]).astype(np.float32))
    n_clean = 0
    for b, n in enumerate(lengths):
        qprep, amb = prepared[b]
        ref = fused.oracle_decode_on_gpu_cache(b, qprep[0])
        err = np.max(np.abs(got[b] - ref)) / np.max(np.abs(ref))
        assert err <= DECODE_TOL, f"sequence {b}: {err:.3e}"
        # a query head without an ambiguous channel gives exactly what the plain call gives on the prepared query
        for j in range(n_q):
            if not amb[0, j]:
                n_clean += 1
                assert np.array_equal(plain_out[b, j], got[b, j]), (b, j)
    assert n_clean >= n_q // 2                                                     # the exact comparison did run
    assert fused.cache.status() == 0


@pytest.mark.parametrize("copies", [0, 1])
def test_projected_chunk_attention_matches_the_oracle(copies, test_option):
    """wushkv_prefill_attn_projected after wushkv_append_projected: a first chunk on the empty cache, then a second chunk
    over it, against the oracle's chunk attention on oracle-prepared keys and queries (cache content: the GPU's codes).
    Once on the default kernels (tcgen05 transforms that normalise and rotate the rows the bulk tensor copies staged) and
    once without bulk tensor copies (mma.sync transforms with their own row fix-up)."""
    test_option("prefill_no_tma", copies)
    wl = _wl(53, 2, 8, 2, 2)
    lengths = [450, 290]
    plain, fused, masks, qproj = _pair(wl, lengths, 2, True)
    done = [0, 0]
    for counts in ([300, 200], [150, 90]):
        qs = [qproj[b][done[b]:done[b] + c] for b, c in enumerate(counts)]
        outs, _ = fused.prefill(counts, queries=qs)
        plain.append_step(counts)                               # the oracle's cache of the prepared keys (and the plain GPU cache)
        for b, c in enumerate(counts):
            S = done[b] + c
            kc = np.zeros((S, wl.n_kv, 128), np.uint8); vc = np.zeros_like(kc)
            km = np.zeros((S, wl.n_kv, 2)); vm = np.zeros_like(km)
            for h in range(wl.n_kv):
                cc, sc, zc = fused.gpu_codes(b, h, 0, n=S); kc[:, h], km[:, h, 0], km[:, h, 1] = cc, sc, zc
                cc, sc, zc = fused.gpu_codes(b, h, 1, n=S); vc[:, h], vm[:, h, 0], vm[:, h, 1] = cc, sc, zc
            _, _, _, _, kb, vb = plain.oracle[b].arrays()
            qprep, _ = _prepared(qs[b], np.arange(done[b], S), wl.theta, wl.gain_q[None], True)
            ref = O.chunk_attn(qprep, fused.TinvT, kc, km, vc, vm, kb, vb, S, c, 4, 64, 1, 1.0 / np.sqrt(128))
            for r in range(c):
                err = np.max(np.abs(outs[b][r] - ref[r])) / np.max(np.abs(ref[r]))
                assert err <= DECODE_TOL, (b, r, err)
            done[b] = S
    assert fused.cache.status() == 0


def test_position_beyond_the_rotary_table_is_flagged():
    from paper_2609_38121_b200 import binding as B
    wl = _wl(49, 1, 8, 2, 2)
    L = Layer(wl, [40], 2, 4, 64, 1, max_seq_len=128)
    Kp, _ = wl.projected(0, 40)
    L.tokens[0] = (Kp, L.tokens[0][1])
    L.prologue = B.Prologue(wl.theta, 32, normalise=True, eps=EPS)                 # table shorter than the sequence
    L.append_step([40])
    assert L.cache.status() & B.DEV_ROPE_RANGE
    assert int(L.seq_len[0]) == 40
