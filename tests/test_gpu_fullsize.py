"""Parity at the benchmark configs' FULL sizes, in the launch configuration bench.py times: the cache
is built by the same `bench.Session` (library transforms, tensor-core chunk append for the prefill,
single-token append + decode for the step), and the float64 oracle recomputes sampled pieces:
the codes / scale / zero of long token ranges from the regenerated inputs, and the decode output
of sampled (sequence, KV head) groups from the library's own cache content."""
import numpy as np
import pytest

import bench
from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _unpack(sess, b, h, which, pos0, n):
    import torch
    B = sess.B
    codes = torch.empty((n, 128), dtype=torch.uint8, device="cuda")
    scale = torch.empty(n, dtype=torch.float32, device="cuda")
    zero = torch.empty(n, dtype=torch.float32, device="cuda")
    B.unpack_debug(sess.cache.desc, b, h, which, pos0, n, codes, scale, zero)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scale.cpu().numpy().astype(np.float64), zero.cpu().numpy().astype(np.float64)


def _check_append_samples(sess, b, ranges):
    """Oracle quantization of regenerated tokens of sequence b against the packed cache; returns
    (differing codes, compared codes)."""
    cfg, wl = sess.cfg, sess.wl
    S = int(sess.seq_len[b].item())
    K, V = sess.host_tokens(b)
    n_codes = n_diff = 0
    T = sess.T.astype(np.float64)
    for (p0, n) in ranges:
        n = min(n, S)
        p0 = max(0, min(p0, S - n))
        for h in range(wl.n_kv):
            Kp = O.key_transform(T[h], K[p0:p0 + n, h])
            for which in (0, 1):
                gc, gs, gz = _unpack(sess, b, h, which, p0, n)
                for i in range(n):
                    x = Kp[i] if which == 0 else V[p0 + i, h].astype(np.float64)
                    c, dl, z = O.quantize(x, cfg["bits"], W.KAPPA_K if which == 0 else W.KAPPA_V)
                    diff = np.abs(gc[i].astype(np.int32) - c.astype(np.int32))
                    assert diff.max() <= 1
                    n_codes += diff.size
                    n_diff += int(np.count_nonzero(diff))
                    assert abs(gs[i] - dl) <= 1e-3 * abs(dl) + 1e-12
                    assert abs(gz[i] - z) <= 1e-3 * max(abs(z), ((1 << cfg["bits"]) - 1) * dl) + 1e-12
    return n_diff, n_codes


def _check_decode_group(sess, out, b, h):
    """Oracle decode of KV head h of sequence b (its G query heads) on the library's cache content."""
    cfg, wl = sess.cfg, sess.wl
    G = wl.G
    S = int(sess.seq_len[b].item())
    kc, ks, kz = _unpack(sess, b, h, 0, 0, S)
    vc, vs, vz = _unpack(sess, b, h, 1, 0, S)
    km = np.stack([ks, kz], axis=1)[:, None, :]
    vm = np.stack([vs, vz], axis=1)[:, None, :]
    c = sess.cache
    kb = np.full((S, 1, 128), np.nan)
    vb = np.full((S, 1, 128), np.nan)
    sink = c.sink_kv[b, h].float().cpu().numpy().astype(np.float64)      # [2][s_sink][d]
    ring = c.ring_kv[b, h].float().cpu().numpy().astype(np.float64)      # [2][ring_cap][d]
    for p in range(min(S, cfg["s_sink"])):
        kb[p, 0], vb[p, 0] = sink[0, p], sink[1, p]
    for p in range(max(cfg["s_sink"], S - c.ring_cap), S):
        kb[p, 0], vb[p, 0] = ring[0, p % c.ring_cap], ring[1, p % c.ring_cap]
    q = sess.q_host[b, h * G:(h + 1) * G].astype(np.float64)
    ref = O.decode_attn(q, sess.TinvT[h:h + 1].astype(np.float64), kc[:, None], km, vc[:, None], vm, kb, vb, S,
                        cfg["s_sink"], cfg["s_keep"], sess.s_flush, 1.0 / np.sqrt(128))
    assert np.all(np.isfinite(ref))
    got = out[b, h * G:(h + 1) * G]
    return np.max(np.abs(got - ref)) / np.max(np.abs(ref))


def _check_prefill_rows(sess, o_chunk, b, h, rows):
    """Oracle chunk attention (empty cache before the chunk: every key is a chunk position, read as the bf16 rounding of
    the transformed key) for the G query heads of KV head h of sequence b, at the given chunk rows."""
    wl = sess.wl
    G = wl.G
    K, V = sess.host_tokens(b)
    Kp = O.round_bf16(O.key_transform(sess.T[h].astype(np.float64), K[:, h]))
    Vh = V[:, h].astype(np.float64)
    q = sess.q_chunk_host.reshape(sess.batch, sess.chunk, wl.n_q, 128)[b]
    errs = []
    for r in rows:
        for gq in range(G):
            j = h * G + gq
            qc = O.query_compensation(sess.TinvT[h].astype(np.float64), q[r, j][None].astype(np.float64))[0]
            ref = O.attention_one_query(qc, Kp[:r + 1], Vh[:r + 1], 1.0 / np.sqrt(128))
            errs.append(np.max(np.abs(o_chunk[b, r, j] - ref)) / np.max(np.abs(ref)))
    return errs


@pytest.mark.parametrize("name,groups", [
    ("cfg1", [(0, 0), (7, 3), (15, 7)]),          # Llama-3-8B-shaped, batch 16 x 32768, 2-bit
    ("cfg2", [(0, 0), (31, 5), (63, 7)]),         # 4-bit, batch 64, ragged 1024..8192
    ("cfg3", [(0, 0), (0, 5)]),                   # 70B-shaped, batch 1 x 131072, G = 8
    ("cfg4", [(0, 0), (5, 2), (7, 3)]),           # Qwen-shaped, 8 x 8192-token chunk, G = 7, then decode
])
def test_full_size_config(name, groups):
    import torch
    sess = bench.Session(name, n_steps=4)
    sess.step()                                   # one bench step: append + decode
    torch.cuda.synchronize()
    assert sess.cache.status() == 0
    S_all = sess.seq_len.cpu().numpy()
    assert np.array_equal(S_all, sess.lengths_at(1))
    out = sess.O.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(out))
    # Token ranges of one sequence, all KV heads, keys and values: its first positions (sink, first page) and
    # a long run of consecutive positions up to the very end (many page boundaries, the ragged last page, the
    # token appended by the decode step).  Config 4 checks one WHOLE 8192-token chunk: every tile and row of
    # the tensor-core append at the size the benchmark times.  Millions of codes per config, so the
    # 1e-4 bound on the mismatch rate is measured, not extrapolated.
    b0 = groups[1][0]
    S = int(S_all[b0])
    run = sess.chunk if name == "cfg4" else 2048
    ranges = [(0, run)] if name == "cfg4" else [(0, 6), (S - run, run)]
    n_diff, n_codes = _check_append_samples(sess, b0, ranges)
    assert n_codes >= 2 * sess.wl.n_kv * 128 * min(run, S)
    assert n_diff <= 1e-4 * n_codes, (n_diff, n_codes)
    for (b, h) in groups:
        err = _check_decode_group(sess, out, b, h)
        assert err <= 2e-3, f"{name}: sequence {b} KV head {h}: {err:.3e}"
    if sess.chunk:
        # the chunk's own attention outputs (Algorithm 2 line 5) at full size: sampled rows of sampled
        # (sequence, query head) pairs against the oracle's definition, row by row
        o_chunk = sess.O_chunk.cpu().numpy().astype(np.float64).reshape(sess.batch, sess.chunk, sess.wl.n_q, 128)
        assert np.all(np.isfinite(o_chunk))
        rows = [0, 1, 63, 64, 65, 4095, 4096, sess.chunk - 65, sess.chunk - 1]
        for (b, h) in groups:
            errs = _check_prefill_rows(sess, o_chunk, b, h, rows)
            assert max(errs) <= 2e-3, f"{name}: prefill rows of sequence {b} KV head {h}: {max(errs):.3e}"


def test_chunk_over_cached_context():
    """The bench's second prefill workload: config 4's heads, a 512-token chunk per sequence arriving on 4096 cached
    tokens.  Two steps, so the second one starts from the rolled-back cache (lengths and recent window restored):
    codes around the roll-back point, sampled chunk rows and the decode that follows, each against the oracle."""
    import torch
    cached, chunk = 4096, 512
    sess = bench.Session("cfg4", n_steps=4, cached=cached, chunk=chunk)
    assert sess.chunk == chunk and sess.cached == cached
    for _ in range(2):
        sess.step()
    torch.cuda.synchronize()
    assert sess.cache.status() == 0
    S_all = sess.seq_len.cpu().numpy()
    assert np.all(S_all == cached + chunk)
    cfg, wl = sess.cfg, sess.wl
    G, S = wl.G, cached + chunk
    # positions that left the recent window while the chunk was appended: quantized from the restored window rows
    n_diff, n_codes = _check_append_samples(sess, 3, [(cached - 300, 600)])
    assert n_codes == 2 * wl.n_kv * 128 * 600
    assert n_diff <= 1e-4 * n_codes, (n_diff, n_codes)
    out = sess.O.cpu().numpy().astype(np.float64)
    o_chunk = sess.O_chunk.cpu().numpy().astype(np.float64).reshape(sess.batch, chunk, wl.n_q, 128)
    assert np.all(np.isfinite(o_chunk))
    q_all = sess.q_chunk_host.reshape(sess.batch, chunk, wl.n_q, 128)
    rows = [0, 1, 17, 18, 255, 256, chunk - 2, chunk - 1]
    for (b, h) in [(0, 0), (3, 2), (7, 3)]:
        assert _check_decode_group(sess, out, b, h) <= 2e-3
        kc, ks, kz = _unpack(sess, b, h, 0, 0, S)
        vc, vs, vz = _unpack(sess, b, h, 1, 0, S)
        km = np.stack([ks, kz], axis=1)[:, None, :]
        vm = np.stack([vs, vz], axis=1)[:, None, :]
        K, V = sess.host_tokens(b)
        kb = np.full((S, 1, 128), np.nan)
        vb = np.full((S, 1, 128), np.nan)
        sink = sess.cache.sink_kv[b, h].float().cpu().numpy().astype(np.float64)
        kb[:cfg["s_sink"], 0], vb[:cfg["s_sink"], 0] = sink[0], sink[1]
        kb[cached:, 0] = O.round_bf16(O.key_transform(sess.T[h].astype(np.float64), K[cached:, h]))
        vb[cached:, 0] = V[cached:, h]
        ref = O.chunk_attn(q_all[b][:, h * G:(h + 1) * G], sess.TinvT[h:h + 1].astype(np.float64), kc[:, None], km, vc[:, None], vm,
                           kb, vb, S, chunk, cfg["s_sink"], cfg["s_keep"], sess.s_flush, 1.0 / np.sqrt(128), rows=rows)
        for r in rows:
            got = o_chunk[b, r, h * G:(h + 1) * G]
            err = np.max(np.abs(got - ref[r])) / np.max(np.abs(ref[r]))
            assert err <= 2e-3, f"sequence {b} KV head {h} chunk row {r}: {err:.3e}"
