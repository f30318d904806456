"""Shared helpers of the GPU parity tests: build the same seeded layer on both sides (CUDA library
through its C ABI binding, float64 oracle) and compare stage by stage.  Tolerances are the ones the
benchmark definition states: codes bit-exact except at float rounding ties (at most 1e-4 of them off
by one level), scale / zero within 1e-3 relative, decode output within 2e-3 of its max-abs value when
the oracle is fed the library's own codes."""
from __future__ import annotations

import numpy as np

from oracle import wushkv_oracle as O
from paper_2609_38121_b200 import workloads as W

CODE_MISMATCH_MAX = 1e-4
META_RTOL = 1e-3
DECODE_TOL = 2e-3


def oracle_transforms(wl):
    """(T_K, T_K_invT, T_V) from the workload's calibration batch, all by the oracle (float64)."""
    Kc, Qc, Vraw = wl.calibration()
    n_kv, G = wl.n_kv, wl.G
    Ms, Hs, TV = [], [], []
    for h in range(n_kv):
        M, H = O.gram_hessian(Kc[:, h], np.stack([Qc[:, h * G + g] for g in range(G)]))
        Ms.append(M)
        Hs.append(H)
        Vh = Vraw[:, h].astype(np.float64)
        Wo = wl.W_O[h].astype(np.float64)
        TV.append(O.wush(Vh.T @ Vh, 2 * sum(Wo[g] @ Wo[g].T for g in range(G)), W.GAMMA))
    T, TinvT = O.build_transforms(np.stack(Ms), np.stack(Hs), W.GAMMA)
    return T, TinvT, np.stack(TV)


class Layer:
    """One layer on both sides.  ``lengths`` are the final context lengths; ``chunks`` is a list of
    per-step new-token counts per sequence (list of lists) or None for prefill(S-1) + decode(1)."""

    def __init__(self, wl, lengths, bits, s_sink, s_keep, s_flush, lag=0, kappa_k=W.KAPPA_K, kappa_v=W.KAPPA_V,
                 page_shuffle_seed=None, max_seq_len=None, ring_cap=None, quantizer="affine"):
        import torch
        from paper_2609_38121_b200 import binding as B
        self.torch, self.B, self.wl = torch, B, wl
        self.lengths = [int(x) for x in lengths]
        self.batch = len(self.lengths)
        self.bits, self.s_sink, self.s_keep, self.s_flush, self.lag = bits, s_sink, s_keep, s_flush, lag
        self.kappa_k, self.kappa_v = kappa_k, kappa_v
        self.T, self.TinvT, self.TV = oracle_transforms(wl)
        self.max_seq_len = max_seq_len or max(self.lengths + [64])
        max_pages = (self.max_seq_len + 63) // 64
        order = None
        if page_shuffle_seed is not None:
            order = np.random.default_rng(page_shuffle_seed).permutation(self.batch * max_pages)
        self.cache = B.PagedCache(wl.n_q, wl.n_kv, bits, self.batch, self.max_seq_len, s_sink, s_keep, s_flush,
                                  kappa_k, kappa_v, self.T, self.TinvT, boundary_lag=lag, page_order=order,
                                  ring_cap=ring_cap, quantizer=1 if quantizer == "quest" else 0)
        dev = self.cache.device
        self.slot = torch.arange(self.batch, dtype=torch.int32, device=dev)
        self.seq_len = torch.zeros(self.batch, dtype=torch.int32, device=dev)
        self.oracle = [O.LayerCache(wl.n_kv, 128, bits, kappa_k, kappa_v, self.T, quantizer=quantizer) for _ in range(self.batch)]
        self.tokens = []
        for b, n in enumerate(self.lengths):
            ks, vs = [], []
            for _, K, V in wl.sequence_tokens(b, n, T_V=self.TV):
                ks.append(K)
                vs.append(V)
            self.tokens.append((np.concatenate(ks) if ks else np.zeros((0, wl.n_kv, 128), np.float32),
                                np.concatenate(vs) if vs else np.zeros((0, wl.n_kv, 128), np.float32)))
        self.done = [0] * self.batch
        self.prologue = None          # a binding.Prologue: appends then go through wushkv_append_projected

    def append_step(self, counts, oracle_too=True):
        """Append counts[b] new tokens to sequence b on the GPU (one library call) and in the oracle."""
        torch, B = self.torch, self.B
        counts = [int(c) for c in counts]
        Ks, Vs = [], []
        for b, c in enumerate(counts):
            K, V = self.tokens[b]
            Ks.append(K[self.done[b]:self.done[b] + c])
            Vs.append(V[self.done[b]:self.done[b] + c])
            if oracle_too and c:
                self.oracle[b].append(Ks[-1], Vs[-1])
            self.done[b] += c
        total = sum(counts)
        cu = torch.tensor(np.concatenate([[0], np.cumsum(counts)]).astype(np.int32), device=self.cache.device)
        if total:
            Kn = torch.from_numpy(W.f32_to_bf16_bits(np.concatenate(Ks)).view(np.int16)).to(self.cache.device)
            Vn = torch.from_numpy(W.f32_to_bf16_bits(np.concatenate(Vs)).view(np.int16)).to(self.cache.device)
        else:
            Kn = Vn = torch.zeros(8, dtype=torch.int16, device=self.cache.device)
        if self.prologue is not None:
            B.append_projected(self.cache.desc, self.batch, self.slot, self.seq_len, cu, total, max(counts), Kn, Vn,
                               self.prologue.desc)
        else:
            B.append(self.cache.desc, self.batch, self.slot, self.seq_len, cu, total, max(counts), Kn, Vn)
        torch.cuda.synchronize()

    def fill(self, last_step=1):
        """Prefill all but ``last_step`` tokens of every sequence in one call, then the rest in another."""
        first = [max(n - last_step, 0) for n in self.lengths]
        self.append_step(first)
        self.append_step([n - f for n, f in zip(self.lengths, first)])

    # ---- read-back -------------------------------------------------------------------------------
    def gpu_codes(self, b, h, which, n=None):
        torch, B = self.torch, self.B
        n = self.lengths[b] if n is None else n
        codes = torch.empty((max(n, 1), 128), dtype=torch.uint8, device=self.cache.device)
        scale = torch.empty(max(n, 1), dtype=torch.float32, device=self.cache.device)
        zero = torch.empty(max(n, 1), dtype=torch.float32, device=self.cache.device)
        B.unpack_debug(self.cache.desc, b, h, which, 0, n, codes, scale, zero)
        torch.cuda.synchronize()
        return codes.cpu().numpy()[:n], scale.cpu().numpy()[:n].astype(np.float64), zero.cpu().numpy()[:n].astype(np.float64)

    def check_append_parity(self):
        """Codes, scales and zeros of every position against the oracle.  Returns the fraction of all
        codes of the layer that differ (each by exactly one level, else this asserts)."""
        n_codes = n_diff = 0
        for b in range(self.batch):
            n = self.lengths[b]
            if n == 0:
                continue
            kc, km, vc, vm, kb, vb = self.oracle[b].arrays()
            for h in range(self.wl.n_kv):
                for which, (oc, om) in enumerate(((kc, km), (vc, vm))):
                    gc, gs, gz = self.gpu_codes(b, h, which)
                    diff = np.abs(gc.astype(np.int32) - oc[:, h].astype(np.int32))
                    assert diff.max() <= 1, f"code off by more than one level (b={b} h={h} which={which})"
                    n_codes += diff.size
                    n_diff += int(np.count_nonzero(diff))
                    sref, zref = om[:, h, 0], om[:, h, 1]
                    assert np.all(np.abs(gs - sref) <= META_RTOL * np.abs(sref) + 1e-12), "scale mismatch"
                    # the offset is compared relative to the vector's range (x_min can sit near zero)
                    span = ((1 << self.bits) - 1) * sref
                    assert np.all(np.abs(gz - zref) <= META_RTOL * np.maximum(np.abs(zref), span) + 1e-12), "zero mismatch"
        self.last_code_stats = (n_diff, n_codes)
        return n_diff / max(n_codes, 1)

    def gpu_window_arrays(self, b):
        """bf16 copies the GPU holds for sequence b, scattered to their positions ([S][n_kv][128]
        each, NaN where the GPU keeps no copy)."""
        S = self.lengths[b]
        c = self.cache
        kb = np.full((S, self.wl.n_kv, 128), np.nan)
        vb = np.full((S, self.wl.n_kv, 128), np.nan)
        sink = c.sink_kv[b].float().cpu().numpy().astype(np.float64)       # [n_kv][2][s_sink][d]
        ring = c.ring_kv[b].float().cpu().numpy().astype(np.float64)       # [n_kv][2][ring_cap][d]
        for p in range(min(S, self.s_sink)):
            kb[p] = sink[:, 0, p]
            vb[p] = sink[:, 1, p]
        for p in range(max(0, S - c.ring_cap), S):
            if p >= self.s_sink:
                kb[p] = ring[:, 0, p % c.ring_cap]
                vb[p] = ring[:, 1, p % c.ring_cap]
        return kb, vb

    def decode(self, queries=None, projected=False):
        """One decode step on the GPU; returns (O_gpu [batch][n_q][128], Q float32 used).  ``projected``: the
        queries are projected ones and go through wushkv_decode_attn_projected with this layer's prologue."""
        torch, B = self.torch, self.B
        if queries is None:
            queries = np.stack([self.wl.queries(b, max(self.lengths[b] - 1, 0)) for b in range(self.batch)])
        Q = torch.from_numpy(W.f32_to_bf16_bits(queries).view(np.int16)).to(self.cache.device)
        Oo = torch.full((self.batch, self.wl.n_q, 128), float("nan"), dtype=torch.float32, device=self.cache.device)
        nbytes = B.decode_workspace_bytes(self.cache.desc, self.batch, self.max_seq_len)
        assert nbytes > 0
        ws = torch.empty(nbytes, dtype=torch.uint8, device=self.cache.device)
        if projected:
            B.decode_attn_projected(self.cache.desc, self.batch, self.slot, self.seq_len, self.max_seq_len, Q,
                                    self.prologue.desc, Oo, ws, nbytes)
        else:
            B.decode_attn(self.cache.desc, self.batch, self.slot, self.seq_len, self.max_seq_len, Q, Oo, ws, nbytes)
        torch.cuda.synchronize()
        return Oo.cpu().numpy().astype(np.float64), queries

    def oracle_decode_on_gpu_cache(self, b, q, heads=None):
        """Oracle decode of sequence b fed with the codes / meta / bf16 windows the GPU stored."""
        S = self.lengths[b]
        n_kv = self.wl.n_kv
        kc = np.zeros((S, n_kv, 128), np.uint8)
        vc = np.zeros((S, n_kv, 128), np.uint8)
        km = np.zeros((S, n_kv, 2))
        vm = np.zeros((S, n_kv, 2))
        for h in range(n_kv):
            c, s, z = self.gpu_codes(b, h, 0)
            kc[:, h], km[:, h, 0], km[:, h, 1] = c, s, z
            c, s, z = self.gpu_codes(b, h, 1)
            vc[:, h], vm[:, h, 0], vm[:, h, 1] = c, s, z
        kb, vb = self.gpu_window_arrays(b)
        out = O.decode_attn(q, self.TinvT, kc, km, vc, vm, kb, vb, S, self.s_sink, self.s_keep, self.s_flush,
                            1.0 / np.sqrt(128), lag=self.lag)
        assert np.all(np.isfinite(out)), "oracle read a position the GPU keeps no bf16 copy of"
        return out

    def prefill(self, counts, queries=None, repeat=0):
        """Append counts[b] new tokens per sequence and compute their attention outputs with wushkv_prefill_attn (with
        wushkv_prefill_attn_projected if this layer has a prologue; ``queries`` then holds the projected queries).
        Returns (O_gpu list per sequence [n][n_q][128], queries list per sequence).  ``repeat`` > 0: the attention call is
        made that many more times on the same cache state into fresh buffers, and ``self.repeats`` holds those outputs
        (whole arrays [total][n_q][128], float32) beside the first call's ``self.first``."""
        torch, B = self.torch, self.B
        counts = [int(c) for c in counts]
        start = list(self.done)
        Ks = [self.tokens[b][0][start[b]:start[b] + c] for b, c in enumerate(counts)]
        Vs = [self.tokens[b][1][start[b]:start[b] + c] for b, c in enumerate(counts)]
        self.append_step(counts)
        total = sum(counts)
        dev = self.cache.device
        qs = queries if queries is not None else [
            self.wl.chunk_queries(b, np.arange(start[b], start[b] + c)) if c else np.zeros((0, self.wl.n_q, 128), np.float32)
            for b, c in enumerate(counts)]
        bits16 = lambda x: torch.from_numpy(W.f32_to_bf16_bits(x).view(np.int16)).to(dev)  # noqa: E731
        Kn, Vn, Qn = bits16(np.concatenate(Ks)), bits16(np.concatenate(Vs)), bits16(np.concatenate(qs))
        cu = torch.tensor(np.concatenate([[0], np.cumsum(counts)]).astype(np.int32), device=dev)
        Oo = torch.full((total, self.wl.n_q, 128), float("nan"), dtype=torch.float32, device=dev)
        nbytes = B.prefill_workspace_bytes(self.cache.desc, self.batch, total)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        if self.prologue is not None:
            B.prefill_attn_projected(self.cache.desc, self.batch, self.slot, self.seq_len, cu, total, max(counts), Kn, Vn, Qn,
                                     self.prologue.desc, Oo, ws, nbytes)
        else:
            B.prefill_attn(self.cache.desc, self.batch, self.slot, self.seq_len, cu, total, max(counts), Kn, Vn, Qn, Oo, ws, nbytes)
        torch.cuda.synchronize()
        self.first, self.repeats = Oo.cpu().numpy(), []
        for _ in range(repeat):
            O2 = torch.full((total, self.wl.n_q, 128), float("nan"), dtype=torch.float32, device=dev)
            ws2 = torch.empty(nbytes, dtype=torch.uint8, device=dev)
            if self.prologue is not None:
                B.prefill_attn_projected(self.cache.desc, self.batch, self.slot, self.seq_len, cu, total, max(counts), Kn, Vn, Qn,
                                         self.prologue.desc, O2, ws2, nbytes)
            else:
                B.prefill_attn(self.cache.desc, self.batch, self.slot, self.seq_len, cu, total, max(counts), Kn, Vn, Qn, O2, ws2, nbytes)
            torch.cuda.synchronize()
            self.repeats.append(O2.cpu().numpy())
        out = self.first.astype(np.float64)
        offs = np.concatenate([[0], np.cumsum(counts)])
        return [out[offs[b]:offs[b + 1]] for b in range(self.batch)], qs

    def check_prefill_parity(self, counts, tol=DECODE_TOL, rows=None):
        """Chunk attention of the GPU against the oracle's on the cache content the GPU stored (codes and meta of
        the old positions; the bf16 roundings of the transformed keys for the window and chunk positions come from
        the oracle's own cache, which the append parity check ties to the GPU's).  ``rows``: chunk rows to check
        per sequence (default: all)."""
        outs, qs = self.prefill(counts)
        worst = 0.0
        for b, c in enumerate(counts):
            if c == 0:
                continue
            S = self.done[b]
            n_kv = self.wl.n_kv
            kc = np.zeros((S, n_kv, 128), np.uint8)
            vc = np.zeros((S, n_kv, 128), np.uint8)
            km = np.zeros((S, n_kv, 2))
            vm = np.zeros((S, n_kv, 2))
            for h in range(n_kv):
                cc, sc, zc = self.gpu_codes(b, h, 0, n=S)
                kc[:, h], km[:, h, 0], km[:, h, 1] = cc, sc, zc
                cc, sc, zc = self.gpu_codes(b, h, 1, n=S)
                vc[:, h], vm[:, h, 0], vm[:, h, 1] = cc, sc, zc
            _, _, _, _, kb, vb = self.oracle[b].arrays()
            sel = np.arange(c) if rows is None else np.asarray([r for r in rows if r < c])
            ref = O.chunk_attn(qs[b], self.TinvT, kc, km, vc, vm, kb, vb, S, c, self.s_sink, self.s_keep, self.s_flush,
                               1.0 / np.sqrt(128), lag=self.lag, rows=None if rows is None else [int(r) for r in sel])
            assert np.all(np.isfinite(outs[b])), "non-finite prefill output"
            for r in sel:
                err = np.max(np.abs(outs[b][r] - ref[r])) / np.max(np.abs(ref[r]))
                worst = max(worst, err)
                assert err <= tol, f"prefill mismatch: sequence {b}, chunk row {r}: {err:.3e} of max-abs"
        return worst

    def check_decode_parity(self, tol=DECODE_TOL):
        Og, Q = self.decode()
        worst = 0.0
        for b in range(self.batch):
            if self.lengths[b] == 0:
                assert np.all(Og[b] == 0)
                continue
            ref = self.oracle_decode_on_gpu_cache(b, Q[b])
            err = np.max(np.abs(Og[b] - ref)) / np.max(np.abs(ref))
            worst = max(worst, err)
            assert err <= tol, f"decode mismatch for sequence {b}: {err:.3e} of max-abs"
        return worst
