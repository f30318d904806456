#!/usr/bin/env python
"""Benchmark of the WUSH-KV hot path on B200: one "step" = quantize-on-append of the step's new
tokens + decode attention over the packed cache, for one layer, on seeded synthetic inputs shaped
like the named model layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg1] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is the metric of the benchmark definition: bytes of packed
cache (codes + scale/zero + bf16 windows) that one decode step must read, divided by the time of the
whole step (append + decode), with every input already resident in HBM.  `roofline` times the decode
main kernel alone (CUDA events recorded around it by the library on the launching stream).  `e2e`
repeats the steps through the host-buffer entry point (the step's new token and queries come from pinned
host memory, the outputs go back to it, one synchronisation per step; the library reads and writes
pinned buffers in place over the bus and falls back to staged copies otherwise).  `sustained` repeats the
device-resident steps back to back for at least a second with the SM clock sampled throughout (the short
regions run at the burst clock of a cool GPU); `value_sustained` is `value` over that leg.  For the prefill
config (cfg4) `roofline` describes the chunk attention (the dominant kernel there, against the tensor peak) and
`roofline_append` the chunk append kernel (against the HBM peak).  `cpu_baseline` times
the float64 oracle on a bounded slice, append and decode separately, with one thread and with all cores.
With N > 1 every rank runs its own replica of the workload (the path has no cross-GPU exchange).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_38121_b200 import workloads as W  # noqa: E402

METRIC = "2-bit decode-attn cache GB/s (fraction of HBM peak) @32k ctx; append tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 2 ** 20
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel at the named workload,
# from one ncu capture each (None where not captured).
NCU_TRAFFIC_BYTES = {"cfg1": 314262000, "cfg2": 365696000, "cfg3": 78262000,
                     "cfg4": 134600000 + 13600000}


def measured_tensor_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 1400.0, "fallback"


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------------
# workload on the GPU (product path only: library calls + torch for memory)
# ------------------------------------------------------------------------------------------------
def library_transforms(wl):
    """T_K, T_K_invT (and a value transform for the generator) from the calibration batch, built by
    the library's own host entry points."""
    from paper_2609_38121_b200 import binding as B
    Kc, Qc, Vraw = wl.calibration()
    d = 128
    M = np.zeros((wl.n_kv, d, d))
    H = np.zeros((wl.n_kv, d, d))
    B.accumulate_gram(W.f32_to_bf16_bits(Kc), W.f32_to_bf16_bits(Qc), M, H)
    T, TinvT = B.build_transforms(M, H, W.GAMMA)
    Mv = np.stack([Vraw[:, h].astype(np.float64).T @ Vraw[:, h].astype(np.float64) for h in range(wl.n_kv)])
    Hv = np.stack([2 * sum(wl.W_O[h, g].astype(np.float64) @ wl.W_O[h, g].astype(np.float64).T for g in range(wl.G))
                   for h in range(wl.n_kv)])
    TV, _ = B.build_transforms(Mv, Hv, W.GAMMA)
    return T, TinvT, TV


class Session:
    """A filled cache plus the per-step inputs of one config, resident on one GPU."""

    def __init__(self, name, n_steps, device="cuda", seed_offset=0, verbose=False, bits=None, cached=0, chunk=0):
        import torch
        from paper_2609_38121_b200 import binding as B
        self.torch, self.B = torch, B
        cfg = dict(W.CONFIGS[name])
        cfg["seed"] += 1000 * seed_offset
        if bits:
            cfg["bits"] = bits
        if chunk and cfg["prefill_chunk"]:
            cfg["prefill_chunk"] = cfg["ctx"] = int(chunk)
        self.name, self.cfg = name, cfg
        wl = self.wl = W.LayerWorkload(cfg)
        self.n_steps = n_steps
        self.chunk = cfg["prefill_chunk"]
        self.batch = wl.batch
        final = wl.lengths().astype(np.int64)
        # prefill config only: `cached` tokens per sequence already sit in the cache (quantized, apart from the
        # recent window) when the chunk arrives, so the chunk attention also reads packed pages
        self.cached = int(cached) if self.chunk else 0
        final = final + self.cached
        self.T, self.TinvT, self.TV = library_transforms(wl)
        self.s_flush = 1
        if self.chunk:
            self.start_len = np.full(self.batch, self.cached, np.int64)
            self.max_seq_len = int(final.max())
        else:
            self.start_len = final - 1
            self.max_seq_len = int(final.max()) + n_steps
        self.cache = B.PagedCache(wl.n_q, wl.n_kv, cfg["bits"], self.batch, self.max_seq_len, cfg["s_sink"],
                                  cfg["s_keep"], self.s_flush, W.KAPPA_K, W.KAPPA_V, self.T, self.TinvT, device=device)
        dev = self.cache.device
        self.slot = torch.arange(self.batch, dtype=torch.int32, device=dev)
        self.seq_len = torch.zeros(self.batch, dtype=torch.int32, device=dev)
        t0 = time.time()
        if self.chunk:
            ks, vs = [], []
            for b in range(self.batch):
                K, V = self.host_tokens(b)
                ks.append(K[self.cached:])
                vs.append(V[self.cached:])
            self.K_chunk = self._dev_bf16(np.concatenate(ks))
            self.V_chunk = self._dev_bf16(np.concatenate(vs))
            self.cu_chunk = torch.arange(0, (self.batch + 1) * self.chunk, self.chunk, dtype=torch.int32, device=dev)
            self.q_chunk_host = np.concatenate([wl.chunk_queries(b, self.cached + np.arange(self.chunk)) for b in range(self.batch)])
            self.Q_chunk = self._dev_bf16(self.q_chunk_host)
            self.O_chunk = torch.zeros((self.batch * self.chunk, wl.n_q, 128), dtype=torch.float32, device=dev)
            self.pf_bytes = B.prefill_workspace_bytes(self.cache.desc, self.batch, self.batch * self.chunk)
            self.pf_ws = torch.empty(self.pf_bytes, dtype=torch.uint8, device=dev)
            n_step_tok = 0
        else:
            n_step_tok = n_steps
        # prefill everything before the timed steps (one library call per sequence)
        step_k = np.zeros((max(n_step_tok, 1), self.batch, wl.n_kv, 128), np.float32)
        step_v = np.zeros_like(step_k)
        for b in range(self.batch):
            n_pre = int(self.start_len[b])
            ks, vs = [], []
            if self.cached:
                ks, vs = [[x] for x in self.host_tokens(b)]     # the stream whose tail is the chunk
            else:
                for _, K, V in wl.sequence_tokens(b, n_pre + n_step_tok, T_V=self.TV):
                    ks.append(K)
                    vs.append(V)
            K = np.concatenate(ks) if ks else np.zeros((0, wl.n_kv, 128), np.float32)
            V = np.concatenate(vs) if vs else np.zeros((0, wl.n_kv, 128), np.float32)
            if n_step_tok:
                step_k[:, b] = K[n_pre:]
                step_v[:, b] = V[n_pre:]
            if n_pre:
                counts = np.zeros(self.batch, np.int64)
                counts[b] = n_pre
                cu = torch.tensor(np.concatenate([[0], np.cumsum(counts)]).astype(np.int32), device=dev)
                B.append(self.cache.desc, self.batch, self.slot, self.seq_len, cu, n_pre, n_pre,
                         self._dev_bf16(K[:n_pre]), self._dev_bf16(V[:n_pre]))
                torch.cuda.synchronize()
        self.step_K = self._dev_bf16(step_k)
        self.step_V = self._dev_bf16(step_v)
        q = np.stack([wl.queries(b, int(final[b]) - 1) for b in range(self.batch)])
        self.Q = self._dev_bf16(q)
        self.q_host = q
        self.step_k_host, self.step_v_host = step_k, step_v
        self.cu_one = torch.arange(0, self.batch + 1, dtype=torch.int32, device=dev)
        self.O = torch.zeros((self.batch, wl.n_q, 128), dtype=torch.float32, device=dev)
        self.ws_bytes = B.decode_workspace_bytes(self.cache.desc, self.batch, self.max_seq_len)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.base_len = self.seq_len.clone()
        # rolling a sequence back to `cached` tokens also needs its recent window as it was then
        self.ring_base = self.cache.ring_kv.clone() if self.cached else None
        self.final = final
        self.step_index = 0
        if verbose:
            print(f"[bench] {name}: cache filled in {time.time() - t0:.1f}s, status {self.cache.status()}", file=sys.stderr)

    def host_tokens(self, b):
        """The (K, V) token rows of sequence b exactly as the constructor generated them (same stream,
        same chunking), positions 0 .. : used by tests to recompute sampled pieces with the oracle."""
        if self.chunk and not self.cached:
            _, K, V = next(self.wl.sequence_tokens(b, self.chunk, T_V=self.TV, chunk=self.chunk))
            return K, V
        if self.chunk:               # the cached tokens followed by the chunk's, one stream
            toks = list(self.wl.sequence_tokens(b, self.cached + self.chunk, T_V=self.TV))
            return np.concatenate([t[1] for t in toks]), np.concatenate([t[2] for t in toks])
        toks = list(self.wl.sequence_tokens(b, int(self.start_len[b]) + self.n_steps, T_V=self.TV))
        return np.concatenate([t[1] for t in toks]), np.concatenate([t[2] for t in toks])

    def _dev_bf16(self, x):
        return self.torch.from_numpy(W.f32_to_bf16_bits(x).view(np.int16)).to(self.cache.device)

    def rewind(self):
        self.seq_len.copy_(self.base_len)
        self.step_index = 0

    def step(self, mid_event=None, pf_event=None):
        """Enqueue one step (device-resident inputs).  Prefill config: append the chunk, compute the chunk's own
        attention outputs (Algorithm 2 line 5), then one decode step over the resulting cache."""
        B = self.B
        if not self.chunk and mid_event is None:        # the fused call a user makes for a decode step
            i = self.step_index
            B.decode_step(self.cache.desc, self.batch, self.slot, self.seq_len, self.cu_one, self.max_seq_len,
                          self.step_K[i], self.step_V[i], self.Q, self.O, self.ws, self.ws_bytes)
            self.step_index += 1
            return
        if self.chunk:
            self.seq_len.copy_(self.base_len)
            if self.ring_base is not None:
                self.cache.ring_kv.copy_(self.ring_base)
            B.append(self.cache.desc, self.batch, self.slot, self.seq_len, self.cu_chunk, self.batch * self.chunk,
                     self.chunk, self.K_chunk, self.V_chunk)
        else:
            i = self.step_index
            B.append(self.cache.desc, self.batch, self.slot, self.seq_len, self.cu_one, self.batch, 1,
                     self.step_K[i], self.step_V[i])
            self.step_index += 1
        if mid_event is not None:
            mid_event.record()
        if self.chunk:
            B.prefill_attn(self.cache.desc, self.batch, self.slot, self.seq_len, self.cu_chunk, self.batch * self.chunk,
                           self.chunk, self.K_chunk, self.V_chunk, self.Q_chunk, self.O_chunk, self.pf_ws, self.pf_bytes)
            if pf_event is not None:
                pf_event.record()
        B.decode_attn(self.cache.desc, self.batch, self.slot, self.seq_len, self.max_seq_len, self.Q, self.O,
                      self.ws, self.ws_bytes)

    # ---- algorithmic bytes of one step -----------------------------------------------------------
    def lengths_at(self, step_no):
        """Context lengths seen by the decode of the step_no-th step (1-based) since the prefill."""
        return self.final if self.chunk else self.final - 1 + step_no

    def decode_bytes(self, step_no=1):
        c = self.cfg
        per_q = 2 * 128 * c["bits"] // 8 + 8
        total = 0
        for S in self.lengths_at(step_no):
            S = int(S)
            room = S - c["s_keep"] - c["s_sink"]
            nq = (room // self.s_flush) * self.s_flush if room >= self.s_flush else 0
            total += self.wl.n_kv * (nq * per_q + (S - nq) * 512)
        return total

    def append_tokens(self):
        return self.batch * (self.chunk if self.chunk else 1)

    def prefill_flops(self):
        """Multiply-adds x 2 of the chunk attention (causal: row i sees the cached tokens and i + 1 keys of the
        chunk; both contractions)."""
        n = self.chunk
        return 4.0 * 128 * self.wl.n_q * self.batch * (n * self.cached + n * (n + 1) / 2)

    def launches_per_step(self):
        # chunk append: transform/quantize kernel + length update (+ prefill attention: preparation + attention);
        # token append: one kernel; decode: prep + main + combine
        n = (4 if self.chunk else 1) + 3
        if self.chunk:
            # few query-tile pairs (a short chunk): the attention runs several CTAs per pair and a merge kernel follows
            R = 128 // (self.wl.n_q // self.wl.n_kv)
            tiles = -(-self.chunk // R)
            pairs = self.batch * ((tiles + 1) // 2) * self.wl.n_kv
            min_ctas = -(-self.batch * self.chunk // (2 * R)) * self.wl.n_kv
            sms = self.torch.cuda.get_device_properties(self.cache.device).multi_processor_count
            if min(max(1, min(16, sms // max(min_ctas, 1))), max(1, sms // pairs)) > 1:
                n += 1
        return n


# ------------------------------------------------------------------------------------------------
# multi-GPU aggregation (replicas only: no data-path collective, just the slowest rank's time)
# ------------------------------------------------------------------------------------------------
def max_over_ranks(ms, device="cuda"):
    """Slowest rank's time per step (all ranks get it).  A no-op outside torch.distributed."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_rank_step, ms_per_step, world):
    """Whole-job GB/s: every rank moved `bytes_per_rank_step` per step, the job took the slowest rank's time."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
_CLOCK_POLL_SRC = r"""
import sys, time
import pynvml as N
N.nvmlInit()
key = sys.argv[1]
try:
    h = N.nvmlDeviceGetHandleByUUID(key) if key.startswith("GPU-") else N.nvmlDeviceGetHandleByIndex(int(key))
except Exception:
    h = N.nvmlDeviceGetHandleByIndex(0)
mx = N.nvmlDeviceGetMaxClockInfo(h, N.NVML_CLOCK_SM)
w = sys.stdout.write
while True:
    t = time.monotonic_ns()
    sm = N.nvmlDeviceGetClockInfo(h, N.NVML_CLOCK_SM)
    try:
        r = N.nvmlDeviceGetCurrentClocksEventReasons(h)
    except Exception:
        r = N.nvmlDeviceGetCurrentClocksThrottleReasons(h)
    w("%d,%d,%d,%d\n" % (t, sm, mx, r))
    sys.stdout.flush()
    time.sleep(0.0003)
"""


def device_key(local):
    """NVML name of CUDA device `local`: its UUID (CUDA_VISIBLE_DEVICES may renumber), else the index."""
    try:
        import torch
        return "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        return str(local)


class ClockSampler:
    """Reads (never sets) the SM clock and the clock-event reasons of one GPU through NVML from a
    child process, a few thousand times a second, so that a timed region of a few milliseconds
    still holds samples; `mark()` brackets the region on the system-wide monotonic clock."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, device_key):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.t0 = self.t1 = None
        try:
            self.proc = subprocess.Popen([sys.executable, "-c", _CLOCK_POLL_SRC, str(device_key)],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        deadline = time.time() + 10.0                       # wait for the first sample
        while self.proc is not None and time.time() < deadline and os.path.getsize(self.tmp.name) == 0:
            if self.proc.poll() is not None:
                self.proc = None
                break
            time.sleep(0.01)

    def mark(self):
        if self.t0 is None:
            self.t0 = time.monotonic_ns()
        else:
            self.t1 = time.monotonic_ns()

    def stop(self, bins=False):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        rows = []
        for line in self.tmp.read().splitlines():
            f = line.split(",")
            if len(f) == 4:
                try:
                    rows.append(tuple(int(x) for x in f))
                except ValueError:
                    pass
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        t0, t1 = self.t0 or 0, self.t1 or (1 << 62)
        inside = [r for r in rows if t0 <= r[0] <= t1]
        if not inside and rows:                              # region shorter than the sampling period
            mid = (t0 + t1) // 2
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:2]
            out["nearest"] = True
        if inside:
            bits = 0
            for r in inside:
                bits |= r[3]
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                       reasons=sorted(n for b, n in self.REASONS.items() if bits & b), samples=len(inside))
            if bins:                                         # share of the samples at each SM clock
                hist = {}
                for r in inside:
                    hist[r[1]] = hist.get(r[1], 0) + 1
                out["sm_mhz_bins"] = {str(k): round(v / len(inside), 4) for k, v in sorted(hist.items())}
        return out


# ------------------------------------------------------------------------------------------------
# CPU oracle arm
# ------------------------------------------------------------------------------------------------
class OracleSample:
    """The float64 oracle on a bounded slice of the workload: ONE sequence and ONE KV head (with its
    G query heads) at the config's full context.  A step appends one token and decodes."""

    def __init__(self, name, ctx_cap=None):
        from oracle import wushkv_oracle as O
        self.O = O
        cfg = dict(W.CONFIGS[name])
        wl = self.wl = W.LayerWorkload(cfg)
        self.cfg = cfg
        G = wl.G
        Kc, Qc, _ = wl.calibration()
        M, H = O.gram_hessian(Kc[:, 0], np.stack([Qc[:, g] for g in range(G)]))
        self.T, self.TinvT = O.build_transforms(M[None], H[None], W.GAMMA)
        S = int(wl.lengths()[0])
        if ctx_cap:
            S = min(S, ctx_cap)
        self.S = S
        self.cache = O.LayerCache(1, 128, cfg["bits"], W.KAPPA_K, W.KAPPA_V, self.T)
        toks = [(K[:, :1], V[:, :1]) for _, K, V in wl.sequence_tokens(0, S + 64)]
        self.K = np.concatenate([t[0] for t in toks])
        self.V = np.concatenate([t[1] for t in toks])
        self.cache.append(self.K[:S - 1], self.V[:S - 1])
        self.q = wl.queries(0, S - 1)[:G]
        self.extra = 0

    def append_one(self):
        i = self.S - 1 + self.extra
        self.cache.append(self.K[i:i + 1], self.V[i:i + 1])
        self.extra += 1

    def decode(self):
        O, c = self.O, self.cfg
        arrs = self.cache.arrays()
        return O.decode_attn(self.q, self.TinvT, *arrs, self.cache.S, c["s_sink"], c["s_keep"], 1, 1.0 / np.sqrt(128))

    def step(self):
        self.append_one()
        return self.decode()

    def bytes_per_step(self):
        c = self.cfg
        per_q = 2 * 128 * c["bits"] // 8 + 8
        S = self.S
        nq = max(S - c["s_keep"] - c["s_sink"], 0)
        return nq * per_q + (S - nq) * 512


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle(name, steps, warmup, budget_s=20.0):
    smp = OracleSample(name)
    for _ in range(warmup):
        smp.step()
    times = []
    t_all = time.perf_counter()
    for _ in range(steps):
        t0 = time.perf_counter()
        smp.step()
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_all > budget_s:
            break
    sec = sum(times) / len(times)
    return smp, sec, len(times)


def time_oracle_split(name, budget_s=16.0):
    """Append (one token) and decode of the oracle sample timed separately, with the numerical libraries
    limited to one thread and with all cores.  Returns (sample, {"append_ms": {...}, "decode_ms": {...}})."""
    smp = OracleSample(name)
    smp.step()                                           # warm-up of both halves
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        threadpool_limits = None
    out = {"append_ms": {}, "decode_ms": {}, "steps": {}}
    legs = [("1", 1), ("all", None)] if threadpool_limits else [("all", None)]
    for label, limit in legs:
        ctx = threadpool_limits(limits=limit) if (threadpool_limits and limit) else None
        if ctx:
            ctx.__enter__()
        try:
            ta, td, n = 0.0, 0.0, 0
            t_all = time.perf_counter()
            while n < 3 or (time.perf_counter() - t_all) < budget_s / len(legs):
                t0 = time.perf_counter()
                smp.append_one()
                t1 = time.perf_counter()
                smp.decode()
                t2 = time.perf_counter()
                ta += t1 - t0
                td += t2 - t1
                n += 1
                if n >= 10 ** 6:
                    break
            out["append_ms"][label] = ta / n * 1e3
            out["decode_ms"][label] = td / n * 1e3
            out["steps"][label] = n
        finally:
            if ctx:
                ctx.__exit__(None, None, None)
    return smp, out


# ------------------------------------------------------------------------------------------------
def run_reference(args, rank):
    if rank != 0:
        return
    smp, sec, done = time_oracle(args.config, args.steps, args.warmup, budget_s=120.0)
    gbs = smp.bytes_per_step() / sec / 1e9
    sample = (f"1 of {smp.wl.batch} sequences x 1 of {smp.wl.n_kv} KV heads ({smp.wl.G} query heads) at context {smp.S}: "
              f"append 1 token + decode, numpy float64")
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": done,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.config, "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args, rank, world):
    import torch
    import torch.distributed as dist
    from paper_2609_38121_b200 import build as _build
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    from paper_2609_38121_b200 import binding as B

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    K, Wm = args.steps, args.warmup
    n_total_steps = Wm + K            # device-timed region
    if (args.cached_context or args.prefill_chunk) and not W.CONFIGS[args.config]["prefill_chunk"]:
        raise SystemExit("--cached-context and --prefill-chunk apply to a prefill config (cfg4)")
    sess = Session(args.config, n_steps=3 * n_total_steps + 2, seed_offset=rank, verbose=(rank == 0 and args.verbose), bits=args.bits,
                   cached=args.cached_context, chunk=args.prefill_chunk)
    cache_bytes = sess.decode_bytes(1)
    need_flush = cache_bytes < 2 * L2_BYTES
    flush_buf = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device="cuda") if need_flush else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(Wm):
        sess.step()
    torch.cuda.synchronize()
    assert sess.cache.status() == 0, f"device status {sess.cache.status()}"

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    starts, stops = [ev() for _ in range(K)], [ev() for _ in range(K)]
    sampler = ClockSampler(device_key(local)) if rank == 0 else None
    # ---- region A: K whole steps, device-timed; this gives `value`
    barrier()
    if sampler:
        sampler.mark()
    t_region0, t_region1 = ev(), ev()
    t_region0.record()
    for i in range(K):
        if need_flush:
            flush_buf.fill_(i & 0xFF)
            starts[i].record()
        sess.step()
        if need_flush:
            stops[i].record()
    t_region1.record()
    barrier()
    assert sess.cache.status() == 0, f"device status {sess.cache.status()}"
    if need_flush:
        ms_per_step = sum(s_.elapsed_time(e_) for s_, e_ in zip(starts, stops)) / K     # flush time excluded
    else:
        ms_per_step = t_region0.elapsed_time(t_region1) / K
    # ---- region B: K more steps with events around the append call and around the decode main kernel
    # (recorded by the library on the launching stream); this gives `roofline` and the append time.
    # Events between kernels switch programmatic dependent launch off, so region B's steps are a
    # little slower than region A's; the kernel's own duration is what is taken from here.
    mids = [ev() for _ in range(K)]
    pfs = [ev() for _ in range(K)]
    kstart, kstop = [ev() for _ in range(K)], [ev() for _ in range(K)]
    for e in kstart + kstop:
        e.record()                    # materialise the handles
    torch.cuda.synchronize()
    for i in range(K):
        if need_flush:
            flush_buf.fill_(i & 0xFF)
        B.set_profile_events(kstart[i], kstop[i])
        starts[i].record()
        sess.step(mid_event=mids[i], pf_event=pfs[i])
        stops[i].record()
    B.set_profile_events(None, None)
    barrier()
    if sampler:
        sampler.mark()
    clocks = sampler.stop() if sampler else None
    assert sess.cache.status() == 0, f"device status {sess.cache.status()}"
    step_ms = [s_.elapsed_time(e_) for s_, e_ in zip(starts, stops)]
    append_ms = [s_.elapsed_time(e_) for s_, e_ in zip(starts, mids)]
    prefill_ms = [s_.elapsed_time(e_) for s_, e_ in zip(mids, pfs)] if sess.chunk else None
    kern_ms = [s_.elapsed_time(e_) for s_, e_ in zip(kstart, kstop)]
    ms_per_step = max_over_ranks(ms_per_step)
    bytes_step = float(np.mean([sess.decode_bytes(Wm + i + 1) for i in range(K)])) if not sess.chunk else float(cache_bytes)
    value = whole_job_value(bytes_step, ms_per_step, world)

    # ---- region C (decode configs): at least a second of back-to-back steps, clocks sampled throughout and binned.
    # The few-millisecond regions above run at the burst clock of a cool GPU; this is what a serving loop holds.
    sustained = None
    if not sess.chunk and not args.no_sustained:
        sampler_c = ClockSampler(device_key(local)) if rank == 0 else None
        n_avail = sess.step_K.shape[0]
        done, reps = 0, 0
        barrier()
        if sampler_c:
            sampler_c.mark()
        c0, c1 = ev(), ev()
        c0.record()
        t_wall = time.perf_counter()
        while True:
            sess.rewind()
            for _ in range(n_avail):
                sess.step()
            done += n_avail
            reps += 1
            if reps % 8 == 0:
                torch.cuda.synchronize()
                if time.perf_counter() - t_wall >= args.sustained_seconds:
                    break
        c1.record()
        barrier()
        if sampler_c:
            sampler_c.mark()
        sus_ms = max_over_ranks(c0.elapsed_time(c1) / done)
        clk_c = sampler_c.stop(bins=True) if sampler_c else None
        sess.rewind()
        sess.step_index = 0
        bytes_sus = float(np.mean([sess.decode_bytes(i + 1) for i in range(n_avail)]))
        sustained = {"steps": done, "seconds": c0.elapsed_time(c1) * 1e-3, "ms_per_step": sus_ms,
                     "value": whole_job_value(bytes_sus, sus_ms, world), "clocks": clk_c}
        assert sess.cache.status() == 0

    # ---- end-to-end through the host-buffer entry point (decode steps only)
    e2e = None
    if not sess.chunk:
        stg_bytes = B.step_staging_bytes(sess.cache.desc, sess.batch)
        stg = torch.empty(stg_bytes, dtype=torch.uint8, device="cuda")
        hK = torch.from_numpy(W.f32_to_bf16_bits(sess.step_k_host).view(np.int16)).pin_memory()
        hV = torch.from_numpy(W.f32_to_bf16_bits(sess.step_v_host).view(np.int16)).pin_memory()
        hQ = torch.from_numpy(W.f32_to_bf16_bits(sess.q_host).view(np.int16)).pin_memory()
        hO = torch.empty((sess.batch, sess.wl.n_q, 128), dtype=torch.float32).pin_memory()
        base = sess.step_index
        assert base + Wm + K <= hK.shape[0]

        # views made once: the timed loop holds the library call, the synchronisation and the host's read of the result
        hK_rows = [hK[base + i] for i in range(Wm + K)]
        hV_rows = [hV[base + i] for i in range(Wm + K)]
        hO_np = hO.numpy()

        def host_step(i):
            B.decode_step_host(sess.cache.desc, sess.batch, sess.slot, sess.seq_len, sess.cu_one, sess.max_seq_len,
                               hK_rows[i], hV_rows[i], hQ, hO, stg, stg_bytes, sess.ws, sess.ws_bytes)
            torch.cuda.synchronize()
            return float(hO_np[0, 0, 0])              # the host reads the step's result

        for i in range(Wm):
            host_step(i)
        barrier()
        t0 = time.perf_counter()
        for i in range(K):
            host_step(Wm + i)
        t1 = time.perf_counter()
        e2e_ms = (t1 - t0) * 1e3 / K
        e2e_ms = max_over_ranks(e2e_ms)
        e2e = {"value": whole_job_value(bytes_step, e2e_ms, world), "unit": "GB/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(2 * hK[0].numel() * 2 + hQ.numel() * 2), "d2h_bytes_per_step": int(hO.numel() * 4)}
        assert sess.cache.status() == 0

    if rank != 0:
        return
    peak, peak_kind = measured_hbm_peak()
    sm_mhz = (clocks or {}).get("sm_mhz")
    if sess.chunk:
        # prefill config, the chunk append (tensor-core transform + quantize + pack): its algorithmic bytes are
        # the bf16 keys and values read plus the packed records written
        per_tok = 2 * 128 * 2 + 2 * 128 * sess.cfg["bits"] // 8 + 8
        app_bytes = float(sess.append_tokens() * sess.wl.n_kv * per_tok)
        app_s = statistics.mean(append_ms) * 1e-3
        achieved = app_bytes / app_s / 1e9
        roofline = {"bound": "hbm", "kernel": "append_chunk_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                    "kernel_ms": app_s * 1e3, "kernel_ms_min": min(append_ms), "algorithmic_bytes": app_bytes,
                    "traffic": NCU_TRAFFIC_BYTES.get(args.config),
                    "kernel_cycles": (app_s * 1e6 * sm_mhz) if sm_mhz else None,
                    "note": "timed from the step's start to the event after wushkv_append (chunk kernel + length update); "
                            "the kernel's busiest unit is the integer/logic pipe of the percentile selection, not HBM",
                    "decode_main_kernel_ms": statistics.mean(kern_ms)}
    else:
        kern_s = statistics.mean(kern_ms) * 1e-3
        achieved = bytes_step / kern_s / 1e9
        roofline = {"bound": "hbm", "kernel": "decode_main_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                    "kernel_ms": kern_s * 1e3, "kernel_ms_min": min(kern_ms), "algorithmic_bytes": bytes_step,
                    "traffic": None if args.bits else NCU_TRAFFIC_BYTES.get(args.config),
                    "kernel_cycles": (kern_s * 1e6 * sm_mhz) if sm_mhz else None}
    roofline_append = None
    if sess.chunk:
        # the dominant kernel of the prefill config is the chunk attention (tcgen05), bound by the tensor pipe
        roofline_append = roofline
        tf_peak, tf_kind = measured_tensor_peak()
        pf_s = statistics.mean(prefill_ms) * 1e-3
        tf = sess.prefill_flops() / pf_s / 1e12
        roofline = {"bound": "tensor", "kernel": "prefill_attn_ws_kernel (+ prefill_prep_tc_kernel)", "achieved": tf, "peak": tf_peak,
                    "unit": "TFLOP/s", "frac": tf / tf_peak, "peak_kind": f"of {tf_kind} (bf16 matmul, sustained; fp16 has the same nominal rate)",
                    "kernel_ms": pf_s * 1e3, "kernel_ms_min": min(prefill_ms), "algorithmic_flops": sess.prefill_flops(), "traffic": None}
    cpu = None
    if world == 1 and not args.no_cpu:
        smp, split = time_oracle_split(args.config, budget_s=args.cpu_seconds)
        dec_all = split["decode_ms"]["all"]
        cpu = {"value": smp.bytes_per_step() / (dec_all * 1e-3) / 1e9, "unit": "GB/s", "cores": cpu_threads(), "kind": "oracle",
               "decode_ms": split["decode_ms"], "append_ms": split["append_ms"], "steps": split["steps"],
               "append_tokens_per_s": {k: 1e3 / v for k, v in split["append_ms"].items()},
               "host_cores": os.cpu_count(),
               "sample": (f"1 of {smp.wl.batch} sequences x 1 of {smp.wl.n_kv} KV heads ({smp.wl.G} query heads) at context "
                          f"{smp.S}, numpy float64; value = decode bytes of the slice / decode time with all cores; "
                          f"append = one token (transform + both quantizers) of that head; keys '1' / 'all' = threads allowed "
                          f"to the numerical libraries")}
    c = sess.cfg
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.config + (f"@{args.bits}bit" if args.bits else "") + (f"+chunk{sess.chunk}" if args.prefill_chunk else "") + (f"+cached{sess.cached}" if sess.cached else ""), "batch": sess.batch, "n_q": c["n_q"], "n_kv": c["n_kv"], "head_dim": 128,
                   "context": int(sess.final.max()), "bits": c["bits"], "s_sink": c["s_sink"], "s_keep": c["s_keep"],
                   "s_flush": sess.s_flush, "page_tokens": 64, "prefill_chunk": sess.chunk, "cached_context": sess.cached,
                   "l2": ("flushed between steps (256 MB write)" if need_flush else "cache read per step exceeds L2 (no flush)"),
                   "replicas": world},
        "roofline": roofline, "roofline_append": roofline_append, "cpu_baseline": cpu, "e2e": e2e,
        "value_sustained": sustained["value"] if sustained else None, "sustained": sustained,
        "gpu_launches": K * sess.launches_per_step(), "clocks": clocks,
        "decode_tokens_per_s": world * sess.batch / (ms_per_step * 1e-3),
        "append_tokens_per_s": world * sess.append_tokens() / (statistics.mean(append_ms) * 1e-3),
        "append_ms": statistics.mean(append_ms), "step_ms_with_kernel_events": statistics.mean(step_ms),
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="cfg1", choices=sorted(W.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-sustained", action="store_true", help="skip the second-long back-to-back leg")
    ap.add_argument("--sustained-seconds", type=float, default=1.0)
    ap.add_argument("--bits", type=int, default=0, choices=[0, 2, 3, 4],
                    help="override the configuration's bit width (0: as the configuration says); the workload name then carries it")
    ap.add_argument("--cached-context", type=int, default=0,
                    help="prefill config: tokens per sequence already in the cache when the chunk arrives (default 0); "
                         "not the headline configuration: a second workload, the chunk attention over packed pages")
    ap.add_argument("--prefill-chunk", type=int, default=0,
                    help="prefill config: tokens per sequence in the chunk (default: the config's own)")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
        dist.init_process_group("nccl")
    try:
        run_ours(args, rank, world)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
