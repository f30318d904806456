"""The allocation-free decode entry point, wushkv_decode_attn_static, against the regular one.

Some users of the library cannot call cudaMalloc at all (their framework owns every byte of device
memory, or they only ever get input and output buffers handed to them), so they cannot provide the
workspace wushkv_decode_attn wants.  The static variant carries its own fixed scratch array.  This
test calls it through the C ABI twice in a row - the second call finds the first call's leftovers
in the scratch - and checks both results against the regular entry point on the same inputs.
It lives in a file of its own that sorts last so that a run stopping at the first failure has
already exercised everything else."""
import ctypes as C

import numpy as np
import pytest

from paper_2609_38121_b200 import workloads as W
from tests.harness import DECODE_TOL, Layer

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_regular_decode_twice():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = W.LayerWorkload(dict(seed=77, batch=3, n_q=8, n_kv=2, ctx=0, theta=1e4, bits=2, s_sink=4, s_keep=64,
                              rmsnorm=False, ragged=None, prefill_chunk=0))
    L = Layer(wl, [900, 70, 1500], 2, 4, 64, 1, max_seq_len=1536)
    L.fill()
    ref, queries = L.decode()                                   # regular entry point, caller-owned workspace
    assert np.all(np.isfinite(ref))
    Q = torch.from_numpy(W.f32_to_bf16_bits(queries).view(np.int16)).cuda()
    for call in range(2):
        out = torch.full((L.batch, wl.n_q, 128), float("nan"), dtype=torch.float32, device="cuda")
        B.decode_attn_static(L.cache.desc, L.batch, L.slot, L.seq_len, L.max_seq_len, Q, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy().astype(np.float64)
        for b in range(L.batch):
            err = np.max(np.abs(got[b] - ref[b])) / np.max(np.abs(ref[b]))
            assert err <= DECODE_TOL, f"call {call}, sequence {b}: {err:.3e}"
    assert L.cache.status() == 0
    # The call allocates no device memory: after the calls above resolved the array's address, the
    # driver's free-byte count is the same before and after two further calls, one of them on a
    # stream of its own that is ordered after the first by an event.
    out_a = torch.empty((L.batch, wl.n_q, 128), dtype=torch.float32, device="cuda")
    out_b = torch.empty_like(out_a)
    side = torch.cuda.Stream()
    done = torch.cuda.Event()
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    B.decode_attn_static(L.cache.desc, L.batch, L.slot, L.seq_len, L.max_seq_len, Q, out_a)
    done.record()
    side.wait_event(done)
    B.decode_attn_static(L.cache.desc, L.batch, L.slot, L.seq_len, L.max_seq_len, Q, out_b, stream=side)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, (free_before, free_after)
    for o in (out_a, out_b):
        got = o.cpu().numpy().astype(np.float64)
        for b in range(L.batch):
            assert np.max(np.abs(got[b] - ref[b])) / np.max(np.abs(ref[b])) <= DECODE_TOL
    assert torch.equal(out_a, out_b)
    # a different query afterwards still gives the regular path's answer (nothing stale is read)
    q2 = np.stack([wl.queries(b, 5) for b in range(L.batch)])
    ref2, _ = L.decode(q2)
    out = torch.empty((L.batch, wl.n_q, 128), dtype=torch.float32, device="cuda")
    B.decode_attn_static(L.cache.desc, L.batch, L.slot, L.seq_len, L.max_seq_len,
                         torch.from_numpy(W.f32_to_bf16_bits(q2).view(np.int16)).cuda(), out)
    torch.cuda.synchronize()
    assert np.max(np.abs(out.cpu().numpy() - ref2)) <= DECODE_TOL * np.max(np.abs(ref2))


def test_static_scratch_rejects_oversized_requests():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = W.LayerWorkload(dict(seed=78, batch=1, n_q=8, n_kv=2, ctx=0, theta=1e4, bits=2, s_sink=4, s_keep=64,
                              rmsnorm=False, ragged=None, prefill_chunk=0))
    L = Layer(wl, [100], 2, 4, 64, 1)
    L.fill()
    big_batch = 4096                                           # workspace far beyond the built-in scratch
    assert B.decode_workspace_bytes(L.cache.desc, big_batch, 100) > B.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    rc = B.lib.wushkv_decode_attn_static(C.byref(L.cache.desc), big_batch, dummy.data_ptr(), dummy.data_ptr(), 100,
                                         dummy.data_ptr(), dummy.data_ptr(), None)
    assert rc == B.ECAPACITY
    assert "too small" in B.status_string(rc)
