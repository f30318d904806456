"""Device-side failure paths: every wait in the kernels is bounded, and what goes wrong is reported in
*dev_status instead of trapping.  The failures are made without faulting anything: a copy (or an MMA
commit) that the kernel is told not to issue, with a short wait limit, so that the bounded wait runs out
and the kernel returns; a token count that contradicts the host's hint; a value range beyond what the
decode kernel's fp16 operand can carry."""
import numpy as np
import pytest

from paper_2609_38121_b200 import workloads as W
from tests.harness import Layer

pytestmark = pytest.mark.gpu


def _wl(n_q, n_kv, seed, batch=1):
    return W.LayerWorkload(dict(seed=seed, batch=batch, n_q=n_q, n_kv=n_kv, ctx=0, theta=1e4, bits=2, s_sink=4,
                                s_keep=64, rmsnorm=False, ragged=None, prefill_chunk=0))


def test_copy_that_never_arrives_is_flagged_and_the_next_call_is_healthy(test_option):
    from paper_2609_38121_b200 import binding as B
    wl = _wl(8, 2, seed=61, batch=2)
    L = Layer(wl, [1500, 1500], 2, 4, 64, 1)
    L.fill()
    good, _ = L.decode()
    assert L.cache.status() == 0
    test_option("drop_copy_unit", 0)          # first work unit: sequence 0, KV head 0, first packed page
    test_option("wait_limit", 64)
    out, _ = L.decode()                       # returns: the warp that waits for the page gives up
    assert L.cache.status() & B.DEV_COPY_TIMEOUT
    assert np.array_equal(out[1], good[1])    # the other sequence never depended on that warp
    test_option("drop_copy_unit", -1)
    test_option("wait_limit", 0)
    L.cache.dev_status.zero_()
    again, _ = L.decode()
    assert L.cache.status() == 0
    assert np.array_equal(again, good)


def test_chunk_mma_that_is_never_committed_is_flagged(test_option):
    from paper_2609_38121_b200 import binding as B
    wl = _wl(8, 2, seed=62)
    test_option("drop_chunk_mma", 1)
    test_option("wait_limit", 64)
    bad = Layer(wl, [300], 2, 4, 64, 1)
    bad.append_step([300], oracle_too=False)  # tensor-core path (chunk >= 128 tokens); its first tile never reports
    assert bad.cache.status() & B.DEV_COPY_TIMEOUT
    test_option("drop_chunk_mma", 0)
    test_option("wait_limit", 0)
    ok = Layer(wl, [300], 2, 4, 64, 1)
    ok.fill()
    assert ok.cache.status() == 0
    assert ok.check_append_parity() <= 1e-4
    assert ok.check_decode_parity() <= 2e-3


def test_chunk_transform_wait_that_runs_out_is_flagged(test_option):
    """The tcgen05 transform kernel of the chunk attention with a bulk tensor copy that is announced but never issued: its
    roles give up within the limit, the status bit is set, tensor memory is freed; the next call is healthy."""
    from paper_2609_38121_b200 import binding as B
    wl = _wl(8, 2, seed=67)
    L = Layer(wl, [300], 2, 4, 64, 1)
    test_option("drop_prefill", 3)
    test_option("wait_limit", 2000)
    L.prefill([300])
    assert L.cache.status() & B.DEV_COPY_TIMEOUT
    test_option("drop_prefill", 0)
    test_option("wait_limit", 0)
    ok = Layer(wl, [300], 2, 4, 64, 1)
    assert ok.check_prefill_parity([300]) <= 2e-3
    assert ok.cache.status() == 0


@pytest.mark.parametrize("one_tile", [0, 1])
@pytest.mark.parametrize("what", [1, 2])
def test_chunk_attention_wait_that_runs_out_is_flagged(what, one_tile, test_option):
    """The tcgen05 chunk attention with score MMAs that are never committed (1) or a bulk tensor copy that is announced
    but never issued (2): the bounded wait runs out, the kernel flags it, frees its tensor memory and returns; the next
    call is healthy."""
    from paper_2609_38121_b200 import binding as B
    wl = _wl(8, 2, seed=66)
    L = Layer(wl, [300], 2, 4, 64, 1)
    test_option("prefill_one_tile", one_tile)
    test_option("drop_prefill", what)
    test_option("wait_limit", 2000)
    outs, _ = L.prefill([300])
    assert L.cache.status() & B.DEV_COPY_TIMEOUT
    test_option("drop_prefill", 0)
    test_option("wait_limit", 0)
    ok = Layer(wl, [300], 2, 4, 64, 1)
    assert ok.check_prefill_parity([300]) <= 2e-3
    assert ok.cache.status() == 0


def test_more_tokens_than_the_decode_hint_promised():
    """max_new == 1 selects the single-token kernel; a sequence that brings two tokens is flagged and left alone."""
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = _wl(4, 1, seed=63, batch=2)
    L = Layer(wl, [100, 100], 2, 4, 64, 1)
    L.append_step([90, 90], oracle_too=False)
    cu = torch.tensor([0, 2, 3], dtype=torch.int32, device="cuda")
    tok = torch.zeros((3, 1, 128), dtype=torch.int16, device="cuda")
    B.append(L.cache.desc, 2, L.slot, L.seq_len, cu, 3, 1, tok, tok)
    torch.cuda.synchronize()
    assert L.cache.status() & B.DEV_BAD_COUNT
    assert L.seq_len.cpu().tolist() == [90, 91]


def test_value_step_beyond_the_fp16_operand_range_is_flagged():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = _wl(4, 1, seed=64)
    L = Layer(wl, [200], 2, 4, 64, 1)
    L.fill()
    assert L.cache.status() == 0              # ordinary values: no flag
    K = torch.zeros((1, 1, 128), dtype=torch.int16, device="cuda")
    v = np.zeros((1, 1, 128), np.float32)
    v[0, 0, ::2] = 8192.0                     # range 8192: step 2731 at 2 bits
    V = torch.from_numpy(W.f32_to_bf16_bits(v).view(np.int16)).cuda()
    cu = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    B.append(L.cache.desc, 1, L.slot, L.seq_len, cu, 1, 1, K, V)
    torch.cuda.synchronize()
    assert L.cache.status() & B.DEV_VALUE_RANGE
