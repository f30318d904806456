"""GPU parity tests proper: the CUDA library, called through its C ABI, against the float64 oracle on
the same seeded inputs.  Sizes are what the oracle finishes in seconds while still spanning several
pages, several splits and ragged tails."""
import numpy as np
import pytest

from paper_2609_38121_b200 import workloads as W
from tests.harness import CODE_MISMATCH_MAX, Layer

pytestmark = pytest.mark.gpu


def _wl(n_q, n_kv, seed, batch=1, theta=1e4, rmsnorm=False):
    return W.LayerWorkload(dict(seed=seed, batch=batch, n_q=n_q, n_kv=n_kv, ctx=0, theta=theta, bits=2, s_sink=4,
                                s_keep=64, rmsnorm=rmsnorm, ragged=None, prefill_chunk=0))


def _check_window_copies(L):
    """bf16 sink / ring contents: keys are bf16(T k) (rare one-ulp flips from fp32 vs fp64 summation
    order are allowed), values are the input itself, bit for bit."""
    for b in range(L.batch):
        S = L.lengths[b]
        if S == 0:
            continue
        kc, km, vc, vm, kb_o, vb_o = L.oracle[b].arrays()
        kb, vb = L.gpu_window_arrays(b)
        have = np.isfinite(kb[:, 0, 0])
        assert have[:min(S, L.s_sink)].all() and have[max(0, S - L.cache.ring_cap):].all()
        assert np.array_equal(vb[have], vb_o[have])
        d = np.abs(kb[have] - kb_o[have])
        ulp = np.maximum(np.abs(kb_o[have]), 1e-30) * 2.0 ** -7
        # fp32 accumulation error scales with the vector, not with an entry that cancels to almost zero
        slack = 4e-6 * np.max(np.abs(kb_o[have]), axis=-1, keepdims=True)
        assert np.all(d <= ulp + slack), "bf16 key copy differs by more than one ulp"
        assert np.mean(d > 0) < 2e-3


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_config0_tiny_layer(bits):
    """Benchmark config 0: batch 1, 8 query / 2 KV heads, 2048 context, sink 4, recent 64."""
    wl = W.LayerWorkload("cfg0")
    L = Layer(wl, [2048], bits, 4, 64, 1)
    L.fill()
    assert L.seq_len.cpu().tolist() == [2048]
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    _check_window_copies(L)
    assert L.check_decode_parity() <= 2e-3
    assert L.cache.status() == 0


@pytest.mark.parametrize("n_q,n_kv,bits", [(8, 1, 2), (8, 1, 4), (7, 1, 2), (14, 2, 4), (2, 2, 2), (6, 2, 2), (5, 1, 4), (3, 1, 2),
                                            (8, 2, 3), (8, 1, 3), (3, 1, 3)])
def test_group_sizes(n_q, n_kv, bits):
    """Every query-group size 1..8 takes one of the two fragment modes; G = 7 with RMSNorm is the
    Qwen-shaped layer of config 4, G = 8 the 70B-shaped layer of config 3."""
    wl = _wl(n_q, n_kv, seed=10 + n_q, theta=1e6, rmsnorm=(n_q // n_kv == 7))
    L = Layer(wl, [700], bits, 4, 128, 1)
    L.fill()
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    assert L.check_decode_parity() <= 2e-3
    assert L.cache.status() == 0


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_ragged_batch_shuffled_pages_and_flush_sizes(bits):
    """Ragged lengths (config 2's structure, scaled down), page table in random order, S_flush > 1
    so that the recent window breathes, and appends that straddle page boundaries."""
    wl = _wl(8, 2, seed=21, batch=5, theta=5e5)
    lengths = [1, 63, 64, 65, 1000]
    for s_flush, lag in ((8, 0), (16, 1)):
        L = Layer(wl, lengths, bits, 4, 64, s_flush, lag=lag, page_shuffle_seed=3, max_seq_len=1024)
        steps = [[0, 10, 60, 3, 500], [1, 50, 3, 61, 436], [0, 2, 0, 0, 63], [0, 1, 1, 1, 1]]
        for st in steps:
            L.append_step(st)
        assert L.seq_len.cpu().tolist() == lengths
        assert L.check_append_parity() <= CODE_MISMATCH_MAX
        _check_window_copies(L)
        assert L.check_decode_parity() <= 2e-3
        assert L.cache.status() == 0


@pytest.mark.parametrize("s_sink,s_keep,s_flush", [(64, 256, 8), (16, 128, 16), (4, 64, 64)])
def test_serving_window_sizes(s_sink, s_keep, s_flush):
    """The window sizes of the paper's downstream (Section 5.3: 64 / 256 / 8) and perplexity (Section 5.2:
    16 / 128 / 16) runs, and a page-sized flush: long sink and recent windows, a boundary that moves in
    steps of S_flush, lengths around the point where quantization starts."""
    wl = _wl(8, 2, seed=23, batch=4)
    edge = s_sink + s_keep + s_flush
    lengths = [1100, edge - 1, edge, edge + s_flush + 3]
    L = Layer(wl, lengths, 2, s_sink, s_keep, s_flush)
    L.fill()
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    _check_window_copies(L)
    assert L.check_decode_parity() <= 2e-3
    assert L.cache.status() == 0


@pytest.mark.parametrize("path,bits", [("tensor", 2), ("cuda", 2), ("tensor", 3), ("cuda", 3), ("tensor_copies", 2), ("tensor_copies", 4)])
def test_prefill_chunk_paths(path, bits, test_option):
    """Config 4's structure scaled down: several sequences appended as one chunk each in ONE call
    (tile boundaries fall inside sequences and a ragged last tile), Qwen-shaped heads (G = 7, RMSNorm),
    through the tensor-core transform and through the CUDA-core chunk path; then one decode step."""
    if path == "cuda":
        test_option("append_path_cuda", 1)
    if path == "tensor_copies":                     # the tensor-core path staged with 16-byte copies instead of bulk tensor copies
        test_option("append_no_tma", 1)
    wl = _wl(28, 4, seed=41, batch=3, theta=1e6, rmsnorm=True)
    L = Layer(wl, [700, 131, 390], bits, 4, 128, 1)
    L.append_step([699, 130, 389])
    L.append_step([1, 1, 1])
    assert L.seq_len.cpu().tolist() == [700, 131, 390]
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    _check_window_copies(L)
    assert L.check_decode_parity() <= 2e-3
    assert L.cache.status() == 0


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_quest_quantizer_on_every_append_path(bits):
    """Section 4.3, Eq. 5 instead of Eq. 6: step from the group's RMS, bin-centre reconstruction.  One sequence
    goes through the tensor-core chunk path, one through the CUDA-core rows path, and every sequence gets a
    decode-time token; the packed cache is then decoded as usual."""
    wl = _wl(8, 2, seed=45, batch=3)
    L = Layer(wl, [400, 90, 131], bits, 4, 64, 8, quantizer="quest")
    L.append_step([399, 0, 0])        # chunk of >= 128 tokens: tensor-core transform, quad quantizer
    L.append_step([0, 89, 130])       # tensor-core path again (max_new 130) with a ragged tile
    L.append_step([1, 1, 1])          # single-token kernel
    assert L.seq_len.cpu().tolist() == [400, 90, 131]
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    assert L.check_decode_parity() <= 2e-3
    L2 = Layer(wl, [70, 33, 5], bits, 4, 64, 8, quantizer="quest")
    L2.append_step([69, 32, 4])       # max_new < 128: CUDA-core rows path
    L2.append_step([1, 1, 1])
    assert L2.check_append_parity() <= CODE_MISMATCH_MAX
    assert L2.check_decode_parity() <= 2e-3
    assert L.cache.status() == 0 and L2.cache.status() == 0


def test_window_edges_and_empty_sequences():
    """Degenerate cases of Section 4.4: nothing cached, everything inside the sink, nothing quantized
    yet (S <= S_sink + S_keep + S_flush - 1), exactly one flush group quantized."""
    wl = _wl(4, 1, seed=30, batch=6)
    s_sink, s_keep, s_flush = 4, 64, 8
    lengths = [0, 3, 4, s_sink + s_keep + s_flush - 1, s_sink + s_keep + s_flush, 200]
    L = Layer(wl, lengths, 2, s_sink, s_keep, s_flush, max_seq_len=256)
    L.fill()
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    _check_window_copies(L)
    assert L.check_decode_parity() <= 2e-3
    assert L.cache.status() == 0


def test_no_sink_and_kappa_one():
    wl = _wl(4, 1, seed=31)
    L = Layer(wl, [333], 4, 0, 1, 1, kappa_k=1.0, kappa_v=0.5)
    L.fill()
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    assert L.check_decode_parity() <= 2e-3


def test_decode_is_deterministic_and_split_invariant(test_option):
    """The split count changes only the summation order: outputs for different splits agree to fp32
    rounding, and two identical calls agree bit for bit."""
    wl = _wl(8, 2, seed=32)
    L = Layer(wl, [3000], 2, 4, 64, 1)
    L.fill()
    outs = []
    for ctas in (5, 5, 1, 64):
        test_option("decode_ctas", ctas)
        outs.append(L.decode()[0])
    assert np.array_equal(outs[0], outs[1])
    scale = np.max(np.abs(outs[0]))
    assert np.max(np.abs(outs[2] - outs[0])) <= 5e-4 * scale
    assert np.max(np.abs(outs[3] - outs[0])) <= 5e-4 * scale


@pytest.mark.parametrize("bits,n_q,n_kv", [(2, 8, 2), (4, 14, 2), (3, 8, 2)])
def test_fused_step_equals_append_then_decode(bits, n_q, n_kv):
    """wushkv_decode_step (queries transformed beside the append) gives, bit for bit, the cache and the
    outputs of wushkv_append + wushkv_decode_attn; several steps are enqueued back to back."""
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = _wl(n_q, n_kv, seed=41)
    lengths, steps = [700, 67, 3, 333], 3
    first = [n - steps for n in lengths]
    two, one = Layer(wl, lengths, bits, 4, 64, 1), Layer(wl, lengths, bits, 4, 64, 1)
    two.append_step(first, oracle_too=False)
    one.append_step(first, oracle_too=False)
    dev = one.cache.device
    qs = [np.stack([wl.queries(b, first[b] + i) for b in range(len(lengths))]) for i in range(steps)]
    ref = []
    for i in range(steps):
        two.append_step([1] * len(lengths), oracle_too=False)
        ref.append(two.decode(queries=qs[i])[0])
    bits16 = lambda x: torch.from_numpy(W.f32_to_bf16_bits(x).view(np.int16)).to(dev)  # noqa: E731
    Ks = [bits16(np.stack([one.tokens[b][0][first[b] + i] for b in range(len(lengths))])) for i in range(steps)]
    Vs = [bits16(np.stack([one.tokens[b][1][first[b] + i] for b in range(len(lengths))])) for i in range(steps)]
    Qs = [bits16(q) for q in qs]
    outs = [torch.full((len(lengths), n_q, 128), float("nan"), dtype=torch.float32, device=dev) for _ in range(steps)]
    cu = torch.arange(len(lengths) + 1, dtype=torch.int32, device=dev)
    nbytes = B.decode_workspace_bytes(one.cache.desc, one.batch, one.max_seq_len)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    for i in range(steps):                                   # no host synchronisation between the steps
        B.decode_step(one.cache.desc, one.batch, one.slot, one.seq_len, cu, one.max_seq_len, Ks[i], Vs[i], Qs[i],
                      outs[i], ws, nbytes)
    torch.cuda.synchronize()
    assert one.cache.status() == 0
    assert one.seq_len.cpu().tolist() == lengths
    for i in range(steps):
        assert np.array_equal(outs[i].cpu().numpy().astype(np.float64), ref[i]), f"step {i}"
    for b in range(len(lengths)):
        for h in range(n_kv):
            for which in (0, 1):
                for x, y in zip(one.gpu_codes(b, h, which), two.gpu_codes(b, h, which)):
                    assert np.array_equal(x, y)
        for x, y in zip(one.gpu_window_arrays(b), two.gpu_window_arrays(b)):
            assert np.array_equal(x, y, equal_nan=True)


def test_batch_larger_than_the_in_kernel_plan():
    """7000 short sequences: the work plan no longer fits the main kernel's staging area (it is read from
    the preparation kernel's copy instead), a warp's slice spans many (sequence, head) segments and
    takes several rounds, and most sequences are sink-only or nothing-quantized."""
    wl = _wl(2, 1, seed=71, batch=7000)
    rng = np.random.default_rng(71)
    lengths = [int(x) for x in rng.integers(0, 6, size=7000)]
    lengths[17] = 300
    L = Layer(wl, lengths, 2, 1, 2, 1)
    L.fill()
    Og, Q = L.decode()
    assert L.cache.status() == 0
    worst = 0.0
    for b in list(range(0, 7000, 97)) + [17, 6999]:
        if lengths[b] == 0:
            assert np.all(Og[b] == 0)
            continue
        ref = L.oracle_decode_on_gpu_cache(b, Q[b])
        worst = max(worst, np.max(np.abs(Og[b] - ref)) / np.max(np.abs(ref)))
    assert worst <= 2e-3
    assert all(np.all(Og[b] == 0) for b in range(7000) if lengths[b] == 0)


@pytest.mark.parametrize("log2_scale", [-6, 5])
def test_value_scale_invariance(log2_scale):
    """Scaling every value by a power of two scales the stored steps and offsets exactly and leaves the
    codes unchanged, so the outputs must scale with it up to what the fp16 operand p * Delta_v of the
    value contraction loses at the ends of its range (tiny probabilities fall into the subnormals at the
    low end; at the high end the stored step must stay below 1024, which with this workload's outlier
    channels is reached at a scale of 2^6)."""
    wl = _wl(8, 2, seed=61)
    outs = []
    for f in (1.0, 2.0 ** log2_scale):
        L = Layer(wl, [900, 130], 2, 4, 64, 1)
        L.tokens = [(K, V * np.float32(f)) for (K, V) in L.tokens]
        L.append_step([n - 1 for n in L.lengths], oracle_too=False)
        L.append_step([1] * L.batch, oracle_too=False)
        outs.append(L.decode()[0])
        if f != 1.0:
            codes_scaled = L.gpu_codes(0, 1, 1)[0]
        else:
            codes_plain = L.gpu_codes(0, 1, 1)[0]
    assert np.array_equal(codes_scaled, codes_plain)
    assert np.all(np.isfinite(outs[1]))
    assert np.max(np.abs(outs[1] * 2.0 ** -log2_scale - outs[0])) <= 5e-4 * np.max(np.abs(outs[0]))


@pytest.mark.parametrize("mode", ["mapped", "copy"])
def test_host_step_equals_device_step(mode, test_option):
    """wushkv_decode_step_host (pinned host buffers read and written in place, or staged copies when
    the "host_io_copy" option is set) gives the outputs and the cache of wushkv_decode_step, bit for bit."""
    import torch
    from paper_2609_38121_b200 import binding as B
    if mode == "copy":
        test_option("host_io_copy", 1)
    wl = _wl(8, 2, seed=43)
    lengths, steps = [400, 70, 2], 2
    first = [n - steps for n in lengths]
    dev_l, host_l = Layer(wl, lengths, 2, 4, 64, 1), Layer(wl, lengths, 2, 4, 64, 1)
    dev_l.append_step(first, oracle_too=False)
    host_l.append_step(first, oracle_too=False)
    dev = dev_l.cache.device
    nb = len(lengths)
    bits16 = lambda x: torch.from_numpy(W.f32_to_bf16_bits(x).view(np.int16))  # noqa: E731
    cu = torch.arange(nb + 1, dtype=torch.int32, device=dev)
    nbytes = B.decode_workspace_bytes(dev_l.cache.desc, nb, dev_l.max_seq_len)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    stg_bytes = B.step_staging_bytes(host_l.cache.desc, nb)
    stg = torch.empty(stg_bytes, dtype=torch.uint8, device=dev)
    for i in range(steps):
        K = bits16(np.stack([dev_l.tokens[b][0][first[b] + i] for b in range(nb)]))
        V = bits16(np.stack([dev_l.tokens[b][1][first[b] + i] for b in range(nb)]))
        Q = bits16(np.stack([wl.queries(b, first[b] + i) for b in range(nb)]))
        O_dev = torch.full((nb, 8, 128), float("nan"), dtype=torch.float32, device=dev)
        B.decode_step(dev_l.cache.desc, nb, dev_l.slot, dev_l.seq_len, cu, dev_l.max_seq_len, K.to(dev), V.to(dev), Q.to(dev),
                      O_dev, ws, nbytes)
        hK, hV, hQ = K.pin_memory(), V.pin_memory(), Q.pin_memory()
        hO = torch.full((nb, 8, 128), float("nan"), dtype=torch.float32).pin_memory()
        B.decode_step_host(host_l.cache.desc, nb, host_l.slot, host_l.seq_len, cu, host_l.max_seq_len, hK, hV, hQ, hO,
                           stg, stg_bytes, ws, nbytes)
        torch.cuda.synchronize()
        assert np.array_equal(hO.numpy(), O_dev.cpu().numpy()), f"step {i}"
    assert host_l.seq_len.cpu().tolist() == lengths and host_l.cache.status() == 0
    for b in range(nb):
        for h in range(2):
            for which in (0, 1):
                for x, y in zip(host_l.gpu_codes(b, h, which), dev_l.gpu_codes(b, h, which)):
                    assert np.array_equal(x, y)


def test_device_side_errors_are_flagged_not_fatal():
    """A position beyond the page table and a page id outside the pool set status bits; the calls
    still return and the rest of the batch is processed."""
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = _wl(4, 1, seed=33, batch=2)
    L = Layer(wl, [200, 200], 2, 4, 64, 1, max_seq_len=256)
    L.fill()
    assert L.cache.status() == 0
    good, _ = L.decode()
    # sequence 0 claims to be at the end of its page table: the append is skipped and flagged
    L.seq_len[0] = 256
    cu = torch.tensor([0, 1, 1], dtype=torch.int32, device="cuda")
    tok = torch.zeros((1, 1, 128), dtype=torch.int16, device="cuda")
    B.append(L.cache.desc, 2, L.slot, L.seq_len, cu, 1, 1, tok, tok)
    torch.cuda.synchronize()
    assert L.cache.status() & B.DEV_PAGE_TABLE_FULL
    # a corrupt page table entry inside the quantized range is skipped by decode and flagged
    L.seq_len[0] = 200
    L.cache.dev_status.zero_()
    L.cache.page_table[0, 1] = 10 ** 6
    out, _ = L.decode()
    assert L.cache.status() & B.DEV_BAD_PAGE_ID
    assert np.all(np.isfinite(out))
    assert np.array_equal(out[1], good[1])            # the healthy sequence is untouched


def test_host_side_capacity_and_alignment_errors():
    import torch
    from paper_2609_38121_b200 import binding as B
    wl = _wl(4, 1, seed=34)
    L = Layer(wl, [100], 2, 4, 64, 1)
    L.fill()
    Q = torch.zeros((1, 4, 128), dtype=torch.int16, device="cuda")
    Oo = torch.zeros((1, 4, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.WushkvError) as e:
        B.decode_attn(L.cache.desc, 1, L.slot, L.seq_len, 100, Q, Oo, ws, 16)
    assert e.value.status == B.ECAPACITY
    with pytest.raises(B.WushkvError) as e:
        B.decode_attn(L.cache.desc, 1, L.slot, L.seq_len, 100, Q, Oo, ws[8:], (1 << 20) - 8)
    assert e.value.status == B.EINVAL
    L.cache.desc.ring_cap = 10
    with pytest.raises(B.WushkvError) as e:
        B.decode_attn(L.cache.desc, 1, L.slot, L.seq_len, 100, Q, Oo, ws, 1 << 20)
    assert e.value.status == B.ECAPACITY
