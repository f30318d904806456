"""GPU parity of chunk (prefill) attention over the mixed cache, wushkv_prefill_attn, against the oracle's
chunk_attn: Algorithm 2 line 5 for a chunk, Sections 4.4 and 5.3."""
import numpy as np
import pytest

from paper_2609_38121_b200 import workloads as W
from tests.harness import CODE_MISMATCH_MAX, Layer

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["tcgen05", "tcgen05_copies", "tcgen05_one_tile", "tcgen05_one_tile_copies", "mma_sync"], autouse=True)
def attention_path(request, test_option):
    """Every case runs on the warp-specialised tcgen05 kernel with bulk tensor copies (default), on the same kernel with
    plain 16-byte loads, on the one-tile-per-CTA tcgen05 kernel (both ways) and on the mma.sync kernel."""
    if request.param == "mma_sync":
        test_option("prefill_legacy", 1)
    if request.param.startswith("tcgen05_one_tile"):
        test_option("prefill_one_tile", 1)
    if request.param.endswith("copies"):
        test_option("prefill_no_tma", 1)
    return request.param


def _wl(n_q, n_kv, seed, batch=1, theta=1e4, rmsnorm=False):
    return W.LayerWorkload(dict(seed=seed, batch=batch, n_q=n_q, n_kv=n_kv, ctx=0, theta=theta, bits=2, s_sink=4,
                                s_keep=64, rmsnorm=rmsnorm, ragged=None, prefill_chunk=0))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_prefill_on_an_empty_cache(bits):
    """The whole prompt as one chunk: every key is a chunk position (full precision, causal); several query tiles,
    a ragged last tile, a sequence shorter than one tile."""
    wl = _wl(8, 2, seed=91, batch=3)
    L = Layer(wl, [333, 70, 9], bits, 4, 64, 1)
    assert L.check_prefill_parity([333, 70, 9]) <= 2e-3
    assert L.check_append_parity() <= CODE_MISMATCH_MAX
    assert L.cache.status() == 0


@pytest.mark.parametrize("bits,n_q,n_kv", [(2, 8, 2), (4, 14, 2), (3, 8, 2)])
def test_chunk_over_a_quantized_cache(bits, n_q, n_kv):
    """A chunk appended to a long cache: sink rows, packed pages (first and last one partly outside the quantized
    range), the old part of the recent window, then the chunk; ragged batch, shuffled page table, G = 4 and 7."""
    wl = _wl(n_q, n_kv, seed=92, batch=3)
    L = Layer(wl, [900, 450, 260], bits, 4, 64, 8, page_shuffle_seed=7)
    L.append_step([700, 300, 259])
    assert L.check_prefill_parity([200, 150, 1]) <= 2e-3        # the last sequence: a chunk of one token
    assert L.check_decode_parity() <= 2e-3                       # the cache is in order for the next decode step
    assert L.cache.status() == 0


@pytest.mark.parametrize("n_q,n_kv", [(2, 2), (6, 2), (5, 1), (12, 2), (16, 2)])
def test_head_group_sizes(n_q, n_kv):
    """G = 1, 3, 5, 6 and 8 query heads per KV head: a 128-row tile packs 128 / G chunk positions, which leaves rows
    unused when G does not divide 128, and a pair of tiles may end inside the chunk or be half empty; a chunk over a
    short quantized cache, ragged batch."""
    wl = _wl(n_q, n_kv, seed=96, batch=2)
    L = Layer(wl, [500, 310], 2, 4, 64, 8)
    L.append_step([300, 190])
    assert L.check_prefill_parity([200, 120]) <= 2e-3
    assert L.cache.status() == 0


@pytest.mark.parametrize("split", [1, 2, 3, 7, 16])
@pytest.mark.parametrize("bits", [2, 4])
def test_key_tiles_shared_between_ctas(split, bits, attention_path, test_option):
    """A short chunk over a long cache with the pair's key tiles cut into 1 .. 16 shares (one CTA each, partial results merged):
    shares that hold only packed pages, only the chunk's own tiles, nothing at all for the earlier query tile, or no tile."""
    if not attention_path.startswith("tcgen05") or "one_tile" in attention_path:
        pytest.skip("shares exist in the warp-specialised kernel only")
    test_option("prefill_split", split)
    wl = _wl(8, 2, seed=99, batch=2)
    L = Layer(wl, [1300, 200], bits, 4, 64, 8)
    L.append_step([1200, 120])
    assert L.check_prefill_parity([100, 80]) <= 2e-3
    assert L.cache.status() == 0


def test_chunk_attention_is_bit_identical_from_run_to_run():
    """The same call on the same cache state three times: the roles of the warp-specialised kernel meet in an order that
    depends on timing, the arithmetic must not (tile order of every accumulation is fixed)."""
    wl = _wl(14, 2, seed=98, batch=2)
    L = Layer(wl, [1500, 700], 2, 4, 64, 8)
    L.append_step([900, 300])
    L.prefill([600, 400], repeat=2)
    for other in L.repeats:
        assert np.array_equal(L.first.view(np.uint32), other.view(np.uint32))
    assert L.cache.status() == 0


def test_chunk_shorter_than_the_recent_window_and_second_chunk():
    """Chunks of 16 tokens as in the paper's perplexity runs (S_sink 16, S_keep 128, S_flush 16): old recent-window
    rows come from the ring, the quantized boundary sits below the chunk; two chunks in a row."""
    wl = _wl(8, 2, seed=93)
    L = Layer(wl, [432], 2, 16, 128, 16)
    L.append_step([400])
    assert L.check_prefill_parity([16]) <= 2e-3
    assert L.check_prefill_parity([16]) <= 2e-3
    assert L.cache.status() == 0


def test_literal_algorithm2_boundary():
    """boundary_lag = chunk length: the boundary of Algorithm 2 lines 7-8 is moved after attention."""
    wl = _wl(8, 2, seed=94)
    n_new = 40
    L = Layer(wl, [500], 2, 4, 64, 8, lag=n_new)
    L.append_step([460])
    assert L.check_prefill_parity([n_new]) <= 2e-3
    assert L.cache.status() == 0


def test_quest_cache_under_a_chunk():
    wl = _wl(8, 2, seed=95)
    L = Layer(wl, [600], 4, 4, 64, 1, quantizer="quest")
    L.append_step([400])
    assert L.check_prefill_parity([200]) <= 2e-3
    assert L.cache.status() == 0


@pytest.mark.parametrize("chunk", [2048, 96])
def test_long_chunk_over_a_long_quantized_cache(chunk, attention_path):
    """A 2048-token chunk appended to a 32768-token cache (512 packed pages, then the window rows, then 32 causal
    chunk tiles; two CTAs per tile pair), and a 96-token chunk over the same cache (16 CTAs per tile pair, 33 key tiles
    each); sampled chunk rows against the oracle."""
    if attention_path != "tcgen05":
        pytest.skip("the long case runs on the default kernel only")
    wl = _wl(8, 2, seed=97, theta=5e5)
    L = Layer(wl, [32768 + chunk], 2, 4, 128, 1)
    L.append_step([32768])
    worst = L.check_prefill_parity([chunk], rows=[r for r in (0, 1, 17, 63, 64, 95, 1023, 1024, 2000, 2047) if r < chunk])
    assert worst <= 2e-3
    assert L.cache.status() == 0
