import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture
def test_option():
    """Sets process-wide testing aids of the library (wushkv_set_test_option) and restores the
    defaults when the test ends."""
    from paper_2609_38121_b200 import binding as B
    defaults = {"decode_ctas": 0, "append_path_cuda": 0, "host_io_copy": 0, "drop_copy_unit": -1, "wait_limit": 0,
                "drop_chunk_mma": 0, "prefill_legacy": 0, "prefill_one_tile": 0, "prefill_split": 0, "prefill_no_tma": 0, "append_no_tma": 0, "drop_prefill": 0}
    used = []

    def _set(name, value):
        used.append(name)
        B.set_test_option(name, value)

    yield _set
    for name in used:
        B.set_test_option(name, defaults[name])
