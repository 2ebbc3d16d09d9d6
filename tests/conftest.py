import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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
def debug_hooks():
    """Sets the library's process-wide test hooks for one test and puts the defaults back afterwards."""
    from paper_2502_01068_b200 import binding as B
    keys = ("score_path", "score_partition", "fused_heads", "fused_lead", "wait_limit_cycles", "extra_publications",
            "prefill_skip_commit")

    def set_hook(key, value):
        assert key in keys
        B.fastkv_debug_set(key, value)

    yield set_hook
    for key in keys:
        B.fastkv_debug_set(key, 0)
