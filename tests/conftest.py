import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the GPU box)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _no_bounds_violation():
    """With XG_DEBUG_BOUNDS=1 the tests run on the bounds-checking library; none of its checks may fail."""
    yield
    if os.environ.get("XG_DEBUG_BOUNDS") == "1":
        from paper_2601_04426_b200 import binding
        if binding._lib is not None and binding.lib().xg_debug_bounds_enabled():
            binding.debug_bounds_check()
