import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); deselected with -m 'not gpu'")


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


@pytest.fixture(autouse=True)
def _free_device_memory_after_each_test():
    """A failed test's traceback keeps its frame alive; the tens of GB a full-size rig holds must
    not stay allocated for the tests that follow."""
    yield
    import sys
    harness = sys.modules.get("kvr_harness")
    if harness is not None:
        harness.free_live()
