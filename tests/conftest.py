import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture
def snap_option():
    """Set process-wide testing options of the library for one test; restored afterwards."""
    from paper_2511_03092_b200 import binding as B
    changed = []

    def set_option(option, value):
        changed.append((option, B.snap_debug_set_option(option, value)))

    yield set_option
    for option, old in reversed(changed):
        B.snap_debug_set_option(option, old)
