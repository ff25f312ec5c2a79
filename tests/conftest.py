import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (B200)")


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


def pytest_runtest_teardown(item, nextitem):
    """Against the bounds-check build (RELAY_B200_LIB set) every GPU test ends with a poll of the device error word."""
    if os.environ.get("RELAY_B200_LIB") and "gpu" in item.keywords:
        from paper_1810_00952_b200 import binding as B
        B.relay_poll_status()
