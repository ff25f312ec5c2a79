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


def pytest_terminal_summary(terminalreporter):
    """fp32 parity: the plain (unfloored) relative error beside the gated one -- how many tests stay within 1e-4 on every
    non-zero element, and the largest ones."""
    try:
        from parity import STRICT_REL
    except Exception:
        return
    if not STRICT_REL:
        return
    within = sum(1 for v in STRICT_REL.values() if v <= 1e-4)
    terminalreporter.write_line(f"fp32 parity, plain max relative error over non-zero elements: {within} of {len(STRICT_REL)} tests <= 1e-4")
    for k, v in sorted(STRICT_REL.items(), key=lambda kv: -kv[1])[:8]:
        terminalreporter.write_line(f"  {v:.3e}  {k}")
