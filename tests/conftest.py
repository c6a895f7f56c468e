import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


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


def pytest_terminal_summary(terminalreporter):
    """Largest errors the parity helpers saw (against the bars in parity_bars.py)."""
    try:
        import parity_bars
    except Exception:
        return
    if any(v > 0 for v in parity_bars.WORST.values()):
        terminalreporter.write_line("largest parity errors of this session: " +
                                    ", ".join(f"{k} {v:.3e}" for k, v in parity_bars.WORST.items()))
