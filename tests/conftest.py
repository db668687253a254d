import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HERE = os.path.dirname(os.path.abspath(__file__))
if HERE not in sys.path:
    sys.path.insert(0, HERE)
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


def pytest_terminal_summary(terminalreporter):
    """Worst GPU-vs-oracle error seen per tensor kind during this run, beside its bounds."""
    try:
        import gpu_util
    except Exception:
        return
    if not gpu_util.OBSERVED:
        return
    terminalreporter.write_line("observed worst GPU-vs-oracle errors (row-norm relative; c: element-wise relative):")
    for name, err in sorted(gpu_util.OBSERVED.items()):
        terminalreporter.write_line(f"  {name:7s} {err:.3e}   tolerance {gpu_util.ROW_TOL:.0e}   regression bound {gpu_util.REGRESSION[name]:.1e}")
