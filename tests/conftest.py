import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    """Skip gpu-marked tests when no device is present, so a plain `pytest tests`
    on a CPU machine stays green."""
    try:
        import torch
        have = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """Worst errors and near-tie counts the staged comparison saw in this run."""
    try:
        import parity
    except Exception:
        return
    if parity.OBSERVED:
        terminalreporter.write_sep("-", "staged comparison with the oracle: observed")
        for k in sorted(parity.OBSERVED):
            terminalreporter.write_line(f"{k}: {parity.OBSERVED[k]:.6g}")
