import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


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


def pytest_terminal_summary(terminalreporter):
    """Exact-match rates of the parity cases against the oracle (the band rule accepts a swap at a
    pool or result boundary within tolerance; this says how often one happened)."""
    from tests import parity
    if parity.REPORT:
        terminalreporter.write_sep("-", "parity: share of judged queries whose id sets equal the oracle's")
        for line in parity.REPORT:
            terminalreporter.write_line(line)
