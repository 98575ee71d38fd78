import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


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
    """Parity statistics gathered by the GPU tests: near-tie heads, index mismatches, max-abs errors."""
    try:
        from _harness import PARITY_STATS
    except Exception:
        return
    if PARITY_STATS:
        import json
        terminalreporter.write_sep("-", "parity statistics")
        for rec in PARITY_STATS:
            terminalreporter.write_line("PARITY " + json.dumps(rec))
