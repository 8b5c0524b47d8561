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
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Table of every CUDA-vs-oracle comparison of the session: the bounded figure that was
    asserted and the plain max-abs/RMS figure beside it."""
    try:
        from tests import parity
    except Exception:
        return
    if not parity.REPORT:
        return
    tr = terminalreporter
    tr.write_sep("-", "parity figures (max-abs error / output RMS; bounded = asserted, raw = plain)")
    for case, stage, bounded, raw, note in parity.REPORT:
        tr.write_line("%-30s %-7s bounded %.3e  raw %.3e  %s" % (case, stage, bounded, raw, note))
