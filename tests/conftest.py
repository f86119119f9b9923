import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """Totals of the verification parity tests: requests that differed from the oracle inside a
    near tie (the one allowed exception) against all decisions compared."""
    try:
        import parity_util
    except Exception:
        return
    t = parity_util.TOTALS
    if t["checks"]:
        terminalreporter.write_line(
            "verify parity: %d decisions compared in %d checks; requests that differ inside a near tie: "
            "%d by an accept / width / warp decision (bar 1e-4 of the decisions), %d by a sampled token "
            "(bar 1e-3)" % (t["decisions"], t["checks"], t["decision"], t["draw"]))


def pytest_sessionfinish(session, exitstatus):
    try:
        import parity_util
    except Exception:
        return
    t = parity_util.TOTALS
    if t["decision"] > 1e-4 * t["decisions"] or t["draw"] > parity_util.DRAW_RATE * t["decisions"]:
        session.exitstatus = 1
