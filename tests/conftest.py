import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (B200); run with -m gpu")


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
    """One line on how far from a rounding tie the GPU's codes ever disagreed with the oracle's."""
    try:
        import parity_util
    except Exception:
        return
    o = parity_util.OBSERVED
    if o["codes_compared"]:
        terminalreporter.write_line(
            "parity: %d codes compared with the oracle, %d differ (%.2e), each within %.3e of a rounding tie "
            "(window %.1e)" % (o["codes_compared"], o["codes_mismatching"],
                               o["codes_mismatching"] / o["codes_compared"], o["tie_dist_max"], parity_util.TIE_WINDOW))
