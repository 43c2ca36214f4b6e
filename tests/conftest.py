import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """How the kept lists of this run compared with the oracle's (see helpers.assert_indices_match)."""
    try:
        from helpers import INDEX_LOG
    except ImportError:
        return
    if INDEX_LOG["lists"]:
        terminalreporter.write_line("kept lists compared with the oracle: %d, identical: %d, largest distance of a "
                                    "differing entry from the threshold: %.3f tolerances"
                                    % (INDEX_LOG["lists"], INDEX_LOG["identical"], INDEX_LOG["worst"]))
