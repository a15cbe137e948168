import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_collection_modifyitems(config, items):
    # nothing marked gpu may even try to start without a device
    try:
        import torch
        has = torch.cuda.is_available()
    except Exception:
        has = False
    if has:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    # parity counters per workload, action mismatches next to a CDF edge included
    try:
        import json
        from parity_util import SESSION_STATS
    except Exception:
        return
    if SESSION_STATS:
        terminalreporter.write_line("parity counters: " + json.dumps(SESSION_STATS, sort_keys=True))
