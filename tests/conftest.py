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
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionfinish(session, exitstatus):
    """A run against the bounds-checked library (PPOW_LIBRARY=checked) fails if any check failed."""
    if os.environ.get("PPOW_LIBRARY") != "checked":
        return
    try:
        import torch
        if not torch.cuda.is_available():
            return
        from paper_2605_14978_b200 import binding as B
        status, failures, site = B.ppow_checked_failures()
    except Exception as e:                                   # the library could not be asked: that is a failure too
        print("\nbounds-checked build: could not read the counters: %r" % (e,))
        session.exitstatus = 3
        return
    print("\nbounds-checked build: %d failed checks (status %d, first site %d)" % (failures, status, site))
    if status != 0 or failures != 0:
        session.exitstatus = 3
