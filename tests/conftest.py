import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built library")


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
    """With a bounds-checking build of the library (GG_B200_LIB=...libgg_b200_bounds.so) the run must end with no
    checked access outside its buffer."""
    if not os.environ.get("GG_B200_LIB"):
        return
    from paper_2506_00486_b200 import binding
    if binding._lib is None:
        return
    n = binding.lib().gg_debug_bounds_violations()
    print(f"\nbounds-checking build: {n} checked accesses outside their buffers")
    if n > 0:
        session.exitstatus = 1
