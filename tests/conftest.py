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


def pytest_sessionfinish(session, exitstatus):
    """Runs of the suite under the bounds-checking build of the library (B2_EXPECT_CLEAN_BOUNDS=1,
    B2BLAS_LIB pointing at it) end by reading the checker's report: any access outside the extents
    of a call's arguments fails the run."""
    if not os.environ.get("B2_EXPECT_CLEAN_BOUNDS"):
        return
    from paper_2411_07211_b200 import binding
    rep = binding.debug_bounds_report()
    if rep is None:
        print("\nbounds check: the loaded library is not the bounds-checking build")
        session.exitstatus = 1
    elif rep[0] != 0:
        print(f"\nbounds check: {rep[0]} accesses outside the arguments' extents; first at {rep[1]:#x} ({rep[2]} bytes)")
        session.exitstatus = 1
    else:
        print("\nbounds check: clean")
