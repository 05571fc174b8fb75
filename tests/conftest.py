import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def _have_gpu() -> bool:
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def pytest_collection_modifyitems(config, items):
    if _have_gpu():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _bounds_checking_build_saw_nothing():
    """When the run uses the bounds-checking build of the library (BLOAD_LIBRARY names libbload_debug.so), every global
    access of its copy, metadata and table kernels was checked against the buffers of its call; at the end of the session
    the record of refused accesses must be empty."""
    yield
    if os.path.basename(os.environ.get("BLOAD_LIBRARY", "")) == "libbload_debug.so" and _have_gpu():
        import paper_2310_10879_b200 as B
        st = B.bload_debug_status()
        assert st is not None, "BLOAD_LIBRARY does not name a bounds-checking build"
        assert st[0] == 0, "out-of-bounds accesses were refused: count %d, first in kernel %d, %s at address %#x" % (
            st[0], st[1], "write" if st[2] else "read", st[3])
