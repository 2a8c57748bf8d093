import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """Compile libmars.so in-tree if it is missing or older than its sources (nvcc cross-compiles
    without a GPU).  A failed build is reported by the tests that need the library."""
    try:
        from paper_2601_15498_b200 import build
        build.build()
    except Exception as e:  # pragma: no cover
        print(f"libmars build skipped: {e}")
    yield


@pytest.fixture(autouse=True)
def _hooks_cleared():
    """No test inherits a forced launch shape from the one before it."""
    yield
    try:
        import hookctl
        hookctl.clear_all()
    except Exception:  # pragma: no cover  (library not built: the tests that need it report that)
        pass
