import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


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


@pytest.fixture(autouse=True)
def _bounds_checked_build_is_clean(request):
    """When the suite runs against the bounds-checked build (MUSE_LIBRARY=libmuse_debug.so), no GPU test
    may leave an out-of-range index on record."""
    yield
    if "gpu" not in request.keywords or "debug" not in os.environ.get("MUSE_LIBRARY", ""):
        return
    from paper_2509_10406_b200 import binding as mb
    n, text = mb.muse_debug_report(reset=True)
    assert n == 0, text
