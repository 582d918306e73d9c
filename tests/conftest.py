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
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_sessionstart(session):
    """Build the CUDA library once if it is missing or older than its sources (nvcc cross-compiles
    without a GPU). A failure here is not hidden: the tests that need the library then fail."""
    try:
        from paper_2509_24014_b200 import build
        build.build_library()
    except Exception as exc:  # pragma: no cover
        print(f"[conftest] could not build libsparsed.so: {exc}")
