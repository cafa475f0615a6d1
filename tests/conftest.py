import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


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
    """Build the C-ABI library if it is missing or older than its sources (nvcc cross-compiles
    without a GPU), so that the tests never run against a stale binary."""
    try:
        from paper_2503_14075_b200 import build
        build.build()
    except Exception as e:  # pragma: no cover - the ABI test reports the failure properly
        print("could not build libtwig.so:", e)
