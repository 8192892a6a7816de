import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (the parity tests proper)")
    config.addinivalue_line("markers", "slow: full-size workloads")


def pytest_sessionstart(session):
    """Compile the CUDA library if the tree does not hold it yet (a fresh checkout): nvcc works
    without a GPU.  An existing library is used as it is."""
    from paper_2412_18052_b200 import build as cuda_build
    if not os.path.exists(cuda_build.LIB):
        cuda_build.build()


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
