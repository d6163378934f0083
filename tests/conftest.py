import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")
    config.addinivalue_line("markers", "slow: full-size workload (the oracle takes seconds to minutes); "
                                       "part of -m gpu, deselect with -m 'gpu and not slow'")


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
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _cuda_library_is_current():
    """Build the CUDA library in-tree if it is missing or older than its sources (a no-op otherwise),
    so that a fresh checkout runs the tests against the code it contains."""
    from paper_1711_04713_b200 import build
    build.build_library()
