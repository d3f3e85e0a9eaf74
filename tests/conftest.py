import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the CUDA path through the C ABI)")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """Build (or refresh) libekv.so and the oracle once per session; both builds are no-ops when up to date.
    The library itself never builds or falls back on its own: a missing libekv.so is a loud ImportError."""
    from paper_2608_23658_b200 import build as ekv_build
    ekv_build.build()
    import oracle
    oracle.build()
