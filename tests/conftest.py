import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    import torch
    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _cuda_library_is_built():
    """On a GPU machine the library is compiled before the first test if it is missing or older than its sources (a no-op
    otherwise); the product itself never builds anything behind the caller's back and fails loudly without it."""
    import torch
    if torch.cuda.is_available():
        from paper_2603_03383_b200 import build
        build.build()
