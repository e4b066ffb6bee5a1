import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); skipped by -m 'not gpu'")


@pytest.fixture(scope="session")
def cuda_device():
    import torch

    if not torch.cuda.is_available():
        pytest.fail("a test marked gpu ran on a machine without a CUDA device")
    return torch.device("cuda:0")


@pytest.fixture(scope="session", autouse=True)
def built_library():
    """Compile libodsgd.so when it is missing or older than its sources (nvcc cross-compiles
    without a GPU); a failed build fails the session loudly instead of skipping anything."""
    from paper_2005_06728_b200 import build

    return build.build()
