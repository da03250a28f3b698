import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """Make sure the CUDA library and the C oracle exist (both build in-tree; a no-op when they are current)."""
    from paper_2207_07736_b200 import build as cuda_build
    import oracle
    cuda_build.build()
    oracle.build()
