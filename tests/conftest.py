import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session", autouse=True)
def _cuda_library_is_built():
    """Compile the CUDA library (nvcc cross-compiles without a GPU) when it is missing or stale."""
    from paper_2504_17096_b200 import build as cuda_build
    if cuda_build.is_stale():
        cuda_build.build()
