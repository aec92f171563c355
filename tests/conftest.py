import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """Build libaq.so when it is missing and nvcc is present (no GPU needed)."""
    from paper_2605_24011_b200 import build as B
    if not os.path.exists(B.OUT) and os.path.exists(B.NVCC):
        B.build()
    yield
