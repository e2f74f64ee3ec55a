import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the kernels through the C-ABI library)")


@pytest.fixture(scope="session")
def orc():
    from oracle import oracle
    oracle.build()
    return oracle


@pytest.fixture
def debug_flags():
    """Set the library's debug switches for one test; the defaults come back afterwards."""
    from paper_1804_10727_b200 import idf
    yield idf.set_debug_flags
    idf.set_debug_flags(0)
