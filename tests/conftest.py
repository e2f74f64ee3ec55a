import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the kernels through the C-ABI library)")
    config.addinivalue_line("markers", "own_routing: leave the choice between the per-layer kernels and the all-layers launch to the library")


@pytest.fixture(scope="session")
def orc():
    from oracle import oracle
    oracle.build()
    return oracle


@pytest.fixture(autouse=True)
def _per_layer_kernels_by_default(request):
    """The GPU tests were written against the per-layer kernels, with groupings of rows chosen to hit their corner
    cases; by default the library answers small pushes with the single all-layers launch instead.  So every GPU test
    runs with that launch switched off unless it asks for the library's own routing (marker `own_routing`); the tests
    of the all-layers launch (test_fused_gpu.py) set the switches themselves."""
    if "gpu" not in request.keywords or "own_routing" in request.keywords:
        yield
        return
    from paper_1804_10727_b200 import idf
    idf.set_debug_flags(idf.DEBUG_NO_FUSED)
    yield
    idf.set_debug_flags(0)


@pytest.fixture
def debug_flags(request):
    """Set the library's debug switches for one test; the defaults come back afterwards."""
    from paper_1804_10727_b200 import idf
    base = 0 if "own_routing" in request.keywords else idf.DEBUG_NO_FUSED
    yield lambda flags: idf.set_debug_flags(flags | base)
    idf.set_debug_flags(0)
