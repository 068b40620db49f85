import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


import pytest


@pytest.fixture(scope="session", autouse=True)
def _native_pieces_are_built():
    """Compile what is stale before any test runs: the CUDA library (nvcc
    cross-compiles without a GPU) and the oracle (gcc)."""
    from paper_2604_14561_b200 import build
    import oracle
    build.build()
    oracle.build()
