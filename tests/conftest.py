import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


@pytest.fixture(scope="session", autouse=True)
def _oracle_built():
    """Compile the CPU checker once per session (building it is not using it)."""
    from oracle import build as oracle_build
    oracle_build.build()
    yield
