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


@pytest.fixture(scope="module")
def cq():
    """The binding module behind guard bands: every output a GPU test receives sits between canary bytes that are
    checked after each call (tests/guards.py).  Fails, rather than skips, without a CUDA device."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2410_07505_b200 import build, cq as _cq
    build.build()
    _cq.lib()
    from guards import Guarded
    return Guarded(_cq)
