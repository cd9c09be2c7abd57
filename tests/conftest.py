import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle():
    """The CPU oracle (compiled on demand with gcc)."""
    import oracle as _oracle
    _oracle.lib()
    return _oracle


@pytest.fixture(params=[16, 23], ids=["rng16", "rng23"])
def rng_bits(request):
    """Resolution of the quantizer's uniform number: both supported values."""
    return request.param
