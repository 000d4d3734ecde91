import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


@pytest.fixture(scope="session")
def oracle_pool(oracle):
    """Worker processes (spawn start method, so a CUDA context in the parent is
    no obstacle) that each run the single-threaded oracle on a slice of candidates."""
    pool = oracle.make_pool()
    yield pool
    pool.terminate()
