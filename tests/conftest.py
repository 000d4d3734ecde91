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


_ORACLE_RESULTS = {}


@pytest.fixture(scope="session")
def oracle_on(oracle, oracle_pool):
    """oracle_on(key, w, configs) -> (p99, miss) of the oracle for `configs` on workload w, computed
    once per session and key (the full-size samples take minutes of CPU time)."""
    import numpy as np

    def run(key, w, configs):
        if key not in _ORACLE_RESULTS:
            _ORACLE_RESULTS[key] = oracle.estimate_many_parallel(
                w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits,
                np.ascontiguousarray(configs), w.slo_us, pool=oracle_pool)
        return _ORACLE_RESULTS[key]
    return run
