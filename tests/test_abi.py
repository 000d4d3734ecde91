"""Host-side checks that need no GPU: the shared library loads, exports every
symbol the header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1812_01776_b200 import build, estimator
    build.build()
    return estimator.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "il_estimator.h")).read()
    return sorted(set(re.findall(r"IL_API\s+[\w\s\*]*?\b(il_\w+)\s*\(", text)))


def test_header_declares_the_three_core_calls():
    names = declared_symbols()
    for core in ("il_estimator_create", "il_estimate", "il_estimator_destroy"):
        assert core in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_lists_every_declared_symbol():
    from paper_1812_01776_b200 import estimator
    assert sorted(estimator.EXPORTS) == declared_symbols()


def test_strerror_covers_codes(lib):
    seen = set()
    for code in range(0, -11, -1):
        msg = lib.il_strerror(code).decode()
        assert msg and msg != "unknown error"
        seen.add(msg)
    assert len(seen) == 11
    assert lib.il_strerror(-99).decode() == "unknown error"


def test_create_dag_rejects_bad_joins_on_the_host(lib):
    """A second incoming edge must come from a stage above the first parent and below the stage itself,
    and a stage keeps at most two outgoing edges; checked before any CUDA call."""
    from paper_1812_01776_b200 import estimator as E
    import workloads
    w = workloads.join_small(1, n=32)
    for p2 in ([-1, -1, -1, 1], [-1, -1, -1, 3], [-1, -1, -1, 0], [0, -1, -1, 2]):
        with pytest.raises(E.ILError) as e:
            E.il_estimator_create_dag(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits,
                                      join=(p2, w.join[1], w.join[2]))
        assert e.value.code == E.IL_ERR_BAD_TOPOLOGY
    with pytest.raises(E.ILError) as e:                     # stage 0 would have three outgoing edges
        E.il_estimator_create_dag(np.array([-1, 0, 0, 0], np.int32), w.cond_bit, w.cond_val, w.latency_us,
                                  w.arrival_us, w.branch_bits, join=w.join)
    assert e.value.code == E.IL_ERR_BAD_TOPOLOGY
    with pytest.raises(E.ILError) as e:                     # no such branch bit on the second edge
        E.il_estimator_create_dag(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits,
                                  join=(w.join[0], np.array([-1, -1, -1, 8], np.int8), w.join[2]))
    assert e.value.code == E.IL_ERR_BAD_TOPOLOGY


def test_create_rejects_bad_arguments_on_the_host(lib):
    """Validation comes before any CUDA call, so these run without a device."""
    from paper_1812_01776_b200 import estimator as E
    import workloads
    w = workloads.make(3, n_queries=64, n_candidates=1)

    def code(**kw):
        a = dict(parent=w.parent, cond_bit=w.cond_bit, cond_val=w.cond_val,
                 latency_us=w.latency_us, arrival_us=w.arrival_us, branch_bits=w.branch_bits)
        a.update(kw)
        try:
            h = E.il_estimator_create(**a)
        except E.ILError as e:
            return e.code
        E.il_estimator_destroy(h)
        return 0

    bad = w.parent.copy(); bad[2] = 2
    assert code(parent=bad) == E.IL_ERR_BAD_TOPOLOGY
    bad = w.parent.copy(); bad[2] = 0                       # three children of one stage
    assert code(parent=bad) == E.IL_ERR_BAD_TOPOLOGY
    bad = w.cond_bit.copy(); bad[3] = 9                     # no such branch bit
    assert code(cond_bit=bad) == E.IL_ERR_BAD_TOPOLOGY
    bad = w.latency_us.copy(); bad[1, 1, 5] = 0
    assert code(latency_us=bad) == E.IL_ERR_BAD_PROFILE
    bad = w.arrival_us.copy(); bad[10] = bad[9] - 1
    assert code(arrival_us=bad) == E.IL_ERR_BAD_TRACE
    bad = w.arrival_us.copy(); bad[0] = -1
    assert code(arrival_us=bad) == E.IL_ERR_BAD_TRACE
    bad = w.arrival_us.copy(); bad[-1] = 2 ** 62
    assert code(arrival_us=bad) == E.IL_ERR_BAD_TRACE
    assert code(branch_bits=None) == E.IL_ERR_INVALID_ARG
    # with valid inputs and no GPU the call must fail loudly, not fall back
    import torch
    if not torch.cuda.is_available():
        assert code() == E.IL_ERR_CUDA


def test_null_handle_calls(lib):
    assert lib.il_estimate(None, None, 1, 0, None, None) == -1
    assert lib.il_estimate_device(None, None, 1, 0, None, None) == -1
    assert lib.il_set_stream(None, None) == -1
    lib.il_estimator_destroy(None)
