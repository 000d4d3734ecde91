"""Python face of the CPU oracle -- TEST INFRASTRUCTURE ONLY.

Loads ``des_oracle.c`` (compiled on demand with gcc into this folder) through
ctypes.  Only tests, the smoke check and the CPU-baseline leg of the bench may
import this package; the product path never does, and this package imports
nothing from the CUDA package.

The simulated semantics are documented at the top of ``des_oracle.c``
(InferLine Section 4.2 and the passages it cites).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "des_oracle.c")
_LIB = os.path.join(_HERE, "libdes_oracle.so")
_lib = None


class DispatchRecord(ctypes.Structure):
    _fields_ = [("stage", ctypes.c_int32), ("replica", ctypes.c_int32),
                ("batch", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("t_dispatch", ctypes.c_int64), ("t_finish", ctypes.c_int64)]


DISPATCH_DTYPE = np.dtype([("stage", "<i4"), ("replica", "<i4"), ("batch", "<i4"),
                           ("reserved", "<i4"), ("t_dispatch", "<i8"), ("t_finish", "<i8")])

ERRORS = {0: "ok", -1: "invalid argument", -2: "bad topology", -3: "bad profile",
          -4: "bad trace", -5: "bad config", -6: "out of memory", -7: "internal"}


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}: {ERRORS.get(code, '?')}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if (force or not os.path.exists(_LIB)
            or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        lib.orc_estimate_one.restype = ctypes.c_int
        lib.orc_estimate_one.argtypes = [ctypes.c_int32] * 3 + [p] * 4 + [ctypes.c_int64, p, p,
                                         p, ctypes.c_int64, ctypes.c_int32, p, p, p, p,
                                         ctypes.c_int64, p]
        lib.orc_estimate_one_dag.restype = ctypes.c_int
        lib.orc_estimate_one_dag.argtypes = [ctypes.c_int32] * 3 + [p] * 7 + [ctypes.c_int64, p, p,
                                             p, ctypes.c_int64, ctypes.c_int32, p, p, p, p,
                                             ctypes.c_int64, p]
        lib.orc_estimate_many_dag.restype = ctypes.c_int
        lib.orc_estimate_many_dag.argtypes = [ctypes.c_int32] * 3 + [p] * 7 + [ctypes.c_int64, p, p,
                                              p, ctypes.c_int64, ctypes.c_int64, p, p]
        lib.orc_estimate_many.restype = ctypes.c_int
        lib.orc_estimate_many.argtypes = [ctypes.c_int32] * 3 + [p] * 4 + [ctypes.c_int64, p, p,
                                          p, ctypes.c_int64, ctypes.c_int64, p, p]
        lib.orc_traffic_envelope.restype = ctypes.c_int
        lib.orc_traffic_envelope.argtypes = [ctypes.c_int64, p, ctypes.c_int32, p, p]
        lib.orc_p99_miss.restype = ctypes.c_int
        lib.orc_p99_miss.argtypes = [p, ctypes.c_int64, ctypes.c_int64, p, p]
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _prep(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits):
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    cond_bit = np.ascontiguousarray(cond_bit, dtype=np.int8)
    cond_val = np.ascontiguousarray(cond_val, dtype=np.uint8)
    latency_us = np.ascontiguousarray(latency_us, dtype=np.int32)
    arrival_us = np.ascontiguousarray(arrival_us, dtype=np.int64)
    if branch_bits is not None:
        branch_bits = np.ascontiguousarray(branch_bits, dtype=np.uint8)
    S, H, B = latency_us.shape
    assert parent.shape == (S,) and cond_bit.shape == (S,) and cond_val.shape == (S,)
    return parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits, S, H, B


def _prep_join(join, S):
    """join = None or (parent2, cond_bit2, cond_val2): per stage the second incoming edge."""
    if join is None:
        return None, None, None
    parent2 = np.ascontiguousarray(join[0], dtype=np.int32)
    cond_bit2 = np.ascontiguousarray(join[1], dtype=np.int8)
    cond_val2 = np.ascontiguousarray(join[2], dtype=np.uint8)
    assert parent2.shape == (S,) and cond_bit2.shape == (S,) and cond_val2.shape == (S,)
    return parent2, cond_bit2, cond_val2


def estimate_one(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
                 config, slo_us: int, replica_pref: int = 0, want_latency: bool = False,
                 want_log: bool = False, join=None):
    """Simulate one candidate; returns (p99_us, miss[, latency][, dispatch log])."""
    lib = _load()
    parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits, S, H, B = _prep(
        parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits)
    config = np.ascontiguousarray(config, dtype=np.uint8)
    assert config.shape == (S, 4)
    n = arrival_us.shape[0]
    p99, miss, nlog = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    lat = np.empty(n, dtype=np.int64) if want_latency else None
    cap = int(n) * S if want_log else 0
    log = np.zeros(cap, dtype=DISPATCH_DTYPE) if want_log else None
    parent2, cond_bit2, cond_val2 = _prep_join(join, S)
    rc = lib.orc_estimate_one_dag(S, H, B, _ptr(parent), _ptr(cond_bit), _ptr(cond_val),
                              _ptr(parent2), _ptr(cond_bit2), _ptr(cond_val2),
                              _ptr(latency_us), n, _ptr(arrival_us), _ptr(branch_bits),
                              _ptr(config), int(slo_us), int(replica_pref),
                              ctypes.addressof(p99), ctypes.addressof(miss), _ptr(lat),
                              _ptr(log), cap, ctypes.addressof(nlog))
    if rc:
        raise OracleError(rc)
    out = [int(p99.value), int(miss.value)]
    if want_latency:
        out.append(lat)
    if want_log:
        out.append(log[:nlog.value])
    return tuple(out)


def estimate_many(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
                  configs, slo_us: int, join=None) -> Tuple[np.ndarray, np.ndarray]:
    """Simulate configs[c] for every c, one after the other, on this thread."""
    lib = _load()
    parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits, S, H, B = _prep(
        parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits)
    configs = np.ascontiguousarray(configs, dtype=np.uint8)
    assert configs.ndim == 3 and configs.shape[1:] == (S, 4)
    C = configs.shape[0]
    p99 = np.zeros(C, dtype=np.int64)
    miss = np.zeros(C, dtype=np.int64)
    parent2, cond_bit2, cond_val2 = _prep_join(join, S)
    rc = lib.orc_estimate_many_dag(S, H, B, _ptr(parent), _ptr(cond_bit), _ptr(cond_val),
                               _ptr(parent2), _ptr(cond_bit2), _ptr(cond_val2),
                               _ptr(latency_us), arrival_us.shape[0], _ptr(arrival_us),
                               _ptr(branch_bits), _ptr(configs), C, int(slo_us),
                               _ptr(p99), _ptr(miss))
    if rc:
        raise OracleError(rc)
    return p99, miss


def estimate_workload(w, lo: int = 0, hi: Optional[int] = None):
    """estimate_many over candidates [lo, hi) of a workloads.Workload-like object."""
    hi = w.configs.shape[0] if hi is None else hi
    return estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                         w.branch_bits, w.configs[lo:hi], w.slo_us, join=getattr(w, "join", None))


def _worker(args):
    (parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits, configs, slo_us) = args
    return estimate_many(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
                         configs, slo_us)


def _noop(_):
    return os.getpid()


def make_pool(processes: Optional[int] = None):
    """A pool of worker processes (``spawn`` start method, so it is safe to
    create after a CUDA context exists in the parent) that have the oracle
    library loaded.  Pass it to estimate_many_parallel to keep process start-up
    out of a timed region; close it with ``pool.terminate()``."""
    import multiprocessing as mp
    build()
    P = max(1, processes or (os.cpu_count() or 1))
    pool = mp.get_context("spawn").Pool(P)
    pool.map(_noop, range(4 * P), chunksize=1)      # make every worker import this module
    return pool


def estimate_many_parallel(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
                           configs, slo_us: int, processes: Optional[int] = None, pool=None):
    """Disjoint slices of the candidates on separate processes (each candidate
    is still simulated by one thread).  Uses the ``spawn`` start method so it is
    safe to call after a CUDA context exists in the parent."""
    import multiprocessing as mp
    build()
    configs = np.ascontiguousarray(configs, dtype=np.uint8)
    C = configs.shape[0]
    P = max(1, min(processes or (os.cpu_count() or 1), C))
    if pool is not None:
        n_chunks = min(C, P * 8)
        bounds = np.linspace(0, C, n_chunks + 1).astype(np.int64)
        jobs = [(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
                 configs[bounds[i]:bounds[i + 1]], slo_us) for i in range(n_chunks)]
        parts = pool.map(_worker, jobs, chunksize=1)
        return (np.concatenate([p[0] for p in parts]), np.concatenate([p[1] for p in parts]))
    if P == 1:
        return estimate_many(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
                             configs, slo_us)
    # small interleaved chunks balance the (very uneven) cost per candidate
    n_chunks = min(C, P * 8)
    bounds = np.linspace(0, C, n_chunks + 1).astype(np.int64)
    jobs = [(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits,
             configs[bounds[i]:bounds[i + 1]], slo_us) for i in range(n_chunks)]
    with mp.get_context("spawn").Pool(P) as pool:
        parts = pool.map(_worker, jobs, chunksize=1)
    return (np.concatenate([p[0] for p in parts]), np.concatenate([p[1] for p in parts]))


def p99_miss(latency, slo_us: int) -> Tuple[int, int]:
    """k-th smallest latency with k = ceil(0.99 n), and the count above slo_us."""
    lib = _load()
    latency = np.ascontiguousarray(latency, dtype=np.int64)
    p99, miss = ctypes.c_int64(0), ctypes.c_int64(0)
    rc = lib.orc_p99_miss(_ptr(latency), latency.shape[0], int(slo_us),
                          ctypes.addressof(p99), ctypes.addressof(miss))
    if rc:
        raise OracleError(rc)
    return int(p99.value), int(miss.value)


def traffic_envelope(arrival_us, window_us) -> np.ndarray:
    """Largest number of arrivals in any half-open window of each given length
    (Section 5 of the paper: the traffic envelope the Planner hands to the Tuner)."""
    lib = _load()
    arrival_us = np.ascontiguousarray(arrival_us, dtype=np.int64)
    window_us = np.ascontiguousarray(window_us, dtype=np.int64)
    out = np.zeros(window_us.shape[0], dtype=np.int64)
    rc = lib.orc_traffic_envelope(arrival_us.shape[0], _ptr(arrival_us), window_us.shape[0],
                                  _ptr(window_us), _ptr(out))
    if rc:
        raise OracleError(rc)
    return out
