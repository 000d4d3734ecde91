"""ctypes binding of the Estimator's C ABI.

The functions named ``il_*`` mirror the C entry points one to one and only
convert arguments.  ``Estimator`` is a convenience wrapper that owns a handle
and uses torch for device buffers, the stream and the workspace.  There is no
fallback: if the shared library is missing or no CUDA device is present the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# IL_ESTIMATOR_CHECKED=1 in the environment selects the bounds-checked build of the same sources
_LIB_PATH = os.path.join(_HERE, "libil_estimator_checked.so" if os.environ.get("IL_ESTIMATOR_CHECKED") == "1"
                         else "libil_estimator.so")
_lib = None

IL_OK = 0
IL_ERR_INVALID_ARG, IL_ERR_BAD_TOPOLOGY, IL_ERR_BAD_PROFILE, IL_ERR_BAD_TRACE = -1, -2, -3, -4
IL_ERR_BAD_CONFIG, IL_ERR_NOMEM, IL_ERR_CUDA, IL_ERR_ITER_LIMIT = -5, -6, -7, -8
IL_ERR_TOO_LARGE = -9
IL_ERR_BOUNDS = -10
IL_VARIANT_AUTO, IL_VARIANT_WIDE, IL_VARIANT_STAGED, IL_VARIANT_LANES, IL_VARIANT_PACKED = 0, 1, 2, 3, 4
IL_STATIC_SCRATCH_BYTES = 32 * 1024 * 1024
IL_KNOB_LANE_RING_LOG2, IL_KNOB_ITER_LIMIT, IL_KNOB_SHARE_PREFIXES, IL_KNOB_LANE_CTAS, IL_KNOB_BITS_IN_RECORDS = 1, 2, 3, 4, 5

EXPORTS = ["il_estimator_create", "il_estimator_destroy", "il_estimate", "il_estimate_device",
           "il_set_stream", "il_workspace_bytes", "il_workspace_min_bytes", "il_set_workspace",
           "il_get_stats", "il_stage_visits", "il_strerror", "il_last_cuda_error",
           "il_measure_int_issue", "il_estimate_device_static", "il_set_variant", "il_estimate_latencies", "il_traffic_envelope", "il_kernel_name",
           "il_set_test_knob", "il_feasible", "il_feasible_device", "il_estimator_create_dag"]


class ILError(RuntimeError):
    def __init__(self, code: int, what: str = ""):
        lib = load_library()
        msg = lib.il_strerror(code).decode()
        if code == IL_ERR_CUDA:
            msg += f" (cudaError {lib.il_last_cuda_error()})"
        super().__init__(f"{what}: {msg} [{code}]" if what else f"{msg} [{code}]")
        self.code = code


class _Profiles(ctypes.Structure):
    _fields_ = [("n_stages", ctypes.c_int32), ("n_hw", ctypes.c_int32),
                ("max_batch", ctypes.c_int32), ("parent", ctypes.c_void_p),
                ("cond_bit", ctypes.c_void_p), ("cond_val", ctypes.c_void_p),
                ("latency_us", ctypes.c_void_p)]


class _JoinEdges(ctypes.Structure):
    _fields_ = [("parent2", ctypes.c_void_p), ("cond_bit2", ctypes.c_void_p), ("cond_val2", ctypes.c_void_p)]


class _Trace(ctypes.Structure):
    _fields_ = [("n_queries", ctypes.c_int64), ("arrival_us", ctypes.c_void_p),
                ("branch_bits", ctypes.c_void_p)]


class StageConfig(ctypes.Structure):
    _fields_ = [("hw", ctypes.c_uint8), ("max_batch", ctypes.c_uint8),
                ("replicas", ctypes.c_uint8), ("reserved", ctypes.c_uint8)]


class Stats(ctypes.Structure):
    _fields_ = [("candidates", ctypes.c_int64), ("query_events", ctypes.c_int64),
                ("batches", ctypes.c_int64), ("algorithmic_ops", ctypes.c_int64),
                ("chunks", ctypes.c_int64),
                ("kernel_launches", ctypes.c_int64), ("sim_ms", ctypes.c_double),
                ("select_ms", ctypes.c_double), ("total_ms", ctypes.c_double),
                ("fallback_candidates", ctypes.c_int64), ("stage_runs", ctypes.c_int64),
                ("error_detail", ctypes.c_int64), ("early_exits", ctypes.c_int64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libil_estimator.so (built in-tree by paper_1812_01776_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_1812_01776_b200.build` "
                          "(needs nvcc); there is no fallback path")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i64 = ctypes.c_void_p, ctypes.c_int64
    lib.il_estimator_create.restype = ctypes.c_int
    lib.il_estimator_create.argtypes = [ctypes.POINTER(_Profiles), ctypes.POINTER(_Trace),
                                        ctypes.POINTER(vp)]
    lib.il_estimator_create_dag.restype = ctypes.c_int
    lib.il_estimator_create_dag.argtypes = [ctypes.POINTER(_Profiles), ctypes.POINTER(_JoinEdges),
                                            ctypes.POINTER(_Trace), ctypes.POINTER(vp)]
    lib.il_estimator_destroy.restype = None
    lib.il_estimator_destroy.argtypes = [vp]
    lib.il_estimate.restype = ctypes.c_int
    lib.il_estimate.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.il_estimate_device.restype = ctypes.c_int
    lib.il_estimate_device.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.il_feasible.restype = ctypes.c_int
    lib.il_feasible.argtypes = [vp, vp, i64, i64, vp]
    lib.il_feasible_device.restype = ctypes.c_int
    lib.il_feasible_device.argtypes = [vp, vp, i64, i64, vp]
    lib.il_estimate_device_static.restype = ctypes.c_int
    lib.il_estimate_device_static.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.il_estimate_latencies.restype = ctypes.c_int
    lib.il_estimate_latencies.argtypes = [vp, vp, vp]
    lib.il_traffic_envelope.restype = ctypes.c_int
    lib.il_traffic_envelope.argtypes = [vp, vp, ctypes.c_int32, vp]
    lib.il_kernel_name.restype = ctypes.c_char_p
    lib.il_kernel_name.argtypes = [vp]
    lib.il_set_variant.restype = ctypes.c_int
    lib.il_set_variant.argtypes = [vp, ctypes.c_int]
    lib.il_set_stream.restype = ctypes.c_int
    lib.il_set_stream.argtypes = [vp, vp]
    lib.il_set_test_knob.restype = ctypes.c_int
    lib.il_set_test_knob.argtypes = [vp, ctypes.c_int, i64]
    lib.il_workspace_bytes.restype = ctypes.c_int
    lib.il_workspace_bytes.argtypes = [vp, i64, ctypes.POINTER(ctypes.c_size_t)]
    lib.il_workspace_min_bytes.restype = ctypes.c_int
    lib.il_workspace_min_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    lib.il_set_workspace.restype = ctypes.c_int
    lib.il_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.il_get_stats.restype = ctypes.c_int
    lib.il_get_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    lib.il_stage_visits.restype = ctypes.c_int
    lib.il_stage_visits.argtypes = [vp, vp]
    lib.il_strerror.restype = ctypes.c_char_p
    lib.il_strerror.argtypes = [ctypes.c_int]
    lib.il_last_cuda_error.restype = ctypes.c_int
    lib.il_last_cuda_error.argtypes = []
    lib.il_measure_int_issue.restype = ctypes.c_int
    lib.il_measure_int_issue.argtypes = [vp, ctypes.POINTER(ctypes.c_double),
                                         ctypes.POINTER(ctypes.c_double)]
    _lib = lib
    return lib


def _check(rc: int, what: str):
    if rc != IL_OK:
        raise ILError(rc, what)


def il_strerror(code: int) -> str:
    return load_library().il_strerror(code).decode()


# ---- one-to-one wrappers (host numpy arrays / raw device pointers) ----------

def il_estimator_create_dag(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits=None, join=None):
    """il_estimator_create_dag: as il_estimator_create, with join = (parent2, cond_bit2, cond_val2),
    per stage the second incoming edge (parent2[s] = -1: none), or None."""
    return il_estimator_create(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits, _join=join,
                               _dag=True)


def il_estimator_create(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits=None, _join=None,
                        _dag=False):
    """il_estimator_create: host arrays in, opaque handle out."""
    lib = load_library()
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    cond_bit = np.ascontiguousarray(cond_bit, dtype=np.int8)
    cond_val = np.ascontiguousarray(cond_val, dtype=np.uint8)
    latency_us = np.ascontiguousarray(latency_us, dtype=np.int32)
    arrival_us = np.ascontiguousarray(arrival_us, dtype=np.int64)
    if latency_us.ndim != 3:
        raise ValueError("latency_us must be [S][H][Bmax]")
    S, H, B = latency_us.shape
    if parent.shape != (S,) or cond_bit.shape != (S,) or cond_val.shape != (S,):
        raise ValueError("parent / cond_bit / cond_val must have one entry per stage")
    if branch_bits is not None:
        branch_bits = np.ascontiguousarray(branch_bits, dtype=np.uint8)
        if branch_bits.shape != arrival_us.shape:
            raise ValueError("branch_bits must have one entry per query")
    pr = _Profiles(S, H, B, parent.ctypes.data, cond_bit.ctypes.data, cond_val.ctypes.data,
                   latency_us.ctypes.data)
    tr = _Trace(arrival_us.shape[0], arrival_us.ctypes.data,
                None if branch_bits is None else branch_bits.ctypes.data)
    handle = ctypes.c_void_p()
    if _dag:
        jn = None
        if _join is not None:
            parent2 = np.ascontiguousarray(_join[0], dtype=np.int32)
            cond_bit2 = np.ascontiguousarray(_join[1], dtype=np.int8)
            cond_val2 = np.ascontiguousarray(_join[2], dtype=np.uint8)
            if parent2.shape != (S,) or cond_bit2.shape != (S,) or cond_val2.shape != (S,):
                raise ValueError("the join arrays must have one entry per stage")
            jn = ctypes.byref(_JoinEdges(parent2.ctypes.data, cond_bit2.ctypes.data, cond_val2.ctypes.data))
        _check(lib.il_estimator_create_dag(ctypes.byref(pr), jn, ctypes.byref(tr), ctypes.byref(handle)),
               "il_estimator_create_dag")
        return handle
    _check(lib.il_estimator_create(ctypes.byref(pr), ctypes.byref(tr), ctypes.byref(handle)),
           "il_estimator_create")
    return handle


def il_estimator_destroy(handle) -> None:
    if handle:
        load_library().il_estimator_destroy(handle)


def il_estimate(handle, configs: np.ndarray, slo_us: int) -> Tuple[np.ndarray, np.ndarray]:
    """il_estimate: host configs [n][S][4] uint8 in, host (p99_us, miss) int64 out."""
    lib = load_library()
    configs = np.ascontiguousarray(configs, dtype=np.uint8)
    if configs.ndim != 3 or configs.shape[2] != 4:
        raise ValueError("configs must be [n][S][4] uint8")
    n = configs.shape[0]
    p99 = np.empty(n, dtype=np.int64)
    miss = np.empty(n, dtype=np.int64)
    _check(lib.il_estimate(handle, configs.ctypes.data, n, int(slo_us), p99.ctypes.data,
                           miss.ctypes.data), "il_estimate")
    return p99, miss


def il_estimate_device(handle, d_configs: int, n: int, slo_us: int, d_out_p99: int,
                       d_out_miss: int) -> None:
    """il_estimate_device: raw device pointers (ints) in, results written in place."""
    _check(load_library().il_estimate_device(handle, d_configs, int(n), int(slo_us), d_out_p99,
                                             d_out_miss), "il_estimate_device")


def il_feasible(handle, configs: np.ndarray, slo_us: int) -> np.ndarray:
    """il_feasible: host configs [n][S][4] uint8 in, host bool array out (P99 <= slo_us)."""
    configs = np.ascontiguousarray(configs, dtype=np.uint8)
    if configs.ndim != 3 or configs.shape[2] != 4:
        raise ValueError("configs must be [n][S][4] uint8")
    out = np.empty(configs.shape[0], dtype=np.uint8)
    _check(load_library().il_feasible(handle, configs.ctypes.data, configs.shape[0], int(slo_us),
                                      out.ctypes.data), "il_feasible")
    return out.astype(bool)


def il_feasible_device(handle, d_configs: int, n: int, slo_us: int, d_out_feasible: int) -> None:
    """il_feasible_device: raw device pointers (ints) in, one byte per candidate written in place."""
    _check(load_library().il_feasible_device(handle, d_configs, int(n), int(slo_us), d_out_feasible),
           "il_feasible_device")


def il_estimate_device_static(handle, d_configs: int, n: int, slo_us: int, d_out_p99: int,
                              d_out_miss: int) -> None:
    """il_estimate_device_static: like il_estimate_device, but the library
    allocates nothing; scratch is the static array built into the library."""
    _check(load_library().il_estimate_device_static(handle, d_configs, int(n), int(slo_us),
                                                    d_out_p99, d_out_miss),
           "il_estimate_device_static")


def il_estimate_latencies(handle, d_config: int, d_out_latency: int) -> None:
    """il_estimate_latencies: one candidate (device pointer) in, per-query latencies written in place."""
    _check(load_library().il_estimate_latencies(handle, d_config, d_out_latency), "il_estimate_latencies")


def il_traffic_envelope(handle, window_us) -> np.ndarray:
    """il_traffic_envelope: host window lengths in, host maximum counts out."""
    window_us = np.ascontiguousarray(window_us, dtype=np.int64)
    out = np.zeros(window_us.shape[0], dtype=np.int64)
    _check(load_library().il_traffic_envelope(handle, window_us.ctypes.data, window_us.shape[0],
                                              out.ctypes.data), "il_traffic_envelope")
    return out


def il_set_variant(handle, variant: int) -> None:
    _check(load_library().il_set_variant(handle, int(variant)), "il_set_variant")


def il_set_test_knob(handle, knob: int, value: int) -> None:
    """il_set_test_knob: hooks for the tests (ring length of the lane kernel, iteration bound)."""
    _check(load_library().il_set_test_knob(handle, int(knob), int(value)), "il_set_test_knob")


def il_kernel_name(handle) -> str:
    """il_kernel_name: the simulation kernel the next estimate call launches."""
    return load_library().il_kernel_name(handle).decode()


def il_set_stream(handle, cuda_stream: int) -> None:
    _check(load_library().il_set_stream(handle, cuda_stream), "il_set_stream")


def il_workspace_bytes(handle, n_candidates: int) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().il_workspace_bytes(handle, int(n_candidates), ctypes.byref(out)),
           "il_workspace_bytes")
    return int(out.value)


def il_workspace_min_bytes(handle) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().il_workspace_min_bytes(handle, ctypes.byref(out)), "il_workspace_min_bytes")
    return int(out.value)


def il_set_workspace(handle, d_ptr: int, nbytes: int) -> None:
    _check(load_library().il_set_workspace(handle, d_ptr, int(nbytes)), "il_set_workspace")


def il_get_stats(handle) -> dict:
    st = Stats()
    _check(load_library().il_get_stats(handle, ctypes.byref(st)), "il_get_stats")
    return st.as_dict()


def il_stage_visits(handle, n_stages: int) -> np.ndarray:
    out = np.zeros(n_stages, dtype=np.int64)
    _check(load_library().il_stage_visits(handle, out.ctypes.data), "il_stage_visits")
    return out


def il_measure_int_issue(cuda_stream: int = 0) -> Tuple[float, float]:
    """Returns (warp-instructions per second, milliseconds the probe ran)."""
    rate, ms = ctypes.c_double(0), ctypes.c_double(0)
    _check(load_library().il_measure_int_issue(cuda_stream, ctypes.byref(rate), ctypes.byref(ms)),
           "il_measure_int_issue")
    return rate.value, ms.value


# ---- convenience wrapper with torch-owned device memory ---------------------

class Estimator:
    """Owns one handle bound to a workload's profiles and trace.

    torch supplies device buffers, the current stream and the workspace; every
    step of the computation runs inside the library.
    """

    def __init__(self, parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits=None,
                 device: Optional[int] = None, join=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the Estimator needs a CUDA device (sm_100a); there is no CPU path")
        self._torch = torch
        self.device = torch.device("cuda", torch.cuda.current_device() if device is None else device)
        self.n_stages = int(np.asarray(latency_us).shape[0])
        self.n_queries = int(np.asarray(arrival_us).shape[0])
        with torch.cuda.device(self.device):
            if join is None:
                self._h = il_estimator_create(parent, cond_bit, cond_val, latency_us, arrival_us,
                                              branch_bits)
            else:
                self._h = il_estimator_create_dag(parent, cond_bit, cond_val, latency_us, arrival_us,
                                                  branch_bits, join=join)
        self._ws = None
        self.visits = il_stage_visits(self._h, self.n_stages)

    @classmethod
    def from_workload(cls, w, device: Optional[int] = None) -> "Estimator":
        return cls(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits,
                   device=device, join=getattr(w, "join", None))

    def close(self) -> None:
        if getattr(self, "_h", None):
            il_estimator_destroy(self._h)
            self._h = None
            self._ws = None

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def reserve_workspace(self, n_candidates: int, max_bytes: Optional[int] = None) -> int:
        """Allocates the scratch buffer with torch and hands it to the library."""
        torch = self._torch
        want = il_workspace_bytes(self._h, n_candidates)
        with torch.cuda.device(self.device):
            free_b, _ = torch.cuda.mem_get_info()
            if max_bytes is None and want > int(free_b * 0.8):
                # blocks torch keeps cached from earlier tensors count as used: hand them back first
                torch.cuda.empty_cache()
                free_b, _ = torch.cuda.mem_get_info()
            cap = int(free_b * 0.8) if max_bytes is None else int(max_bytes)
            nbytes = max(min(want, cap), il_workspace_min_bytes(self._h))
            if self._ws is None or self._ws.numel() < nbytes:
                il_set_workspace(self._h, 0, 0)
                self._ws = None
                self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            il_set_workspace(self._h, self._ws.data_ptr(), self._ws.numel())
        return self._ws.numel()

    def set_variant(self, variant: int) -> None:
        """One of the IL_VARIANT_* constants (see il_set_variant in the C header)."""
        il_set_variant(self._h, variant)

    def kernel_name(self) -> str:
        return il_kernel_name(self._h)

    def set_test_knob(self, knob: int, value: int) -> None:
        """Test hook (IL_KNOB_*); invalidates a workspace reserved earlier."""
        il_set_workspace(self._h, 0, 0)
        self._ws = None
        il_set_test_knob(self._h, knob, value)

    def use_current_stream(self) -> None:
        il_set_stream(self._h, self._torch.cuda.current_stream(self.device).cuda_stream)

    def estimate(self, configs: np.ndarray, slo_us: int):
        """Host arrays in and out (copies happen inside the library call)."""
        return il_estimate(self._h, configs, slo_us)

    def estimate_device(self, d_configs, slo_us: int, out_p99=None, out_miss=None):
        """torch uint8 tensor [n][S][4] on the device in, int64 tensors out."""
        torch = self._torch
        assert d_configs.is_cuda and d_configs.dtype == torch.uint8 and d_configs.is_contiguous()
        assert d_configs.dim() == 3 and d_configs.shape[1] == self.n_stages and d_configs.shape[2] == 4
        n = d_configs.shape[0]
        if out_p99 is None:
            out_p99 = torch.empty(n, dtype=torch.int64, device=d_configs.device)
        if out_miss is None:
            out_miss = torch.empty(n, dtype=torch.int64, device=d_configs.device)
        il_estimate_device(self._h, d_configs.data_ptr(), n, slo_us, out_p99.data_ptr(),
                           out_miss.data_ptr())
        return out_p99, out_miss

    def feasible(self, configs: np.ndarray, slo_us: int) -> np.ndarray:
        """Host arrays in and out: True where the candidate meets the objective at P99."""
        return il_feasible(self._h, configs, slo_us)

    def feasible_device(self, d_configs, slo_us: int, out=None):
        """torch uint8 tensor [n][S][4] on the device in, uint8 tensor [n] out (1 = feasible)."""
        torch = self._torch
        assert d_configs.is_cuda and d_configs.dtype == torch.uint8 and d_configs.is_contiguous()
        assert d_configs.dim() == 3 and d_configs.shape[1] == self.n_stages and d_configs.shape[2] == 4
        n = d_configs.shape[0]
        if out is None:
            out = torch.empty(n, dtype=torch.uint8, device=d_configs.device)
        il_feasible_device(self._h, d_configs.data_ptr(), n, slo_us, out.data_ptr())
        return out

    def latencies(self, config: np.ndarray):
        """Per-query latencies (int64 numpy array, trace order) of one candidate [S][4]."""
        torch = self._torch
        cfg = torch.from_numpy(np.ascontiguousarray(config, dtype=np.uint8).reshape(self.n_stages, 4)).to(self.device)
        out = torch.empty(self.n_queries, dtype=torch.int64, device=self.device)
        il_estimate_latencies(self._h, cfg.data_ptr(), out.data_ptr())
        return out.cpu().numpy()

    def traffic_envelope(self, window_us) -> np.ndarray:
        """Largest number of arrivals in any window of each given length (microseconds)."""
        return il_traffic_envelope(self._h, window_us)

    def stats(self) -> dict:
        return il_get_stats(self._h)
