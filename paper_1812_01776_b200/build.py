"""Builds libil_estimator.so in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libil_estimator.so")
LIB_CHECKED = os.path.join(HERE, "libil_estimator_checked.so")     # the same sources with -DIL_CHECKED
SOURCES = ["des_kernel.cu", "des_packed_kernel.cu", "des_lane_kernel.cu", "select_kernel.cu", "order_kernel.cu", "envelope_kernel.cu", "prefix_kernel.cu", "il_api.cu", "il_static.cu"]
HEADERS = [os.path.join(CSRC, "il_internal.h"), os.path.join(ROOT, "include", "il_estimator.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the CUDA sources into the shared library (no GPU needed).  checked: the variant
    whose kernels compare every computed index with its array size and record IL_ERR_BOUNDS
    instead of making the access."""
    lib = LIB_CHECKED if checked else LIB
    if force or is_stale(lib):
        tmp = lib + f".tmp{os.getpid()}"
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + (["-DIL_CHECKED"] if checked else []) + \
              ["-I" + os.path.join(ROOT, "include"), "-I" + CSRC, "-o", tmp] + \
              [os.path.join(CSRC, s) for s in SOURCES]
        subprocess.check_call(cmd)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, checked=True))
