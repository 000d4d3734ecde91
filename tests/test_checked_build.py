"""The bounds-checked build (-DIL_CHECKED): the same kernels with every computed index into a stream,
ring, slab or bound input compared with its array size; an index outside is recorded as IL_ERR_BOUNDS
and the access skipped.  A slice of the parity tests runs against it in a process of its own (the
library is chosen when the binding is first loaded): any wrong index would turn into that error code."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_checked_library_builds_and_exports_the_same_symbols():
    import ctypes
    from paper_1812_01776_b200 import build, estimator
    lib = ctypes.CDLL(build.build(checked=True))
    for name in estimator.EXPORTS:
        assert hasattr(lib, name), name
    lib.il_strerror.restype = ctypes.c_char_p
    assert b"checked build" in lib.il_strerror(estimator.IL_ERR_BOUNDS)


@pytest.mark.gpu
def test_parity_slice_on_the_checked_build():
    from paper_1812_01776_b200 import build
    build.build(checked=True)
    env = dict(os.environ, IL_ESTIMATOR_CHECKED="1")
    probe = subprocess.run([sys.executable, "-c",
                            "import paper_1812_01776_b200 as il; print(il.library_path())"],
                           cwd=ROOT, env=env, capture_output=True, text=True)
    assert "libil_estimator_checked.so" in probe.stdout, probe.stdout + probe.stderr
    run = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_shared_prefix.py",
                          "tests/test_feasible.py", "tests/test_join.py", "-m", "gpu", "-x", "-q", "-k",
                          "random_small or deep_pipelines or edge_cases or short_stream_rings or forced_sharing "
                          "or feasible_random_small or largest_table or join_parity or join_equal_instants"],
                         cwd=ROOT, env=env, capture_output=True, text=True)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-2000:]
