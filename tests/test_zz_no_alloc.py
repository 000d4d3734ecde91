"""il_estimate_device_static is the estimate call for processes that may not
allocate GPU memory once they are serving (their device memory belongs to a
model server's pool, and a cudaMalloc would fail or stall the GPU): its scratch
is a static array inside the library.  It must give exactly what
il_estimate_device gives, also when called twice in a row on different
candidates, since the shared array still holds the first call's data."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_regular_entry_point_twice():
    import torch
    import paper_1812_01776_b200 as il
    from paper_1812_01776_b200 import estimator as E
    assert torch.cuda.is_available()
    w = workloads.make(3, n_queries=3000, n_candidates=96)
    with il.Estimator.from_workload(w) as est:
        for lo, hi in [(0, 64), (40, 96)]:       # two calls in a row, different candidates
            d_cfg = torch.from_numpy(np.ascontiguousarray(w.configs[lo:hi])).cuda()
            ref_p99, ref_miss = est.estimate_device(d_cfg, w.slo_us)
            p99 = torch.full((hi - lo,), -1, dtype=torch.int64, device="cuda")
            miss = torch.full((hi - lo,), -1, dtype=torch.int64, device="cuda")
            il.il_estimate_device_static(est._h, d_cfg.data_ptr(), hi - lo, w.slo_us,
                                         p99.data_ptr(), miss.data_ptr())
            assert torch.equal(p99, ref_p99)      # integers: bit-exact, as in the parity tests
            assert torch.equal(miss, ref_miss)
        # a batch whose latency slab alone exceeds the static array is refused, nothing runs
        n_big = E.IL_STATIC_SCRATCH_BYTES // (8 * 3008) + 1
        big = torch.zeros((n_big, w.n_stages, 4), dtype=torch.uint8, device="cuda")
        out = torch.zeros(n_big, dtype=torch.int64, device="cuda")
        with pytest.raises(E.ILError) as ei:
            il.il_estimate_device_static(est._h, big.data_ptr(), n_big, w.slo_us,
                                         out.data_ptr(), out.data_ptr())
        assert ei.value.code == E.IL_ERR_TOO_LARGE
