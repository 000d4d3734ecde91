"""il_estimate_device_static is the estimate call for processes that may not
allocate GPU memory once they are serving (their device memory belongs to a
model server's pool, and a cudaMalloc would fail or stall the GPU): its scratch
is a static array inside the library.  It must give exactly what
il_estimate_device gives -- and what the oracle gives -- also when called twice
in a row on different candidates, since the shared array still holds the first
call's data; and the amount of free device memory must not move across a call."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu


def _static(il, est, d_cfg, slo):
    import torch
    n = d_cfg.shape[0]
    p99 = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    miss = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    il.il_estimate_device_static(est._h, d_cfg.data_ptr(), n, slo, p99.data_ptr(), miss.data_ptr())
    return p99, miss


def test_static_scratch_matches_regular_entry_point_twice(oracle):
    import torch
    import paper_1812_01776_b200 as il
    from paper_1812_01776_b200 import estimator as E
    assert torch.cuda.is_available()
    w = workloads.make(3, n_queries=3000, n_candidates=96)
    exp_p99, exp_miss = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        for lo, hi in [(0, 64), (40, 96)]:       # two calls in a row, different candidates
            d_cfg = torch.from_numpy(np.ascontiguousarray(w.configs[lo:hi])).cuda()
            ref_p99, ref_miss = est.estimate_device(d_cfg, w.slo_us)
            p99, miss = _static(il, est, d_cfg, w.slo_us)
            assert torch.equal(p99, ref_p99)      # integers: bit-exact, as in the parity tests
            assert torch.equal(miss, ref_miss)
            assert np.array_equal(p99.cpu().numpy(), exp_p99[lo:hi])
            assert np.array_equal(miss.cpu().numpy(), exp_miss[lo:hi])
        # a batch whose latency slab alone exceeds the static array is refused, nothing runs
        n_big = E.IL_STATIC_SCRATCH_BYTES // (8 * 3008) + 1
        big = torch.zeros((n_big, w.n_stages, 4), dtype=torch.uint8, device="cuda")
        out = torch.zeros(n_big, dtype=torch.int64, device="cuda")
        with pytest.raises(E.ILError) as ei:
            il.il_estimate_device_static(est._h, big.data_ptr(), n_big, w.slo_us,
                                         out.data_ptr(), out.data_ptr())
        assert ei.value.code == E.IL_ERR_TOO_LARGE


@pytest.mark.parametrize("variant", [0, 1, 2], ids=["auto", "wide", "staged"])
def test_static_scratch_allocates_nothing_and_matches_the_oracle(oracle, variant):
    """On a handle that never ran the allocating entry point: free device memory is the same
    before and after a call (after one start-up call that resolves the array's address), on
    each kernel the entry point can take, with a candidate count that fills no whole CTA."""
    import torch
    import paper_1812_01776_b200 as il
    w = workloads.make(5, n_queries=2500, n_candidates=61)
    exp_p99, exp_miss = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        d_cfg = torch.from_numpy(w.configs).cuda()
        _static(il, est, d_cfg[:5], w.slo_us)                 # start-up call
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        p99 = torch.full((61,), -1, dtype=torch.int64, device="cuda")
        miss = torch.full((61,), -1, dtype=torch.int64, device="cuda")
        free_mid, _ = torch.cuda.mem_get_info()
        for _ in range(2):
            il.il_estimate_device_static(est._h, d_cfg.data_ptr(), 61, w.slo_us, p99.data_ptr(),
                                         miss.data_ptr())
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_mid <= free_before
        assert np.array_equal(p99.cpu().numpy(), exp_p99)
        assert np.array_equal(miss.cpu().numpy(), exp_miss)


def test_static_scratch_with_times_too_large_to_pack(oracle):
    """Stamps near 2^58 force the kernel with separate time and query streams (12 bytes per
    stream element of the static array instead of 8)."""
    import torch
    import paper_1812_01776_b200 as il
    w = workloads.make(2, n_queries=2000, n_candidates=30)
    exp_p99, exp_miss = oracle.estimate_workload(w)
    w.arrival_us = w.arrival_us + (1 << 58)
    with il.Estimator.from_workload(w) as est:
        assert est.kernel_name() == "des_kernel"
        d_cfg = torch.from_numpy(w.configs).cuda()
        for _ in range(2):
            p99, miss = _static(il, est, d_cfg, w.slo_us)
            assert np.array_equal(p99.cpu().numpy(), exp_p99)
            assert np.array_equal(miss.cpu().numpy(), exp_miss)
