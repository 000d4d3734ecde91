"""Fan-out (Section 2: a pipeline is a DAG of dataflow edges; parallel branches): a query goes down
every edge whose condition holds and is answered when its last copy leaves.  CUDA path against the
oracle on both kernels that implement it, through every entry point."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def il():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1812_01776_b200 as il_
    il_.load_library()
    return il_


@pytest.mark.parametrize("variant", [0, 1, 4], ids=["auto", "wide", "packed-request"])
@pytest.mark.parametrize("seed", range(8))
def test_fan_out_parity(il, oracle, seed, variant):
    w = workloads.fan_out_small(seed, n=900 + 41 * seed, C=30, max_replicas=[3, 8, 32][seed % 3],
                                Bmax=[4, 33, 64][seed % 3])
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        # the warp-per-candidate kernel with packed records has no fan-out: the request falls back
        assert est.kernel_name() == ("des_lane_kernel" if variant == 0 else "des_kernel")
        p99, miss = est.estimate(w.configs, w.slo_us)
        st = est.stats()
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1]), np.nonzero(p99 != exp[0])[0][:5]
        assert st["query_events"] == w.n_candidates * w.query_events()
        assert np.array_equal(est.feasible(w.configs, w.slo_us), exp[0] <= w.slo_us)


@pytest.mark.parametrize("variant", [0, 1], ids=["auto", "wide"])
def test_fan_out_per_query_latencies(il, oracle, variant):
    w = workloads.fan_out_small(21, n=1500, C=5)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        for c in range(w.n_candidates):
            _, _, exp = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                            w.branch_bits, w.configs[c], w.slo_us, want_latency=True)
            assert np.array_equal(est.latencies(w.configs[c]), exp), c


def test_fan_out_other_shapes_and_entry_points(il, oracle):
    """Two conditional edges on different bits (a query may take none, one or both), a long trace in
    several chunks, forced sharing (which must step aside), and the allocation-free entry point."""
    import torch
    w = workloads.fan_out_small(5, n=6000, C=64)
    w.parent = np.array([-1, 0, 0, 1, 1, 2], np.int32)
    w.cond_bit = np.array([-1, 0, 1, -1, 1, -1], np.int8)
    w.cond_val = np.array([0, 1, 0, 0, 1, 0], np.uint8)
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_test_knob(3, 1)
        lo = il.il_workspace_min_bytes(est._h)
        est.reserve_workspace(w.n_candidates, max_bytes=lo + 24 * 6016 * 8)
        d = torch.from_numpy(w.configs).cuda()
        a, b = est.estimate_device(d, w.slo_us)
        assert est.stats()["chunks"] > 1
        assert np.array_equal(a.cpu().numpy(), exp[0]) and np.array_equal(b.cpu().numpy(), exp[1])
        p99 = torch.full((64,), -1, dtype=torch.int64, device="cuda")
        miss = torch.full((64,), -1, dtype=torch.int64, device="cuda")
        il.il_estimate_device_static(est._h, d.data_ptr(), 64, w.slo_us, p99.data_ptr(), miss.data_ptr())
        assert np.array_equal(p99.cpu().numpy(), exp[0]) and np.array_equal(miss.cpu().numpy(), exp[1])
