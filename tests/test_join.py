"""Joins (Section 2: a pipeline is a DAG of dataflow edges; a model may consume two models' outputs):
a query enters the join's queue when the last incoming edge it follows has delivered it.  CUDA path
against the oracle through every entry point, on the three shapes of workloads.join_small."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu

SHAPES = ["diamond", "guarded", "two_joins", "skip"]


@pytest.fixture(scope="module")
def il():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1812_01776_b200 as il_
    il_.load_library()
    return il_


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("seed", range(6))
def test_join_parity(il, oracle, seed, shape):
    w = workloads.join_small(seed, n=900 + 41 * seed, C=30, max_replicas=[3, 8, 32][seed % 3],
                             Bmax=[4, 33, 64][seed % 3], shape=shape)
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(seed % 5)          # whatever is asked for, a join runs on the kernel that merges streams
        assert est.kernel_name() == "des_kernel"
        p99, miss = est.estimate(w.configs, w.slo_us)
        st = est.stats()
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1]), np.nonzero(p99 != exp[0])[0][:5]
        assert st["query_events"] == w.n_candidates * int(est.visits.sum())
        assert np.array_equal(est.feasible(w.configs, w.slo_us), exp[0] <= w.slo_us)


@pytest.mark.parametrize("shape", SHAPES)
def test_join_equal_instants(il, oracle, shape):
    """Tiny service times and runs of equal arrival stamps: many queries become ready at a join in the
    same instant, from both sides, so the order rule (first parent's deliveries, then the second's)
    decides who shares a batch."""
    for seed in (0, 2, 4):
        w = workloads.join_small(seed, n=1200, C=24, max_replicas=3, Bmax=4, tiny_times=True, shape=shape)
        exp = oracle.estimate_workload(w)
        with il.Estimator.from_workload(w) as est:
            p99, miss = est.estimate(w.configs, w.slo_us)
            assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1]), seed
            for c in range(3):
                _, _, lat = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                                w.branch_bits, w.configs[c], w.slo_us, want_latency=True,
                                                join=w.join)
                assert np.array_equal(est.latencies(w.configs[c]), lat), (seed, c)


def test_join_edges_nobody_follows(il, oracle):
    """A join one of whose incoming streams is empty (no query has the bit that opens the edge), and one
    that no query reaches at all."""
    w = workloads.join_small(8, n=800, C=12, shape="guarded")
    w.branch_bits[:] &= 0xFE                       # nobody visits stage 2: the join has one input
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        assert est.visits.tolist() == [800, 800, 0, 800, 800]
        p99, miss = est.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])
    w = workloads.join_small(8, n=800, C=12, shape="two_joins")
    w.cond_bit = np.array([-1, 0, 0, -1, 1, -1], np.int8)      # bit 0 decides between 1 and 2 ...
    w.cond_val = np.array([0, 0, 1, 0, 1, 0], np.uint8)
    w.branch_bits[:] |= 1                          # ... and everyone takes 2: stages 1 and 4 stay empty
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        assert est.visits.tolist() == [800, 0, 800, 800, 0, 800]
        p99, miss = est.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])


def test_join_hand_trace_and_visits(il):
    w = workloads.join_small(3, n=400, shape="guarded")
    with il.Estimator.from_workload(w) as est:
        odd = int((w.branch_bits & 1).sum())
        assert est.visits.tolist() == [400, 400, odd, 400, 400]     # the join is visited once per query


def test_join_device_entry_chunks_and_static(il, oracle):
    """A longer trace in several chunks through the device entry point, and the allocation-free entry
    point on the same handle."""
    import torch
    w = workloads.join_small(7, n=5000, C=64, shape="two_joins")
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        lo = il.il_workspace_min_bytes(est._h)
        est.reserve_workspace(w.n_candidates, max_bytes=lo + 24 * 5024 * 8)
        d = torch.from_numpy(w.configs).cuda()
        a, b = est.estimate_device(d, w.slo_us)
        assert est.stats()["chunks"] > 1
        assert np.array_equal(a.cpu().numpy(), exp[0]) and np.array_equal(b.cpu().numpy(), exp[1])
        p99 = torch.full((64,), -1, dtype=torch.int64, device="cuda")
        miss = torch.full((64,), -1, dtype=torch.int64, device="cuda")
        il.il_estimate_device_static(est._h, d.data_ptr(), 64, w.slo_us, p99.data_ptr(), miss.data_ptr())
        assert np.array_equal(p99.cpu().numpy(), exp[0]) and np.array_equal(miss.cpu().numpy(), exp[1])
