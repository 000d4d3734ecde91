"""Shared-prefix evaluation: candidates that agree on the configurations of all stages on a path
from the root share the simulation of that path.  Results must be the integers the oracle gives,
whatever the amount of sharing."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu

KNOB_SHARE = 3


@pytest.fixture(scope="module")
def il():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1812_01776_b200 as il_
    il_.load_library()
    return il_


def product_configs(rng, S, H, Bmax, max_replicas, per_stage):
    """Full product of a few choices per stage (stage 0 varies fastest)."""
    choices = []
    for s in range(S):
        c = np.zeros((per_stage[s], 4), np.uint8)
        c[:, 0] = rng.integers(0, H, per_stage[s])
        c[:, 1] = rng.integers(1, Bmax + 1, per_stage[s])
        c[:, 2] = rng.integers(1, max_replicas + 1, per_stage[s])
        choices.append(c)
    total = int(np.prod(per_stage))
    idx = np.arange(total)
    cfg = np.zeros((total, S, 4), np.uint8)
    for s in range(S):
        cfg[:, s] = choices[s][idx % per_stage[s]]
        idx = idx // per_stage[s]
    return cfg


@pytest.mark.parametrize("mode", [1, 3], ids=["covering-candidates", "node-by-node"])
@pytest.mark.parametrize("seed", range(10))
def test_forced_sharing_on_random_pipelines(il, oracle, seed, mode):
    """Random chains and trees (cascades included), candidate sets with a lot of sharing (products of
    2-3 choices per stage) and with hardly any (independent draws), equal stamps, R up to 32; the nodes
    simulated by the lane kernel through a covering set of candidates, and one by one."""
    S = 1 + seed % 6
    w = workloads.random_small(seed, S=S, H=3, Bmax=[4, 33, 64][seed % 3], n=700 + 37 * seed, C=24,
                               max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1), qps=400.0, cv=3.0,
                               lat_lo=1, lat_hi=20000, equal_stamp_every=(3 if seed % 4 == 0 else 0))
    rng = np.random.default_rng(seed)
    prod = product_configs(rng, S, 3, w.max_batch, [3, 8, 32][seed % 3], [3, 2, 2, 2, 2, 2][:S])
    w.configs = np.ascontiguousarray(np.concatenate([prod, w.configs, prod[:5]]))
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_test_knob(KNOB_SHARE, mode)
        p99, miss = est.estimate(w.configs, w.slo_us)
        st = est.stats()
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1]), np.nonzero(p99 != exp[0])[0][:5]
        assert st["stage_runs"] < w.n_candidates * S and st["candidates"] == w.n_candidates
        if mode == 1:
            assert st["stage_runs"] % S == 0          # whole candidates
        assert np.array_equal(est.feasible(w.configs, w.slo_us), exp[0] <= w.slo_us)
        est.set_test_knob(KNOB_SHARE, 2)
        p99, miss = est.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and est.stats()["stage_runs"] == w.n_candidates * S


def test_sharing_is_chosen_for_a_product_sweep(il, oracle, oracle_pool):
    """Workload 5's candidate set is a product of per-stage choices: 4,096 candidates (the first three
    stages vary) on a 4,097-query trace have 8 + 64 + 64 + 512 + ... nodes, far fewer than candidates x
    stages, so the library takes the shared path by itself; a uniform draw (workload 3) does not."""
    import torch
    w = workloads.make(5, n_queries=4097, n_candidates=4096)
    exp = oracle.estimate_many_parallel(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                        w.branch_bits, w.configs, w.slo_us, pool=oracle_pool)
    with il.Estimator.from_workload(w) as est:
        est.reserve_workspace(w.n_candidates)
        a, b = est.estimate_device(torch.from_numpy(w.configs).cuda(), w.slo_us)
        st = est.stats()
        assert np.array_equal(a.cpu().numpy(), exp[0]) and np.array_equal(b.cpu().numpy(), exp[1])
        assert st["stage_runs"] * 4 <= w.n_candidates * w.n_stages
        est.set_test_knob(KNOB_SHARE, 3)              # the same nodes one by one
        a, b = est.estimate_device(torch.from_numpy(w.configs).cuda(), w.slo_us)
        assert np.array_equal(a.cpu().numpy(), exp[0]) and np.array_equal(b.cpu().numpy(), exp[1])
        assert est.stats()["stage_runs"] == 8 + 64 + 64 + 512 + 3 * 64 + 512
        est.set_test_knob(KNOB_SHARE, 0)
        got = est.feasible_device(torch.from_numpy(w.configs).cuda(), w.slo_us).cpu().numpy().astype(bool)
        assert np.array_equal(got, exp[0] <= w.slo_us)
    w = workloads.make(3, n_queries=3000, n_candidates=2500)
    with il.Estimator.from_workload(w) as est:
        est.estimate(w.configs, w.slo_us)
        assert est.stats()["stage_runs"] == w.n_candidates * w.n_stages


def test_sharing_with_latencies_above_2_32_and_one_query(il, oracle):
    w = workloads.random_small(102, S=2, H=1, Bmax=2, n=3000, C=4, max_replicas=1,
                               lat_lo=2_000_000_000, lat_hi=2_100_000_000)
    exp = oracle.estimate_workload(w)
    assert exp[0].max() > 2 ** 32
    with il.Estimator.from_workload(w) as est:
        est.set_test_knob(KNOB_SHARE, 1)
        p99, miss = est.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])
    w = workloads.random_small(100, S=1, H=1, Bmax=1, n=1, C=3, max_replicas=1)
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_test_knob(KNOB_SHARE, 1)
        p99, miss = est.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])


def test_sharing_rejects_bad_candidates(il):
    from paper_1812_01776_b200 import estimator as E
    import torch
    w = workloads.make(1, n_candidates=8)
    with il.Estimator.from_workload(w) as est:
        est.set_test_knob(KNOB_SHARE, 1)
        bad = w.configs.copy()
        bad[5, 1, 1] = 17
        with pytest.raises(E.ILError) as ei:
            est.estimate_device(torch.from_numpy(bad).cuda(), w.slo_us)
        assert ei.value.code == E.IL_ERR_BAD_CONFIG
        p99, _ = est.estimate(w.configs, w.slo_us)
        assert (p99 > 0).all()
