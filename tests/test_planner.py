"""The Planner (Section 4.3, Algorithms 1 and 2) on top of the Estimator.

CPU tests drive it with the oracle as the estimator and check the two
guarantees the paper states for the point of termination; the GPU test checks
that the CUDA Estimator leads to the very same plan, step by step."""
import numpy as np
import pytest

import workloads
from paper_1812_01776_b200.planner import Planner


def small_workload():
    # 3-stage chain, 2 hardware types: hw 0 accelerator-like (fast, dear), hw 1 CPU-like (slow, cheap)
    w = workloads.random_small(7, S=3, H=2, Bmax=8, n=1500, C=1, qps=150.0, cv=2.0)
    b = np.arange(1, 9)
    lat = np.zeros((3, 2, 8), np.int32)
    for s, (a0, c0, a1, c1) in enumerate([(4000, 300, 2500, 2600), (9000, 500, 7000, 6500), (3000, 200, 1500, 1800)]):
        lat[s, 0] = a0 + c0 * b
        lat[s, 1] = a1 + c1 * b
    w.latency_us = lat
    return w, np.array([0.70, 0.05])


def oracle_fn(oracle, w, slo):
    return lambda cfgs: oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                             w.arrival_us, w.branch_bits, cfgs, slo)


def test_planner_guarantees_with_the_oracle(oracle):
    w, prices = small_workload()
    slo = 60_000
    visits = w.visits_per_stage()
    pl = Planner(w.parent, w.latency_us, visits, prices, slo, oracle_fn(oracle, w, slo))
    res = pl.minimize_cost()
    assert res.feasible and res.config is not None
    p99, _ = oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                  w.branch_bits, res.config[None], slo)
    assert p99[0] == res.p99_us <= slo
    assert res.cost == pytest.approx(pl.cost(res.config))
    # guarantee 2: no single action reduces the cost without violating the objective
    for new in pl.single_actions(res.config):
        p, _ = oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                    w.branch_bits, new[None], slo)
        assert not (p[0] <= slo and pl.cost(new) < res.cost - 1e-12)
    # the plan is cheaper than the initial feasible configuration, and many questions went out in few calls
    assert res.candidates_evaluated > 20 * res.estimator_calls or res.estimator_calls < 40
    assert any("downgrade" in s or "remove" in s for s in res.steps)


def test_planner_infeasible_objective(oracle):
    w, prices = small_workload()
    slo = 9_000          # below the service time 4300 + 7500... of the fastest hardware
    pl = Planner(w.parent, w.latency_us, w.visits_per_stage(), prices, slo, oracle_fn(oracle, w, slo))
    assert pl.service_time(np.array([[pl.best_hardware(s), 1, 1, 0] for s in range(3)], np.uint8)) > slo
    res = pl.minimize_cost()
    assert not res.feasible and res.config is None and res.estimator_calls == 0


def test_planner_finds_a_plan_whenever_one_exists(oracle):
    """Guarantee 1 on a space small enough to enumerate: 2 stages, replicas 1..6,
    batches {1,2,4}: whenever ANY configuration is feasible, the Planner returns one."""
    w = workloads.random_small(11, S=2, H=2, Bmax=4, n=600, C=1, qps=120.0, cv=1.0)
    b = np.arange(1, 5)
    w.latency_us = np.stack([np.stack([5000 + 400 * b, 3000 + 3500 * b]),
                             np.stack([8000 + 600 * b, 6000 + 7000 * b])]).astype(np.int32)
    prices = np.array([1.0, 0.1])
    grid = np.array([[[h0, b0, r0, 0], [h1, b1, r1, 0]]
                     for h0 in range(2) for b0 in (1, 2, 4) for r0 in range(1, 7)
                     for h1 in range(2) for b1 in (1, 2, 4) for r1 in range(1, 7)], np.uint8)
    for slo in (14_000, 20_000, 45_000):
        p99, _ = oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                      w.branch_bits, grid, slo)
        exists = bool((p99 <= slo).any())
        pl = Planner(w.parent, w.latency_us, w.visits_per_stage(), prices, slo, oracle_fn(oracle, w, slo))
        res = pl.minimize_cost()
        if exists:
            assert res.feasible, slo
        if res.feasible:
            assert res.p99_us <= slo


def test_tuner_handoff_with_the_oracle(oracle):
    from paper_1812_01776_b200.planner import tuner_handoff, envelope_windows
    w, prices = small_workload()
    slo = 60_000
    pl = Planner(w.parent, w.latency_us, w.visits_per_stage(), prices, slo, oracle_fn(oracle, w, slo))
    res = pl.minimize_cost()
    span = int(w.arrival_us[-1] - w.arrival_us[0])
    h = tuner_handoff(pl, res.config, w.n_queries, span, lambda wins: oracle.traffic_envelope(w.arrival_us, wins))
    assert h["window_us"][0] == pl.service_time(res.config) and h["window_us"][-1] == 60_000_000
    assert np.all(np.diff(h["window_us"]) > 0) and np.all(np.diff(h["max_count"]) >= 0)
    assert h["max_count"][-1] == w.n_queries            # the 10 s trace fits in the 60 s window
    assert np.all(h["rho"] > 0) and np.all(h["rho"] < 1)   # a feasible plan keeps every model below saturation
    assert np.array_equal(envelope_windows(1000)[:3], [1000, 2000, 4000])


def tree_workload():
    # 5-stage tree: 0 -> {1 (bit 0 = 0), 2 (bit 0 = 1)}; 1 -> 3; 2 -> 4 guarded by bit 1 (a cascade)
    w = workloads.random_small(21, S=5, H=3, Bmax=16, n=1200, C=1, qps=180.0, cv=2.0, tree=True)
    w.parent = np.array([-1, 0, 0, 1, 2], np.int32)
    w.cond_bit = np.array([-1, 0, 0, -1, 1], np.int8)
    w.cond_val = np.array([0, 0, 1, 0, 1], np.uint8)
    b = np.arange(1, 17)
    lat = np.zeros((5, 3, 16), np.int32)
    rng = np.random.default_rng(5)
    for s in range(5):
        a0, c0 = rng.integers(3000, 9000), rng.integers(150, 500)
        lat[s, 0] = a0 + c0 * b                       # accelerator-like
        lat[s, 1] = a0 * 1.3 + c0 * 3 * b             # mid
        lat[s, 2] = a0 * 0.6 + c0 * 12 * b            # CPU-like
    w.latency_us = lat
    return w, np.array([0.90, 0.40, 0.06])


def two_stage_workload():
    w = workloads.random_small(11, S=2, H=2, Bmax=4, n=600, C=1, qps=120.0, cv=1.0)
    b = np.arange(1, 5)
    w.latency_us = np.stack([np.stack([5000 + 400 * b, 3000 + 3500 * b]),
                             np.stack([8000 + 600 * b, 6000 + 7000 * b])]).astype(np.int32)
    return w, np.array([1.0, 0.1])


@pytest.mark.parametrize("make,slo", [(small_workload, 60_000), (small_workload, 35_000), (tree_workload, 80_000),
                                      (tree_workload, 40_000), (two_stage_workload, 20_000),
                                      (two_stage_workload, 45_000), (small_workload, 9_000)])
def test_batched_planner_equals_the_sequential_algorithms(oracle, make, slo):
    """The Planner batches its questions; Algorithms 1 and 2 written out in the paper's listing
    order, asking one Feasible question at a time (oracle/planner_sequential.py), must reach the
    same plan through the same sequence of accepted actions."""
    from oracle.planner_sequential import SequentialPlanner
    w, prices = make()
    visits = w.visits_per_stage()

    def feasible_one(cfg):
        p99, _, = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                      w.branch_bits, cfg, slo)
        return p99 <= slo

    seq = SequentialPlanner(w.parent, w.latency_us, visits, prices, slo, feasible_one)
    want = seq.minimize_cost()
    got = Planner(w.parent, w.latency_us, visits, prices, slo, oracle_fn(oracle, w, slo)).minimize_cost()
    assert got.feasible == (want is not None)
    if want is not None:
        assert np.array_equal(got.config, want)
        assert len(got.trajectory) == len(seq.trajectory)
        for a, b_ in zip(got.trajectory, seq.trajectory):
            assert np.array_equal(a, b_)
        assert got.cost == pytest.approx(seq.cost(want))
        # one question at a time costs many more estimator calls than the batched Planner makes
        assert seq.questions >= got.estimator_calls


def test_tuner_handoff_on_a_hand_computed_case():
    """Section 5, initialisation: rho_m = lambda * s_m / (k_m * mu_m), mu_m the throughput of one
    replica at the planned batch size.  Two models: the trace has 1,001 arrivals over 10 s
    (lambda = 100.1 per second); model 0 sees every query, model 1 a quarter of them.
    Model 0: batch 4 takes 20 ms -> mu = 200 per second, 2 replicas -> rho = 100.1 / 400 = 0.25025.
    Model 1: batch 1 takes 8 ms  -> mu = 125 per second, 1 replica -> rho = 25.025 / 125 = 0.2002."""
    from paper_1812_01776_b200.planner import tuner_handoff
    lat = np.zeros((2, 1, 4), np.int32)
    lat[0, 0] = [9_000, 12_000, 16_000, 20_000]
    lat[1, 0] = [8_000, 9_000, 10_000, 11_000]
    pl = Planner(np.array([-1, 0]), lat, np.array([1001, 250]), [1.0], 100_000, lambda c: None)
    cfg = np.array([[0, 4, 2, 0], [0, 1, 1, 0]], np.uint8)
    seen = {}

    def env(windows):
        seen["w"] = windows
        return np.arange(1, len(windows) + 1)
    h = tuner_handoff(pl, cfg, 1001, 10_000_000, env)
    assert seen["w"][0] == 9_000 + 8_000                      # service time: batch-1 latencies along the path
    assert h["mu_per_us"] == pytest.approx([200e-6, 125e-6])
    assert h["scale_factor"] == pytest.approx([1.0, 250 / 1001])
    assert h["rho"] == pytest.approx([0.25025, 100.1 * (250 / 1001) / 125])
    assert h["rho"][1] == pytest.approx(0.2)                  # 25 queries per second over 125


@pytest.mark.gpu
def test_planner_same_plan_on_gpu_and_oracle(oracle):
    import torch
    import paper_1812_01776_b200 as il
    assert torch.cuda.is_available()
    w, prices = small_workload()
    slo = 60_000
    visits = w.visits_per_stage()
    ref = Planner(w.parent, w.latency_us, visits, prices, slo, oracle_fn(oracle, w, slo)).minimize_cost()
    with il.Estimator.from_workload(w) as est:
        assert np.array_equal(est.visits, visits)
        got = Planner(w.parent, w.latency_us, est.visits, prices, slo,
                      lambda cfgs: est.estimate(cfgs, slo)).minimize_cost()
        # and with the feasibility-only entry point answering the search's questions
        fea = Planner(w.parent, w.latency_us, est.visits, prices, slo,
                      lambda cfgs: est.estimate(cfgs, slo), feasible=lambda cfgs: est.feasible(cfgs, slo)).minimize_cost()
    for res in (got, fea):
        assert res.feasible == ref.feasible
        assert np.array_equal(res.config, ref.config)
        assert res.cost == ref.cost and res.p99_us == ref.p99_us and res.steps == ref.steps


@pytest.mark.gpu
def test_planner_on_the_image_pipeline(oracle):
    """Planning on workload 2's trace and tables (4 stages, 50,000 queries): the
    plan is feasible and locally optimal according to the oracle."""
    import paper_1812_01776_b200 as il
    w = workloads.make(2, n_candidates=1)
    prices = np.array([0.90, 0.35, 0.10])
    with il.Estimator.from_workload(w) as est:
        pl = Planner(w.parent, w.latency_us, est.visits, prices, w.slo_us,
                     lambda cfgs: est.estimate(cfgs, w.slo_us))
        res = pl.minimize_cost()
    assert res.feasible
    p99, _ = oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                  w.branch_bits, res.config[None], w.slo_us)
    assert p99[0] == res.p99_us <= w.slo_us
    # removing any single replica must break the objective (checked with the oracle)
    for s in range(4):
        if res.config[s, 2] > 1:
            new = res.config.copy(); new[s, 2] -= 1
            p, _ = oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                        w.branch_bits, new[None], w.slo_us)
            assert p[0] > w.slo_us
