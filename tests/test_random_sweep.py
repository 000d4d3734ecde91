"""Randomised differential sweep: a few hundred seeded draws over everything that can vary -- topology (chains,
trees, fan-out, joins), table sizes, replica limits, trace lengths from 1, tiny service times with runs of equal
stamps, duplicate candidates, objectives at both extremes, every kernel variant, short stream rings, every setting
of prefix sharing, branch bits inside the stream records or looked up, host and device entry points -- each compared with the oracle on P99, misses, feasibility and
(for a quarter of them) the per-query latencies.  Sweeps of 18,655 and, with the branch-bit knob, 13,186 such draws
(seeds from 5001) ran clean on a B200; the cases here are the first few hundred of the same generator."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu


def draw(seed):
    rng = np.random.default_rng(seed)
    kind = rng.integers(0, 10)
    S = int(rng.integers(1, 9))
    Bmax = int(rng.choice([1, 2, 4, 7, 16, 33, 64]))
    R = int(rng.choice([1, 2, 3, 8, 14, 15, 16, 32]))
    n = int(rng.integers(1, 2500))
    C = int(rng.integers(1, 70))
    tiny = bool(rng.integers(0, 3) == 0)
    eq = int(rng.choice([0, 0, 2, 3, 5]))
    if kind == 8:
        w = workloads.fan_out_small(seed, n=n, C=C, max_replicas=R, Bmax=Bmax, tiny_times=tiny)
    elif kind == 9:
        w = workloads.join_small(seed, n=n, C=C, max_replicas=R, Bmax=Bmax, tiny_times=tiny,
                                 shape=str(rng.choice(["diamond", "guarded", "two_joins", "skip"])))
    else:
        w = workloads.random_small(seed, S=S, H=int(rng.integers(1, 5)), Bmax=Bmax, n=n, C=C, max_replicas=R,
                                   tree=bool(rng.integers(0, 2)),
                                   qps=(80000.0 if tiny else float(rng.choice([100, 400, 2000]))),
                                   cv=float(rng.choice([1, 2, 4])), lat_lo=1,
                                   lat_hi=(30 if tiny else int(rng.choice([200, 9000, 40000]))),
                                   equal_stamp_every=eq)
    if rng.integers(0, 4) == 0 and C > 4:      # duplicates: shared prefixes
        w.configs[C // 2:] = w.configs[: C - C // 2]
    w.slo_us = int(rng.choice([w.slo_us, 1, 10**9, int(np.median(w.latency_us)) * w.n_stages]))
    knobs = dict(variant=int(rng.integers(0, 5)), ring=int(rng.choice([0, 0, 6, 7, 9])),
                 share=int(rng.choice([0, 1, 2, 3])), host=bool(rng.integers(0, 2)),
                 per_query=bool(rng.integers(0, 4) == 0), bits_in_records=seed % 2)
    return w, knobs


@pytest.mark.parametrize("block", range(10))
def test_random_sweep(oracle, block):
    import torch
    import paper_1812_01776_b200 as il
    for seed in range(5001 + 40 * block, 5001 + 40 * (block + 1)):
        w, k = draw(seed)
        exp = oracle.estimate_workload(w)
        with il.Estimator.from_workload(w) as est:
            est.set_variant(k["variant"])
            if k["ring"]:
                est.set_test_knob(1, k["ring"])
            est.set_test_knob(3, k["share"])
            est.set_test_knob(5, k["bits_in_records"])
            if k["host"]:
                p99, miss = est.estimate(w.configs, w.slo_us)
            else:
                a, b = est.estimate_device(torch.from_numpy(w.configs).cuda(), w.slo_us)
                p99, miss = a.cpu().numpy(), b.cpu().numpy()
            assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1]), (seed, k)
            assert np.array_equal(est.feasible(w.configs, w.slo_us), exp[0] <= w.slo_us), (seed, k)
            if k["per_query"]:
                lat = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                          w.branch_bits, w.configs[0], w.slo_us, want_latency=True, join=w.join)[2]
                assert np.array_equal(est.latencies(w.configs[0]), lat), (seed, k)
