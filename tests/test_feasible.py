"""Feasibility-only mode (Section 4.3, "Feasible"): one byte per candidate, equal to
P99 <= objective as the oracle computes it, with candidates dropped early once they are decided."""
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


def _slos(exp_p99):
    """Objectives that split the candidates: quantiles of the oracle's P99 values and values next to them."""
    qs = np.quantile(exp_p99, [0.1, 0.5, 0.9]).astype(np.int64)
    return sorted({int(qs[0]), int(qs[1]), int(qs[1]) - 1, int(qs[2]), int(exp_p99.min()) - 1, int(exp_p99.max())})


@pytest.mark.parametrize("variant", [3, 4, 1], ids=["lanes", "packed", "wide"])
@pytest.mark.parametrize("seed", range(8))
def test_feasible_random_small(il, oracle, seed, variant):
    w = workloads.random_small(seed, S=1 + seed % 6, H=3, Bmax=[4, 33, 64][seed % 3], n=700 + 37 * seed,
                               C=40, max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1),
                               qps=400.0, cv=3.0, lat_lo=1, lat_hi=20000,
                               equal_stamp_every=(3 if seed % 4 == 0 else 0))
    exp_p99, _ = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        for slo in _slos(exp_p99):
            got = est.feasible(w.configs, slo)
            assert np.array_equal(got, exp_p99 <= slo), (seed, slo, np.nonzero(got != (exp_p99 <= slo))[0][:5])


@pytest.mark.parametrize("ring_log2", [6, 8])
@pytest.mark.parametrize("seed", [1, 4, 5, 8, 11])
def test_feasible_with_short_stream_rings(il, oracle, seed, ring_log2):
    """Ring overflow in feasibility mode: the candidates given up are evaluated in full by the
    warp-per-candidate kernel and their flags filled in."""
    import torch
    w = workloads.random_small(seed, S=1 + seed % 6, H=3, Bmax=[4, 33, 64][seed % 3], n=700 + 37 * seed,
                               C=40, max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1),
                               qps=400.0, cv=3.0, lat_lo=1, lat_hi=20000)
    exp_p99, _ = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(3)
        est.set_test_knob(1, ring_log2)
        d = torch.from_numpy(w.configs).cuda()
        for slo in _slos(exp_p99)[:3]:
            got = est.feasible_device(d, slo).cpu().numpy().astype(bool)
            assert np.array_equal(got, exp_p99 <= slo), (seed, slo)


@pytest.mark.parametrize("cid,n,C", [(1, None, None), (2, 5000, 300), (3, 6001, 200), (4, 3000, 150), (5, 4097, 260)])
def test_feasible_workloads_reduced(il, oracle, cid, n, C):
    w = workloads.make(cid, n_queries=n, n_candidates=C)
    exp_p99, exp_miss = oracle.estimate_workload(w)
    k = (99 * w.n_queries + 99) // 100
    with il.Estimator.from_workload(w) as est:
        got = est.feasible(w.configs, w.slo_us)
        st = est.stats()
        assert np.array_equal(got, exp_p99 <= w.slo_us)
        assert np.array_equal(got, exp_miss <= w.n_queries - k)
        assert st["candidates"] == w.n_candidates and 0 <= st["early_exits"] <= int((~got).sum())
        # extremes of the objective: nobody / everybody is feasible; negative objectives are allowed
        assert not est.feasible(w.configs, 0).any() and not est.feasible(w.configs, -5).any()
        assert est.feasible(w.configs, int(exp_p99.max())).all() and est.feasible(w.configs, 1 << 62).all()
        assert est.feasible(w.configs[:0], w.slo_us).shape == (0,)


def test_feasible_rejects_bad_candidates(il):
    import torch
    from paper_1812_01776_b200 import estimator as E
    w = workloads.make(1, n_candidates=8)
    with il.Estimator.from_workload(w) as est:
        bad = w.configs.copy()
        bad[3, 0, 2] = 0
        with pytest.raises(E.ILError) as ei:
            est.feasible(bad, w.slo_us)
        assert ei.value.code == E.IL_ERR_BAD_CONFIG
        with pytest.raises(E.ILError) as ei:
            est.feasible_device(torch.from_numpy(bad).cuda(), w.slo_us)
        assert ei.value.code == E.IL_ERR_BAD_CONFIG
        assert est.feasible(w.configs, w.slo_us).dtype == bool      # the handle stays usable


@pytest.mark.parametrize("cid", [2, 3, 5, 4])
def test_feasible_full_size_samples(il, oracle_on, cid):
    """Workloads 2-5 at full trace length on the candidates the full-size parity tests check
    (all 4,096 / a seeded 4,096 / 1,024 / 1,024, plus the extremes): flags against the oracle's P99.
    On workload 2 most of the infeasible candidates must have been dropped early."""
    import torch
    from test_gpu_parity import full_size_sample
    w, idx, ext = full_size_sample(cid)
    both = np.concatenate([w.configs[idx], ext])
    exp = oracle_on(f"w{cid}", w, both)
    with il.Estimator.from_workload(w) as est:
        est.reserve_workspace(both.shape[0])
        got = est.feasible_device(torch.from_numpy(both).cuda(), w.slo_us).cpu().numpy().astype(bool)
        st = est.stats()
    want = exp[0] <= w.slo_us
    assert np.array_equal(got, want), np.nonzero(got != want)[0][:8]
    if cid == 2:
        assert st["early_exits"] > 0.5 * (~got).sum()
