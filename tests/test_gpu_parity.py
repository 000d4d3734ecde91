"""Parity of the CUDA path (through the C ABI) with the CPU oracle: both
outputs are integers and must be equal element by element."""
import json
import os

import numpy as np
import pytest

import workloads
from select_cases import SELECT_CASES, grouped_workload

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def il():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1812_01776_b200 as il_
    il_.load_library()
    return il_


def gpu_run(il, w, configs=None, slo=None, host=True, ws_bytes=None, variant=0, knobs=None):
    import torch
    configs = w.configs if configs is None else configs
    slo = w.slo_us if slo is None else slo
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        for knob, value in (knobs or {}).items():
            est.set_test_knob(knob, value)
        if ws_bytes is not None:
            est.reserve_workspace(len(configs), max_bytes=ws_bytes)
        if host:
            p99, miss = est.estimate(configs, slo)
        else:
            d = torch.from_numpy(np.ascontiguousarray(configs)).cuda()
            a, b = est.estimate_device(d, slo)
            p99, miss = a.cpu().numpy(), b.cpu().numpy()
        return p99, miss, est.stats()


def check(il, oracle, w, **kw):
    exp_p99, exp_miss = oracle.estimate_workload(w)
    p99, miss, st = gpu_run(il, w, **kw)
    bad = np.nonzero((p99 != exp_p99) | (miss != exp_miss))[0]
    assert bad.size == 0, (w.name, bad[:8], p99[bad[:8]], exp_p99[bad[:8]], miss[bad[:8]],
                           exp_miss[bad[:8]], w.configs[bad[:2]])
    assert st["candidates"] == w.n_candidates
    assert st["query_events"] == w.n_candidates * w.query_events()
    return st


def _hand_cases():
    with open(os.path.join(HERE, "golden", "hand_traces.json")) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _hand_cases(), ids=lambda c: c["name"])
def test_hand_traces(il, case):
    bits = np.array(case["branch_bits"], np.uint8) if "branch_bits" in case else None
    join = None
    if "join" in case:
        join = (case["join"]["parent2"], case["join"]["cond_bit2"], case["join"]["cond_val2"])
    with il.Estimator(np.array(case["parent"], np.int32), np.array(case["cond_bit"], np.int8),
                      np.array(case["cond_val"], np.uint8), np.array(case["latency_us"], np.int32),
                      np.array(case["arrival_us"], np.int64), bits, join=join) as est:
        p99, miss = est.estimate(np.array([case["config"]], np.uint8), case["slo_us"])
    assert (int(p99[0]), int(miss[0])) == (case["p99_us"], case["miss"])


@pytest.mark.parametrize("variant", [4, 1, 2, 3], ids=["packed", "wide", "staged", "lanes"])
@pytest.mark.parametrize("seed", range(12))
def test_random_small(il, oracle, seed, variant):
    w = workloads.random_small(seed, S=1 + seed % 6, H=3, Bmax=[4, 33, 64][seed % 3], n=700 + 37 * seed,
                               C=40, max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1),
                               qps=400.0, cv=3.0, lat_lo=1, lat_hi=20000,
                               equal_stamp_every=(3 if seed % 4 == 0 else 0))
    check(il, oracle, w, host=(seed % 2 == 0), variant=variant)


@pytest.mark.parametrize("variant", [4, 1, 2, 3], ids=["packed", "wide", "staged", "lanes"])
@pytest.mark.parametrize("seed", [1, 4, 7, 10])
def test_per_query_latencies(il, oracle, seed, variant):
    """The full answer of the Estimator, query by query, against the oracle."""
    w = workloads.random_small(seed, S=2 + seed % 5, H=3, Bmax=[4, 33, 64][seed % 3], n=900 + 31 * seed,
                               C=6, max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1),
                               qps=400.0, cv=3.0, lat_lo=1, lat_hi=20000,
                               equal_stamp_every=(3 if seed % 4 == 0 else 0))
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        for c in range(w.n_candidates):
            got = est.latencies(w.configs[c])
            _, _, exp = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                            w.branch_bits, w.configs[c], w.slo_us, want_latency=True)
            assert np.array_equal(got, exp), (seed, c, np.nonzero(got != exp)[0][:5])


def test_per_query_latencies_workloads(il, oracle):
    for cid, n in [(2, 20000), (3, 20000), (5, 20000)]:
        w = workloads.make(cid, n_queries=n, n_candidates=4)
        with il.Estimator.from_workload(w) as est:
            for c in range(4):
                _, _, exp = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                                w.branch_bits, w.configs[c], w.slo_us, want_latency=True)
                assert np.array_equal(est.latencies(w.configs[c]), exp), (cid, c)


@pytest.mark.parametrize("variant", [4, 0], ids=["packed", "auto"])
@pytest.mark.parametrize("seed", range(6))
def test_times_scaled_beyond_the_32_bit_loop(il, oracle, seed, variant):
    """Latencies of 2^24 us and more take the 64-bit stage loop of the packed
    kernel (its run step, late-slot merge and single step included)."""
    w = workloads.random_small(200 + seed, S=2 + seed % 4, H=2, Bmax=[4, 33, 64][seed % 3], n=900, C=30,
                               max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1), qps=400.0, cv=3.0,
                               lat_lo=4100, lat_hi=20000, equal_stamp_every=(3 if seed % 3 == 0 else 0))
    w.latency_us = w.latency_us * 4096            # 1.7e7 .. 8.2e7 us: above the 32-bit loop's limit
    w.arrival_us = w.arrival_us * 4096
    w.slo_us = w.slo_us * 4096
    assert w.latency_us.min() >= 1 << 24
    check(il, oracle, w, variant=variant)


@pytest.mark.parametrize("variant", [4, 0], ids=["packed", "auto"])
@pytest.mark.parametrize("seed", range(6))
def test_sparse_traces_move_the_epoch(il, oracle, seed, variant):
    """Gaps between arrivals far beyond 2^30 us (and, for odd seeds, services
    long enough that batches stay in flight across them) exercise the 32-bit
    loop's epoch moves and its hand-over to the 64-bit loop."""
    w = workloads.random_small(300 + seed, S=2 + seed % 3, H=2, Bmax=8, n=600, C=24, max_replicas=4,
                               tree=(seed % 2 == 0), qps=[0.0004, 0.002, 0.01][seed % 3], cv=4.0,
                               lat_lo=1000, lat_hi=(1 << 24) - 1 if seed % 2 else 50000,
                               equal_stamp_every=(2 if seed == 4 else 0))
    assert np.diff(w.arrival_us).max() > (1 << 30)
    check(il, oracle, w, variant=variant)


@pytest.mark.parametrize("ring_log2", [6, 8, 10])
@pytest.mark.parametrize("seed", range(12))
def test_lane_kernel_short_stream_rings(il, oracle, seed, ring_log2):
    """Stream rings of 64 / 256 / 1,024 records on traces of 700 to 1,100 queries: ring positions wrap,
    parents wait for room, and candidates whose oldest batch in flight pins more than a ring are
    handed to the warp-per-candidate kernel.  Results must not change."""
    w = workloads.random_small(seed, S=1 + seed % 6, H=3, Bmax=[4, 33, 64][seed % 3], n=700 + 37 * seed,
                               C=40, max_replicas=[3, 8, 32][seed % 3], tree=(seed % 2 == 1),
                               qps=400.0, cv=3.0, lat_lo=1, lat_hi=20000,
                               equal_stamp_every=(3 if seed % 4 == 0 else 0))
    check(il, oracle, w, host=(seed % 2 == 0), variant=3, knobs={1: ring_log2})


@pytest.mark.parametrize("cid,n,C", [(2, 5000, 300), (3, 6001, 200), (4, 3000, 150), (5, 4097, 260)])
def test_configs_reduced_short_stream_rings(il, oracle, cid, n, C):
    """The five workload shapes with 256-record rings: with the workloads' affine tables most
    candidates finish on the lane kernel, the others take the overflow path."""
    st = check(il, oracle, workloads.make(cid, n_queries=n, n_candidates=C), host=False, variant=3, knobs={1: 8})
    assert 0 <= st["fallback_candidates"] <= C


def test_production_ring_length_rarely_overflows(il, oracle):
    """With the ring length the library uses for long traces (8,192 records) and the workloads'
    tables, a trace five times longer than a ring runs on the lane kernel alone."""
    w = workloads.make(2, n_queries=40000, n_candidates=192)
    st = check(il, oracle, w, host=False, knobs={1: 13})
    assert st["fallback_candidates"] <= 2


def test_config1_full(il, oracle):
    st = check(il, oracle, workloads.make(1))
    # the lane kernel: one reduction over the configurations, then (simulate, select) per chunk
    assert st["batches"] > 0 and st["kernel_launches"] == 1 + 2 * st["chunks"]


@pytest.mark.parametrize("variant", [4, 1, 2, 3], ids=["packed", "wide", "staged", "lanes"])
@pytest.mark.parametrize("cid,n,C", [(2, 5000, 300), (3, 6001, 200), (4, 3000, 150), (5, 4097, 260)])
def test_configs_reduced(il, oracle, cid, n, C, variant):
    check(il, oracle, workloads.make(cid, n_queries=n, n_candidates=C), host=False, variant=variant)


@pytest.mark.parametrize("in_records", [0, 1])
@pytest.mark.parametrize("case", ["w3", "w5", "tree_rings", "fan_out", "feasible"])
def test_branch_bits_in_records_or_looked_up(il, oracle, case, in_records):
    """Pipelines with branch points on the lane kernel: the stream records carry the queries' branch
    bits (the default where the time range leaves room) or every stage looks them up by query index.
    Same integers either way: estimate, stream rings, fan-out, feasibility-only."""
    knobs = {5: in_records}
    if case == "w3":
        check(il, oracle, workloads.make(3, n_queries=6001, n_candidates=200), host=False, variant=3, knobs=knobs)
    elif case == "w5":
        check(il, oracle, workloads.make(5, n_queries=4097, n_candidates=260), host=True, variant=3, knobs=knobs)
    elif case == "tree_rings":
        w = workloads.random_small(7, S=6, H=3, Bmax=33, n=959, C=40, max_replicas=8, tree=True, qps=400.0, cv=3.0,
                                   lat_lo=1, lat_hi=20000, equal_stamp_every=3)
        check(il, oracle, w, host=False, variant=3, knobs={1: 8, **knobs})
    elif case == "fan_out":
        check(il, oracle, workloads.fan_out_small(11, n=1500, C=48, max_replicas=8, Bmax=16), host=False, knobs=knobs)
    else:
        w = workloads.make(3, n_queries=6001, n_candidates=200)
        exp = oracle.estimate_workload(w)[0]
        with il.Estimator.from_workload(w) as est:
            est.set_test_knob(5, in_records)
            for slo in (w.slo_us, int(np.median(exp))):
                assert np.array_equal(est.feasible(w.configs, slo), exp <= slo)


def test_times_too_large_to_pack_fall_back_to_wide_kernel(il, oracle):
    """Arrival stamps near 2^58 leave no room for the query index in a 64-bit
    record: the library must pick the kernel with separate time and query
    streams on its own, with the same results as for the unshifted trace."""
    w = workloads.make(3, n_queries=3000, n_candidates=64)
    exp = oracle.estimate_workload(w)
    w.arrival_us = w.arrival_us + (1 << 58)
    p99, miss, _ = gpu_run(il, w)
    assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])


@pytest.mark.parametrize("variant", [0, 4, 1], ids=["auto", "packed", "wide"])
def test_recommended_workspace_holds_the_batch_in_one_chunk(il, oracle, variant):
    """A workspace of the size the library recommends for a batch takes that batch in one pass: a second
    chunk of a few left-over candidates would cost a whole further walk over the trace."""
    import torch
    w = workloads.make(2, n_queries=3000, n_candidates=700)
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        est.reserve_workspace(w.n_candidates)
        a, b = est.estimate_device(torch.from_numpy(w.configs).cuda(), w.slo_us)
        assert est.stats()["chunks"] == 1
        assert np.array_equal(a.cpu().numpy(), exp[0]) and np.array_equal(b.cpu().numpy(), exp[1])


@pytest.mark.parametrize("variant", [4, 3], ids=["packed", "lanes"])
def test_multi_chunk_small_workspace(il, oracle, variant):
    """A workspace that holds only a few candidates forces many chunks."""
    w = workloads.make(2, n_queries=2000, n_candidates=100)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        lo = il.il_workspace_min_bytes(est._h)
    st = check(il, oracle, w, ws_bytes=lo + 40 * 2000 * 8, variant=variant)
    assert st["chunks"] > 1


def test_edge_cases(il, oracle):
    # one query, one stage
    w = workloads.random_small(100, S=1, H=1, Bmax=1, n=1, C=1, max_replicas=1)
    check(il, oracle, w)
    # all queries at one instant, largest batch and replica counts
    w = workloads.random_small(101, S=3, H=2, Bmax=64, n=1000, C=8, max_replicas=32)
    w.arrival_us[:] = 5
    w.configs[:, :, workloads.CFG_MAX_BATCH] = 64
    w.configs[:, :, workloads.CFG_REPLICAS] = [[32, 1, 32]] * 8
    check(il, oracle, w)
    # a branch nobody takes (a stage with zero visits) and one everybody takes
    w = workloads.make(3, n_queries=500, n_candidates=16)
    w.branch_bits[:] = 0
    check(il, oracle, w)
    w.branch_bits[:] = 1
    check(il, oracle, w)
    # latencies beyond 32 bits: a slow single replica on a long trace
    w = workloads.random_small(102, S=2, H=1, Bmax=2, n=3000, C=4, max_replicas=1,
                               lat_lo=2_000_000_000, lat_hi=2_100_000_000)
    exp = oracle.estimate_workload(w)
    assert exp[0].max() > 2 ** 32
    check(il, oracle, w)
    # zero candidates is a no-op
    with il.Estimator.from_workload(w) as est:
        p99, miss = est.estimate(w.configs[:0], w.slo_us)
        assert p99.shape == (0,) and miss.shape == (0,)


def test_bad_candidates_are_rejected(il):
    import torch
    from paper_1812_01776_b200 import estimator as E
    w = workloads.make(1, n_candidates=8)
    with il.Estimator.from_workload(w) as est:
        for col, val in [(0, 2), (1, 0), (1, 17), (2, 0), (2, 33)]:
            bad = w.configs.copy()
            bad[5, 1, col] = val
            with pytest.raises(E.ILError) as ei:
                est.estimate(bad, w.slo_us)
            assert ei.value.code == E.IL_ERR_BAD_CONFIG
            with pytest.raises(E.ILError) as ei:
                est.estimate_device(torch.from_numpy(bad).cuda(), w.slo_us)
            assert ei.value.code == E.IL_ERR_BAD_CONFIG
        # the handle stays usable
        p99, _ = est.estimate(w.configs, w.slo_us)
        assert (p99 > 0).all()


def test_repeatable_and_stream(il, oracle):
    import torch
    w = workloads.make(2, n_queries=3000, n_candidates=64)
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.reserve_workspace(64)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            est.use_current_stream()
            d = torch.from_numpy(w.configs).cuda()
            for _ in range(3):
                a, b = est.estimate_device(d, w.slo_us)
                assert np.array_equal(a.cpu().numpy(), exp[0])
                assert np.array_equal(b.cpu().numpy(), exp[1])


def full_size_sample(cid):
    """The candidates of workloads 2-5 that the full-size tests check against the oracle: the workload
    the GPU runs, the indices (into its candidates) that are checked, and the extremes checked beside
    them.  Workload 2: all 4,096.  Workload 3: a seeded 4,096 of 65,536.  Workload 5: a seeded 1,024 of
    1,048,576.  Workload 4: every 16th (1,024) of the seeded 16,384-candidate sample the bench times,
    itself drawn from the whole set of 262,144."""
    if cid == 2:
        w = workloads.make(2)
        return w, np.arange(w.n_candidates), _extremes(4, 3, (1, 32), (1, 8))
    if cid == 3:
        w = workloads.make(3)
        return w, np.sort(np.random.default_rng(3).choice(w.n_candidates, size=4096, replace=False)), \
            _extremes(6, 3, (1, 64), (1, 8))
    if cid == 5:
        w = workloads.make(5)
        return w, np.sort(np.random.default_rng(5).choice(w.n_candidates, size=1024, replace=False)), \
            _extremes(8, 4, (1, 64), (1, 32))
    w, _ = workloads.sub_batch(4, 16384)
    return w, np.arange(0, w.n_candidates, 16), _extremes(10, 4, (1, 64), (1, 16))


def _extremes(S, H, mbs, Rs):
    return np.array([[[h, mb, R, 0]] * S for h in range(H) for mb in mbs for R in Rs], np.uint8)


def _run_all(il, w, variant=0):
    """Every candidate of w through il_estimate_device with a torch-owned
    workspace: the launch configuration the bench times."""
    import torch
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        est.reserve_workspace(w.n_candidates)
        d = torch.from_numpy(w.configs).cuda()
        a, b = est.estimate_device(d, w.slo_us)
        p99, miss = a.cpu().numpy(), b.cpu().numpy()
        st = est.stats()
    assert st["candidates"] == w.n_candidates
    return p99, miss


def _assert_equal(w, got, exp, configs):
    bad = np.nonzero((got[0] != exp[0]) | (got[1] != exp[1]))[0]
    assert bad.size == 0, (w.name, bad.size, bad[:5], got[0][bad[:5]], exp[0][bad[:5]],
                           got[1][bad[:5]], exp[1][bad[:5]], configs[bad[:2]])


def _properties(w, p99, miss):
    """What holds for every candidate whatever the size: the two outputs agree on
    feasibility (Section 4.3), and both lie in their ranges."""
    k = (99 * w.n_queries + 99) // 100
    assert np.array_equal(p99 <= w.slo_us, miss <= w.n_queries - k)
    assert (p99 > 0).all() and (miss >= 0).all() and (miss <= w.n_queries).all()


def _sampled_check(il, oracle_on, cid, variant=0, gpu_subset_only=False):
    """All candidates of the workload on the GPU; the sampled candidates plus the extremes against
    the oracle one by one; the size-free properties on all."""
    w, idx, ext = full_size_sample(cid)
    both = np.concatenate([w.configs[idx], ext])
    exp = oracle_on(f"w{cid}", w, both)
    if gpu_subset_only:
        w.configs = np.ascontiguousarray(w.configs[idx])
        idx = np.arange(w.n_candidates)
    p99, miss = _run_all(il, w, variant)
    e = gpu_run(il, w, configs=ext, host=True, variant=variant)
    got = (np.concatenate([p99[idx], e[0]]), np.concatenate([miss[idx], e[1]]))
    _assert_equal(w, got, exp, both)
    _properties(w, p99, miss)


@pytest.mark.parametrize("variant", [0, 4], ids=["auto", "packed"])
def test_config2_full_size_all_4096(il, oracle_on, variant):
    """Workload 2 in full: ALL 4,096 candidates x 50,000 queries against the oracle,
    plus 12 structured extremes (every hardware type, 1 / 8 replicas, max batch 1 / 32)."""
    _sampled_check(il, oracle_on, 2, variant)


def test_config3_full_size_sample_4096(il, oracle_on):
    """All 65,536 candidates x 200,000 queries of the 6-stage tree on the GPU; a seeded
    sample of 4,096 candidates and 12 extremes against the oracle."""
    _sampled_check(il, oracle_on, 3)


def test_config5_full_size_sample_1024(il, oracle_on):
    """All 1,048,576 candidates x 100,000 queries of the 8-stage tree (R up to 32, max batch up
    to 64) on the GPU; a seeded sample of 1,024 candidates and 16 extremes against the oracle.  The
    candidate set is a product of per-stage choices, so the full sweep goes through the shared-prefix
    path; the sampled candidates are also run on the lane kernel alone."""
    _sampled_check(il, oracle_on, 5)
    w, idx, ext = full_size_sample(5)
    exp = oracle_on("w5", w, np.concatenate([w.configs[idx], ext]))
    got = gpu_run(il, w, configs=w.configs[idx], host=False, knobs={3: 2})
    assert got[2]["stage_runs"] == idx.shape[0] * w.n_stages
    assert np.array_equal(got[0], exp[0][:idx.shape[0]]) and np.array_equal(got[1], exp[1][:idx.shape[0]])


@pytest.mark.parametrize("variant", [0, 4], ids=["auto", "packed"])
def test_config4_full_trace_sample_1024(il, oracle_on, variant):
    """The 10-stage pipeline on its full 1,000,000-query trace.  The whole sweep is 262,144
    candidates (2.6e12 query-events, minutes of GPU time), so the GPU runs the seeded
    16,384-candidate sub-batch the bench times, drawn from the WHOLE candidate set; 1,024 of
    those (every 16th) and 16 extremes are checked against the oracle.  The warp-per-candidate
    kernel runs the 1,024 checked candidates only."""
    _sampled_check(il, oracle_on, 4, variant, gpu_subset_only=(variant != 0))


@pytest.mark.parametrize("variant", [3, 4, 1], ids=["lanes", "packed", "wide"])
@pytest.mark.parametrize("case", sorted(SELECT_CASES))
def test_percentile_kernel_on_chosen_latency_multisets(il, oracle, case, variant):
    """The CUDA percentile kernel on the P99 pin cases (all-equal, duplicates, n = 1 / 100 / 101,
    values above 2^32 among small ones): expected values come from numpy's sort of the multiset
    the workload is built to produce, and the oracle must agree with both."""
    sizes, by_size, S = SELECT_CASES[case]
    w, want = grouped_workload(sizes, by_size, S)
    n = want.shape[0]
    k = (99 * n + 99) // 100
    srt = np.sort(want)
    for slo in (int(srt[0]) - 1, int(srt[k - 1]), int(srt[-1]), int(srt[n // 2])):
        w.slo_us = slo
        exp = (int(srt[k - 1]), int((want > slo).sum()))
        assert oracle.estimate_workload(w)[0][0] == exp[0] and oracle.estimate_workload(w)[1][0] == exp[1]
        p99, miss, _ = gpu_run(il, w, variant=variant)
        assert (int(p99[0]), int(miss[0])) == exp, (case, slo)


def test_kernel_choice(il):
    """The default picks the lane kernel, and the wide kernel when times do not fit a record."""
    from paper_1812_01776_b200 import estimator as E
    w = workloads.make(2, n_queries=5000, n_candidates=4)
    with il.Estimator.from_workload(w) as est:
        assert est.kernel_name() == "des_lane_kernel"
        est.set_variant(E.IL_VARIANT_PACKED)
        assert est.kernel_name() == "des_packed_kernel"
        est.set_variant(E.IL_VARIANT_WIDE)
        assert est.kernel_name() == "des_kernel"
    w.arrival_us = w.arrival_us + (1 << 58)
    with il.Estimator.from_workload(w) as est:
        assert est.kernel_name() == "des_kernel"
        est.set_variant(E.IL_VARIANT_LANES)
        assert est.kernel_name() == "des_kernel"
    w = workloads.make(4, n_queries=2_000_000, n_candidates=2)   # 18 x 10^6 stream records per candidate:
    with il.Estimator.from_workload(w) as est:                   # the lane kernel's rings do not grow with that
        assert est.kernel_name() == "des_lane_kernel"


@pytest.mark.parametrize("variant", [3, 4], ids=["lanes", "packed"])
@pytest.mark.parametrize("S,tree", [(11, False), (13, True), (16, False), (16, True)])
def test_deep_pipelines(il, oracle, S, tree, variant):
    """Up to the largest stage count the interface takes (16): from 11 stages on only two candidates
    share a warp of the lane kernel, and some of its lanes stay idle."""
    w = workloads.random_small(400 + S + int(tree), S=S, H=2, Bmax=16, n=1500, C=21, max_replicas=6, tree=tree,
                               qps=300.0, cv=2.0, lat_lo=200, lat_hi=9000, equal_stamp_every=(5 if tree else 0))
    check(il, oracle, w, host=False, variant=variant)


@pytest.mark.parametrize("variant", [0, 4, 1, 2], ids=["auto", "packed", "wide", "staged"])
def test_largest_table_shape(il, oracle, variant):
    """16 stages x 8 hardware types x 64 batch sizes: 32 KB of profile tables, which together with a
    kernel's static shared memory passes the 48 KB a kernel gets without opting in."""
    w = workloads.random_small(500, S=16, H=8, Bmax=64, n=1200, C=19, max_replicas=32, tree=True,
                               qps=300.0, cv=2.0, lat_lo=50, lat_hi=9000)
    check(il, oracle, w, host=False, variant=variant)


@pytest.mark.parametrize("variant", [3, 4, 1, 2], ids=["lanes", "packed", "wide", "staged"])
def test_iteration_bound_is_reported_and_the_handle_survives(il, oracle, variant):
    """Every simulation kernel bounds its loops and reports IL_ERR_ITER_LIMIT instead of spinning.
    The bound cannot be reached on valid input, so the test shortens it through the test knob: the
    call must come back with that code, and the same handle must give oracle-exact results again
    once the bound is restored."""
    from paper_1812_01776_b200 import estimator as E
    w = workloads.make(3, n_queries=3000, n_candidates=40)
    exp = oracle.estimate_workload(w)
    with il.Estimator.from_workload(w) as est:
        est.set_variant(variant)
        est.set_test_knob(E.IL_KNOB_ITER_LIMIT, 50)
        with pytest.raises(E.ILError) as ei:
            est.estimate(w.configs, w.slo_us)
        assert ei.value.code == E.IL_ERR_ITER_LIMIT
        with pytest.raises(E.ILError) as ei:
            est.feasible(w.configs, w.slo_us)
        assert ei.value.code == E.IL_ERR_ITER_LIMIT
        est.set_test_knob(E.IL_KNOB_ITER_LIMIT, 0)
        p99, miss = est.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])
        assert np.array_equal(est.feasible(w.configs, w.slo_us), exp[0] <= w.slo_us)
