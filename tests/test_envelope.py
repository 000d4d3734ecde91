"""Traffic envelope (Section 5 of the paper): the oracle against closed forms
and brute force, then the CUDA entry point against the oracle."""
import numpy as np
import pytest

import workloads


def brute(a, win):
    a = np.asarray(a, np.int64)
    return max(int(((a >= a[j]) & (a - a[j] < win)).sum()) for j in range(len(a)))


def test_oracle_periodic_closed_form(oracle):
    T = 10
    a = np.arange(0, 5000, T, dtype=np.int64) + 3
    wins = np.array([1, 9, 10, 11, 25, 100, 101, 4990, 5000, 10 ** 9], np.int64)
    exp = np.minimum(-(-wins // T), len(a))          # ceil(window / period), capped at n
    assert np.array_equal(oracle.traffic_envelope(a, wins), exp)


@pytest.mark.parametrize("seed", range(8))
def test_oracle_against_brute_force(oracle, seed):
    rng = np.random.default_rng(seed)
    a = np.sort(rng.integers(0, 3000, size=300)).astype(np.int64)     # many equal stamps
    wins = np.array([1, 2, 7, 50, 333, 3000, 10 ** 6], np.int64)
    got = oracle.traffic_envelope(a, wins)
    assert got.tolist() == [brute(a, w) for w in wins]
    assert np.all(np.diff(got) >= 0)                                  # wider windows hold at least as many
    assert got[0] == np.bincount(a).max() and got[-1] == len(a)


@pytest.mark.parametrize("seed", range(6))
def test_oracle_against_every_integer_window_start(oracle, seed):
    """The definition itself on a tiny trace: every half-open window [t, t + w) for EVERY integer
    start t (not only starts at an arrival, which is the reduction the oracle relies on), counted
    one arrival at a time."""
    rng = np.random.default_rng(100 + seed)
    a = np.sort(rng.integers(5, 160, size=int(rng.integers(20, 50)))).astype(np.int64)
    wins = np.array([1, 2, 3, 5, 8, 13, 40, 155, 156, 400], np.int64)
    exp = []
    for w in wins:
        best = 0
        for t in range(int(a[0]) - int(w) - 1, int(a[-1]) + 2):
            best = max(best, sum(1 for x in a if t <= x < t + w))
        exp.append(best)
    assert oracle.traffic_envelope(a, wins).tolist() == exp


def test_oracle_rejects_bad_input(oracle):
    with pytest.raises(oracle.OracleError):
        oracle.traffic_envelope(np.array([5, 4], np.int64), [10])
    with pytest.raises(oracle.OracleError):
        oracle.traffic_envelope(np.array([1, 2], np.int64), [0])


def windows_for(service_time_us):
    """Window lengths as the paper discretises them: from the service time, doubling up to 60 s."""
    out, w = [], int(service_time_us)
    while w < 60_000_000:
        out.append(w)
        w *= 2
    return np.array(out + [60_000_000], np.int64)


@pytest.mark.gpu
@pytest.mark.parametrize("cid,n", [(1, None), (2, None), (3, 70_001), (4, None), (5, None)])
def test_gpu_envelope_matches_oracle(oracle, cid, n):
    import paper_1812_01776_b200 as il
    w = workloads.make(cid, n_queries=n, n_candidates=1)
    wins = np.concatenate([windows_for(20_000), [1, 3, 999, 10 ** 12]]).astype(np.int64)   # unsorted on purpose
    with il.Estimator.from_workload(w) as est:
        got = est.traffic_envelope(wins)
        assert np.array_equal(got, oracle.traffic_envelope(w.arrival_us, wins))
        assert est.traffic_envelope(np.zeros(0, np.int64)).shape == (0,)
        from paper_1812_01776_b200 import estimator as E
        with pytest.raises(E.ILError):
            est.traffic_envelope(np.array([0], np.int64))
