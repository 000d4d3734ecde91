"""Pins for the CPU oracle: closed forms, textbook recursions, hand traces,
brute force and invariants.  None of these reuse the oracle's own code; each
is chosen so that a plausible mistake in the event-heap simulator (a dropped
phase, a wrong tie-break, a transposed table index, an off-by-one rank) fails
at least one of them.
"""
import json
import os

import numpy as np
import pytest

import workloads

HERE = os.path.dirname(os.path.abspath(__file__))


def single_stage(lat_row, R=1, mb=1):
    """One stage, one hardware type, table lat_row (b = 1..len)."""
    lat = np.asarray(lat_row, dtype=np.int32).reshape(1, 1, -1)
    cfg = np.array([[0, mb, R, 0]], dtype=np.uint8)
    return (np.array([-1], np.int32), np.array([-1], np.int8), np.array([0], np.uint8), lat), cfg


def run(oracle, topo, arrivals, cfg, slo=0, bits=None, **kw):
    parent, cbit, cval, lat = topo
    return oracle.estimate_one(parent, cbit, cval, lat, np.asarray(arrivals, np.int64), bits,
                               cfg, slo, **kw)


def rank_k(n):
    return (99 * n + 99) // 100


# --------------------------------------------------------------------------
# closed forms and textbook recursions
# --------------------------------------------------------------------------

@pytest.mark.parametrize("seed,D", [(0, 3000), (1, 5200), (2, 9000)])
def test_lindley_single_server(oracle, seed, D):
    """R=1, max batch 1: waiting times obey Lindley's recursion exactly."""
    rng = np.random.default_rng(seed)
    a = workloads.gamma_arrivals(rng, 5000, 200.0, 4.0)
    topo, cfg = single_stage([D])
    p99, miss, lat = run(oracle, topo, a, cfg, slo=2 * D, want_latency=True)
    w = 0
    exp = np.empty(len(a), np.int64)
    for i in range(len(a)):
        if i:
            w = max(0, w + D - int(a[i] - a[i - 1]))
        exp[i] = w + D
    assert np.array_equal(lat, exp)
    assert p99 == np.sort(exp)[rank_k(len(a)) - 1]
    assert miss == int((exp > 2 * D).sum())


@pytest.mark.parametrize("T,D", [(100, 100), (100, 60), (100, 130), (7, 10)])
def test_deterministic_arrivals_closed_form(oracle, T, D):
    n = 1000
    a = np.arange(n, dtype=np.int64) * T + 17
    topo, cfg = single_stage([D])
    slo = D + 50 * max(D - T, 0) + 1
    p99, miss, lat = run(oracle, topo, a, cfg, slo=slo, want_latency=True)
    i = np.arange(n, dtype=np.int64)
    exp = D + i * max(D - T, 0)
    assert np.array_equal(lat, exp)
    assert p99 == D + (rank_k(n) - 1) * max(D - T, 0)
    assert miss == int((exp > slo).sum())


def test_md1_mean_wait_pollaczek_khinchine(oracle):
    """Poisson arrivals, deterministic service: mean wait -> rho D / (2 (1 - rho))."""
    rng = np.random.default_rng(7)
    lam, D = 100.0, 6000  # rho = 0.6
    n = 1_000_000
    a = workloads.gamma_arrivals(rng, n, lam, 1.0)
    topo, cfg = single_stage([D])
    _, _, lat = run(oracle, topo, a, cfg, want_latency=True)
    rho = lam * D * 1e-6
    expect = rho * D / (2 * (1 - rho))
    got = float(lat.mean()) - D
    assert abs(got - expect) / expect < 0.03


@pytest.mark.parametrize("R,D,seed", [(2, 9000, 0), (3, 14000, 1), (5, 20000, 2), (32, 150000, 3)])
def test_kiefer_wolfowitz_multi_server(oracle, R, D, seed):
    """R identical servers, max batch 1, FIFO: the sorted residual-work vector
    recursion W <- sort((W + D e_1 - gap)^+) gives each query's wait W[0]."""
    rng = np.random.default_rng(seed)
    a = workloads.gamma_arrivals(rng, 4000, 250.0, 2.0)
    topo, cfg = single_stage([D], R=R)
    _, _, lat = run(oracle, topo, a, cfg, want_latency=True)
    W = np.zeros(R, dtype=np.int64)
    exp = np.empty(len(a), np.int64)
    for i in range(len(a)):
        if i:
            W = np.maximum(W - int(a[i] - a[i - 1]), 0)
            W.sort()
        exp[i] = W[0] + D
        W[0] += D
        W.sort()
    assert np.array_equal(lat, exp)


def test_tandem_recursion_linear_pipeline(oracle):
    """Linear chain, R=1 and max batch 1 everywhere: d_s(i) = max(d_{s-1}(i), d_s(i-1)) + D_s."""
    rng = np.random.default_rng(3)
    S = 4
    D = [4000, 7000, 5100, 6900]
    a = workloads.gamma_arrivals(rng, 3000, 150.0, 4.0)
    lat = np.zeros((S, 2, 3), np.int32)
    for s in range(S):
        lat[s, 0] = 99999            # wrong hardware row: must not be used
        lat[s, 1] = [D[s], 1, 1]     # only b = 1 is ever used
    parent = np.arange(-1, S - 1, dtype=np.int32)
    cfg = np.array([[1, 1, 1, 0]] * S, np.uint8)
    topo = (parent, np.full(S, -1, np.int8), np.zeros(S, np.uint8), lat)
    _, _, got = run(oracle, topo, a, cfg, want_latency=True)
    d_prev = a.copy()
    for s in range(S):
        d = np.empty_like(a)
        last = 0
        for i in range(len(a)):
            last = max(int(d_prev[i]), last) + D[s]
            d[i] = last
        d_prev = d
    assert np.array_equal(got, d_prev - a)


@pytest.mark.parametrize("n,m", [(10, 4), (64, 64), (65, 64), (7, 1), (100, 16), (5, 8)])
def test_batch_drain(oracle, n, m):
    """All n queries at t=0, one replica, max batch m: full batches back to
    back, then one partial batch whose time is the table entry of its size."""
    table = [100 + 13 * b + (b * b) % 7 for b in range(1, 65)]
    topo, cfg = single_stage(table, R=1, mb=m)
    a = np.zeros(n, np.int64)
    _, _, lat = run(oracle, topo, a, cfg, want_latency=True)
    exp = np.empty(n, np.int64)
    t, i = 0, 0
    J = -(-n // m)
    for j in range(J):
        b = min(m, n - j * m)
        t += table[b - 1]
        exp[j * m:j * m + b] = t
    assert np.array_equal(lat, exp)
    # closed form of the last batch
    last_b = n - (J - 1) * m
    assert lat[-1] == (J - 1) * table[m - 1] + table[last_b - 1]


def test_never_queue_limit_is_service_time(oracle):
    """Enough replicas that one is always idle and distinct stamps: every batch
    has size 1 and the latency is the sum of batch-1 times along the chain."""
    rng = np.random.default_rng(11)
    S, H, B = 3, 2, 8
    lat = rng.integers(50, 500, size=(S, H, B)).astype(np.int32)
    a = np.cumsum(rng.integers(20, 60, size=500)).astype(np.int64)  # distinct stamps
    parent = np.arange(-1, S - 1, dtype=np.int32)
    cfg = np.array([[1, 8, 32, 0], [0, 4, 32, 0], [1, 8, 32, 0]], np.uint8)
    topo = (parent, np.full(S, -1, np.int8), np.zeros(S, np.uint8), lat)
    p99, miss, got = run(oracle, topo, a, cfg, slo=0, want_latency=True)
    svc = int(lat[0, 1, 0]) + int(lat[1, 0, 0]) + int(lat[2, 1, 0])
    assert np.all(got == svc)
    assert p99 == svc and miss == len(a)


# --------------------------------------------------------------------------
# hand traces
# --------------------------------------------------------------------------

def _hand_cases():
    with open(os.path.join(HERE, "golden", "hand_traces.json")) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _hand_cases(), ids=lambda c: c["name"])
def test_hand_traces(oracle, case):
    topo = (np.array(case["parent"], np.int32), np.array(case["cond_bit"], np.int8),
            np.array(case["cond_val"], np.uint8), np.array(case["latency_us"], np.int32))
    bits = np.array(case["branch_bits"], np.uint8) if "branch_bits" in case else None
    kw = {}
    if "join" in case:
        kw["join"] = (case["join"]["parent2"], case["join"]["cond_bit2"], case["join"]["cond_val2"])
    p99, miss, lat = run(oracle, topo, case["arrival_us"], np.array(case["config"], np.uint8),
                         slo=case["slo_us"], bits=bits, want_latency=True, **kw)
    assert lat.tolist() == case["latency"]
    assert p99 == case["p99_us"]
    assert miss == case["miss"]
    for why, alt in case["alt_p99"].items():
        assert p99 != alt, why


# --------------------------------------------------------------------------
# brute force: a clock-tick simulator on tiny integer times
# --------------------------------------------------------------------------

def tick_simulate(w, cfg):
    """Advance the clock one microsecond at a time and apply the rules at each
    tick.  Exponentially slower than the event heap and shaped differently (no
    heap, no event records): usable only when all times are tiny."""
    S = w.n_stages
    n = w.n_queries
    join = getattr(w, "join", None)
    # edges[s] = [(child, guard bit, guard value)], child by child
    edges = [[] for _ in range(S)]
    for c in range(1, S):
        edges[int(w.parent[c])].append((c, int(w.cond_bit[c]), int(w.cond_val[c])))
        if join is not None and int(join[0][c]) >= 0:
            edges[int(join[0][c])].append((c, int(join[1][c]), int(join[2][c])))
    for e in edges:
        e.sort()

    def follows(q, bit, val):
        return bit < 0 or ((int(w.branch_bits[q]) >> bit) & 1) == val

    def inputs_of(q):
        """per stage, how many of its incoming edges carry query q"""
        seen = [0] * S
        seen[0] = 1
        for s in range(S):                     # parents come before children
            if seen[s]:
                for c, bit, val in edges[s]:
                    seen[c] += follows(q, bit, val)
        return seen

    wanted = [inputs_of(q) for q in range(n)]
    got = [[0] * S for _ in range(n)]
    queue = [[] for _ in range(S)]
    running = [dict() for _ in range(S)]     # replica -> (finish, order, [ids])
    order = 0
    lat = [None] * n
    copies = [1] * n
    nxt = 0
    t = int(w.arrival_us[0])
    left = n
    while left:
        # batches that finish now: stage by stage, within a stage in dispatch order
        fin = sorted((s, o, r) for s in range(S) for r, (f, o, _) in running[s].items() if f == t)
        for s, _, r in fin:
            ids = running[s].pop(r)[2]
            for q in ids:
                went_on = 0
                for child, bit, val in edges[s]:      # every edge whose condition holds
                    if not follows(q, bit, val):
                        continue
                    got[q][child] += 1
                    if got[q][child] == wanted[q][child]:   # the stage has all its inputs for q
                        queue[child].append(q)
                        went_on += 1
                copies[q] += went_on - 1
                if copies[q] == 0:                    # the last copy of the query has left
                    lat[q] = t - int(w.arrival_us[q])
                    left -= 1
        while nxt < n and int(w.arrival_us[nxt]) == t:
            queue[0].append(nxt)
            nxt += 1
        for s in range(S):
            hw, mb, R = int(cfg[s, 0]), int(cfg[s, 1]), int(cfg[s, 2])
            while queue[s]:
                idle = [r for r in range(R) if r not in running[s]]
                if not idle:
                    break
                b = min(len(queue[s]), mb)
                ids, queue[s] = queue[s][:b], queue[s][b:]
                order += 1
                running[s][idle[0]] = (t + int(w.latency_us[s, hw, b - 1]), order, ids)
        t += 1
    return np.array(lat, np.int64)


@pytest.mark.parametrize("seed", range(24))
def test_tick_brute_force_small_random(oracle, seed):
    tree = seed % 2 == 1
    w = workloads.random_small(seed, S=2 + seed % 4, H=2, Bmax=4, n=40, C=6, max_replicas=3,
                               tree=tree, qps=80_000.0, cv=2.0, lat_lo=1, lat_hi=30,
                               equal_stamp_every=(3 if seed % 3 == 0 else 0))
    for c in range(w.n_candidates):
        exp = tick_simulate(w, w.configs[c])
        p99, miss, lat = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                             w.arrival_us, w.branch_bits, w.configs[c], 40,
                                             want_latency=True)
        assert np.array_equal(lat, exp), (seed, c)
        assert p99 == np.sort(exp)[rank_k(len(exp)) - 1]
        assert miss == int((exp > 40).sum())


# --------------------------------------------------------------------------
# routing
# --------------------------------------------------------------------------

def test_tree_routing_all_bit_patterns(oracle):
    """The 8-stage tree of workload 5 with 32 replicas per stage and spaced
    arrivals: each query's latency is the batch-1 service time of its own path,
    for every combination of the three branch bits."""
    w = workloads.make(5, n_queries=8, n_candidates=1)
    lat = w.latency_us
    cfg = np.array([[s % 4, 64, 32, 0] for s in range(8)], np.uint8)
    a = (np.arange(8, dtype=np.int64) + 1) * 10_000_000
    bits = np.arange(8, dtype=np.uint8)
    _, _, got = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, lat, a, bits, cfg, 0,
                                    want_latency=True)
    paths = {(0, 0): [0, 1, 3, 7], (0, 1): [0, 1, 4], (1, 0): [0, 2, 5], (1, 1): [0, 2, 6]}
    for q in range(8):
        b0, b1, b2 = q & 1, (q >> 1) & 1, (q >> 2) & 1
        path = paths[(b0, b1 if b0 == 0 else b2)]
        assert got[q] == sum(int(lat[s, s % 4, 0]) for s in path), q


@pytest.mark.parametrize("cid", [3, 5])
def test_conservation_of_queries(oracle, cid):
    """Every query is served exactly once at each stage on its path: the batch
    sizes logged per stage add up to n_s computed from the bits alone."""
    w = workloads.make(cid, n_queries=3000, n_candidates=8)
    ns = w.visits_per_stage()
    for c in range(w.n_candidates):
        _, _, lat, log = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                             w.arrival_us, w.branch_bits, w.configs[c],
                                             w.slo_us, want_latency=True, want_log=True)
        served = np.bincount(log["stage"], weights=log["batch"], minlength=w.n_stages)
        assert np.array_equal(served.astype(np.int64), ns)
        assert np.all(lat > 0)


# --------------------------------------------------------------------------
# percentile and miss count
# --------------------------------------------------------------------------

@pytest.mark.parametrize("n", [1, 2, 99, 100, 101, 199, 200, 201, 1000, 12345])
def test_p99_rank_and_miss(oracle, n):
    rng = np.random.default_rng(n)
    x = rng.integers(0, 50, size=n).astype(np.int64) * 1000  # many duplicates
    slo = 25_000
    p99, miss = oracle.p99_miss(x, slo)
    k = -(-99 * n // 100)
    assert k == rank_k(n)
    assert p99 == np.sort(x)[k - 1]
    assert miss == int((x > slo).sum())
    # p99 <= slo  <=>  at most n - k entries above slo
    assert (p99 <= slo) == (miss <= n - k)


def test_p99_known_ranks(oracle):
    assert rank_k(2000) == 1980 and rank_k(50_000) == 49_500 and rank_k(100_000) == 99_000
    assert rank_k(200_000) == 198_000 and rank_k(1_000_000) == 990_000
    x = np.arange(1, 101, dtype=np.int64)          # n = 100 -> k = 99
    assert oracle.p99_miss(x, 99) == (99, 1)
    x = np.arange(1, 102, dtype=np.int64)          # n = 101 -> k = 100
    assert oracle.p99_miss(x, 100) == (100, 1)
    assert oracle.p99_miss(np.full(17, 5, np.int64), 5) == (5, 0)
    assert oracle.p99_miss(np.full(17, 5, np.int64), 4) == (5, 17)
    big = np.array([2 ** 40 + 3, 1, 2 ** 40 + 1], np.int64)
    assert oracle.p99_miss(big, 2 ** 40 + 1) == (2 ** 40 + 3, 1)


def test_miss_non_increasing_in_slo(oracle):
    w = workloads.make(1, n_candidates=4)
    for c in range(4):
        prev = None
        for slo in [0, 20_000, 50_000, 150_000, 10 ** 9]:
            _, miss = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                          w.arrival_us, None, w.configs[c], slo)
            assert prev is None or miss <= prev
            prev = miss
        assert prev == 0


# --------------------------------------------------------------------------
# whole-simulator invariants and metamorphic relations
# --------------------------------------------------------------------------

def _cases():
    out = [workloads.random_small(s, S=4, H=3, Bmax=16, n=1500, C=6, max_replicas=6, tree=(s % 2 == 1),
                                  qps=300.0, cv=3.0, lat_lo=500, lat_hi=20000,
                                  equal_stamp_every=(4 if s == 2 else 0)) for s in range(6)]
    out.append(workloads.make(2, n_queries=2000, n_candidates=6))
    out.append(workloads.make(3, n_queries=2000, n_candidates=6))
    return out


@pytest.mark.parametrize("w", _cases(), ids=lambda w: w.name)
def test_invariants_from_dispatch_log(oracle, w):
    S = w.n_stages
    for c in range(w.n_candidates):
        cfg = w.configs[c]
        p99, miss, lat, log = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                                  w.arrival_us, w.branch_bits, cfg, w.slo_us,
                                                  want_latency=True, want_log=True)
        for s in range(S):
            L = log[log["stage"] == s]
            hw, mb, R = int(cfg[s, 0]), int(cfg[s, 1]), int(cfg[s, 2])
            assert np.all((L["batch"] >= 1) & (L["batch"] <= mb))
            assert np.all(np.diff(L["t_dispatch"]) >= 0)
            assert np.all(L["replica"] < R)
            assert np.array_equal(L["t_finish"] - L["t_dispatch"],
                                  w.latency_us[s, hw, L["batch"] - 1])
            for r in range(R):   # a replica never runs two batches at once
                Lr = L[L["replica"] == r]
                assert np.all(Lr["t_dispatch"][1:] >= Lr["t_finish"][:-1])
        # latency floor: sum over the query's path of the smallest usable table entry
        floor = np.zeros(w.n_queries, np.int64)
        reach = np.ones((S, w.n_queries), bool)
        for s in range(S):
            if s:
                reach[s] = reach[w.parent[s]]
                if w.cond_bit[s] >= 0:
                    reach[s] &= ((w.branch_bits >> w.cond_bit[s]) & 1) == w.cond_val[s]
            floor += reach[s] * int(w.latency_us[s, cfg[s, 0], :cfg[s, 1]].min())
        assert np.all(lat >= floor)
        k = rank_k(w.n_queries)
        assert (p99 <= w.slo_us) == (miss <= w.n_queries - k)


@pytest.mark.parametrize("w", _cases()[:4], ids=lambda w: w.name)
def test_time_shift_scale_and_replica_preference(oracle, w):
    args = (w.parent, w.cond_bit, w.cond_val)
    for c in range(w.n_candidates):
        cfg = w.configs[c]
        base = oracle.estimate_one(*args, w.latency_us, w.arrival_us, w.branch_bits, cfg,
                                   w.slo_us, want_latency=True)
        shifted = oracle.estimate_one(*args, w.latency_us, w.arrival_us + 123_456_789_012,
                                      w.branch_bits, cfg, w.slo_us, want_latency=True)
        assert base[0] == shifted[0] and base[1] == shifted[1]
        assert np.array_equal(base[2], shifted[2])
        scaled = oracle.estimate_one(*args, w.latency_us * 7, w.arrival_us * 7, w.branch_bits,
                                     cfg, w.slo_us * 7, want_latency=True)
        assert scaled[0] == 7 * base[0] and scaled[1] == base[1]
        assert np.array_equal(scaled[2], 7 * base[2])
        other = oracle.estimate_one(*args, w.latency_us, w.arrival_us, w.branch_bits, cfg,
                                    w.slo_us, replica_pref=1, want_latency=True)
        assert np.array_equal(base[2], other[2])


def test_more_replicas_never_hurt_without_batching(oracle):
    """Single stage, max batch 1: adding a replica cannot increase any latency."""
    rng = np.random.default_rng(5)
    a = workloads.gamma_arrivals(rng, 3000, 300.0, 4.0)
    prev = None
    for R in range(1, 9):
        topo, cfg = single_stage([11000], R=R)
        p99, _, lat = run(oracle, topo, a, cfg, want_latency=True)
        if prev is not None:
            assert np.all(lat <= prev[1]) and p99 <= prev[0]
        prev = (p99, lat)


def test_batchmates_finish_together(oracle):
    """All queries of one batch leave the stage at the same instant."""
    rng = np.random.default_rng(9)
    a = workloads.gamma_arrivals(rng, 2000, 400.0, 4.0)
    topo, cfg = single_stage([3000 + 900 * b for b in range(1, 9)], R=2, mb=8)
    _, _, lat, log = run(oracle, topo, a, cfg, want_latency=True, want_log=True)
    finish = np.sort(a + lat)
    exp = np.sort(np.repeat(log["t_finish"], log["batch"]))
    assert np.array_equal(finish, exp)


def test_many_equals_one(oracle):
    w = workloads.make(1, n_candidates=16)
    p99, miss = oracle.estimate_workload(w)
    for c in range(16):
        one = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                  None, w.configs[c], w.slo_us)
        assert (p99[c], miss[c]) == one


def test_parallel_driver_matches_serial(oracle):
    w = workloads.make(3, n_queries=1500, n_candidates=24)
    a = oracle.estimate_workload(w)
    b = oracle.estimate_many_parallel(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                      w.arrival_us, w.branch_bits, w.configs, w.slo_us,
                                      processes=2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# --------------------------------------------------------------------------
# input validation
# --------------------------------------------------------------------------

def test_rejects_bad_inputs(oracle):
    w = workloads.make(3, n_queries=50, n_candidates=1)
    ok = dict(parent=w.parent, cond_bit=w.cond_bit, cond_val=w.cond_val, latency_us=w.latency_us,
              arrival_us=w.arrival_us, branch_bits=w.branch_bits, config=w.configs[0],
              slo_us=w.slo_us)

    def code(**kw):
        a = dict(ok)
        a.update(kw)
        try:
            oracle.estimate_one(**a)
        except oracle.OracleError as e:
            return e.code
        return 0

    assert code() == 0
    bad = w.parent.copy(); bad[2] = 2
    assert code(parent=bad) == -2
    bad = w.parent.copy(); bad[2] = 0                       # three children of one stage
    assert code(parent=bad) == -2
    bad = w.cond_bit.copy(); bad[3] = 9                     # no such branch bit
    assert code(cond_bit=bad) == -2
    bad = w.latency_us.copy(); bad[1, 1, 5] = 0
    assert code(latency_us=bad) == -3
    bad = w.arrival_us.copy(); bad[10] = bad[9] - 1
    assert code(arrival_us=bad) == -4
    for col, val in [(0, 3), (1, 0), (1, 65), (2, 0), (2, 33)]:
        bad = w.configs[0].copy(); bad[1, col] = val
        assert code(config=bad) == -5
    assert code(branch_bits=None) == -1


def test_grouped_arrivals_give_the_constructed_latency_multiset(oracle):
    """Simultaneous groups of b queries, spaced apart, one replica, max batch 64: each group is one
    batch of b at every stage, so every query of it has latency sum_s table[s][b].  The oracle must
    reproduce that vector, and its P99 / miss must equal numpy's sort of it (rank ceil(0.99 n))."""
    from select_cases import SELECT_CASES, grouped_workload
    for case, (sizes, by_size, S) in SELECT_CASES.items():
        w, want = grouped_workload(sizes, by_size, S)
        n = want.shape[0]
        k = (99 * n + 99) // 100
        srt = np.sort(want)
        _, _, lat = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                        w.branch_bits, w.configs[0], 0, want_latency=True)
        assert np.array_equal(lat, want), case
        for slo in (int(srt[0]) - 1, int(srt[k - 1]), int(srt[-1])):
            w.slo_us = slo
            p99, miss = oracle.estimate_workload(w)
            assert (int(p99[0]), int(miss[0])) == (int(srt[k - 1]), int((want > slo).sum())), (case, slo)


# --------------------------------------------------------------------------
# fan-out: a query follows every edge whose condition holds and is answered
# when its last copy leaves
# --------------------------------------------------------------------------

def fan_out_workload(seed, n=60, tiny=False):
    return workloads.fan_out_small(seed, n=n, C=8, max_replicas=3, Bmax=4, tiny_times=tiny)


@pytest.mark.parametrize("seed", range(10))
def test_fan_out_tick_brute_force(oracle, seed):
    w = fan_out_workload(seed, n=40, tiny=True)
    for c in range(w.n_candidates):
        exp = tick_simulate(w, w.configs[c])
        _, _, lat = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                        w.branch_bits, w.configs[c], 40, want_latency=True)
        assert np.array_equal(lat, exp), (seed, c)


@pytest.mark.parametrize("seed", range(6))
def test_fan_out_is_the_maximum_over_its_branches(oracle, seed):
    """Branches do not interact (each queue is fed by one parent), so a pipeline 0 -> {1 -> 3, 2} gives
    every query the larger of its latencies in the two chains 0 -> 1 -> 3 and 0 -> 2 taken alone --
    and those are linear pipelines, pinned above by the tandem and Kiefer-Wolfowitz recursions."""
    w = workloads.random_small(50 + seed, S=4, H=2, Bmax=8, n=400, C=6, max_replicas=4, qps=300.0, cv=3.0,
                               lat_lo=100, lat_hi=9000, equal_stamp_every=(4 if seed % 2 else 0))
    w.parent = np.array([-1, 0, 0, 1], np.int32)
    for c in range(w.n_candidates):
        cfg = w.configs[c]
        _, _, both = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                         w.branch_bits, cfg, 0, want_latency=True)
        lin = np.array([-1, 0, 1], np.int32)
        none3, zero3 = np.full(3, -1, np.int8), np.zeros(3, np.uint8)
        _, _, a = oracle.estimate_one(lin, none3, zero3, w.latency_us[[0, 1, 3]], w.arrival_us, None,
                                      cfg[[0, 1, 3]], 0, want_latency=True)
        _, _, b = oracle.estimate_one(lin[:2], none3[:2], zero3[:2], w.latency_us[[0, 2]], w.arrival_us, None,
                                      cfg[[0, 2]], 0, want_latency=True)
        assert np.array_equal(both, np.maximum(a, b)), (seed, c)


def test_fan_out_never_queue_limit_is_the_longest_path(oracle):
    """Section 4.3: the service time is the sum of the batch-1 latencies along the LONGEST path.  With
    replicas to spare and spaced arrivals nothing queues, so every query's latency is exactly that."""
    w = fan_out_workload(3, n=50)
    w.arrival_us = np.arange(50, dtype=np.int64) * 200_000
    cfg = np.array([[1, 4, 3, 0]] * 6, np.uint8)
    d = w.latency_us[:, 1, 0].astype(np.int64)
    _, _, lat = oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                                    w.branch_bits, cfg, 0, want_latency=True)
    for q in range(50):
        paths = [d[0] + d[1] + d[3], d[0] + d[2] + d[5]]
        if w.branch_bits[q] & 1:
            paths.append(d[0] + d[2] + d[4])
        assert lat[q] == max(paths)


# --------------------------------------------------------------------------
# joins: a stage with two incoming edges takes a query when the last of the
# edges the query follows has delivered it
# --------------------------------------------------------------------------

def _one(oracle, w, cfg, **kw):
    return oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits,
                               cfg, 0, want_latency=True, join=w.join, **kw)[2]


@pytest.mark.parametrize("shape", ["diamond", "guarded", "two_joins", "skip"])
@pytest.mark.parametrize("seed", range(8))
def test_join_tick_brute_force(oracle, seed, shape):
    w = workloads.join_small(seed, n=40, C=6, max_replicas=3, Bmax=4, tiny_times=True, shape=shape)
    for c in range(w.n_candidates):
        assert np.array_equal(_one(oracle, w, w.configs[c]), tick_simulate(w, w.configs[c])), (seed, c)


@pytest.mark.parametrize("fast", [1, 2])
@pytest.mark.parametrize("seed", range(5))
def test_join_with_an_instant_branch_is_the_other_chain(oracle, seed, fast):
    """Diamond 0 -> {1, 2} -> 3 in which one branch takes 1 us and never queues (32 replicas, at most
    32 queries leave stage 0 in one instant) while the other needs at least 2 us: the slow branch always
    delivers last, so stage 3 sees exactly what it sees in the linear chain 0 -> slow -> 3, which the
    tandem recursions above pin."""
    slow = 3 - fast
    w = workloads.join_small(20 + seed, n=500, C=6, max_replicas=4, Bmax=8)
    w.latency_us = np.maximum(w.latency_us, 2)
    w.latency_us[fast] = 1
    lin = np.array([-1, 0, 1], np.int32)
    for c in range(w.n_candidates):
        cfg = w.configs[c].copy()
        cfg[fast] = (0, 1, 32, 0)
        a = _one(oracle, w, cfg)
        _, _, b = oracle.estimate_one(lin, np.full(3, -1, np.int8), np.zeros(3, np.uint8),
                                      w.latency_us[[0, slow, 3]], w.arrival_us, None, cfg[[0, slow, 3]], 0,
                                      want_latency=True)
        assert np.array_equal(a, b), (seed, c)


def test_join_never_queue_limit_is_the_longest_path(oracle):
    """Section 4.3 again: with replicas to spare and spaced arrivals the latency is the sum of batch-1
    times along the longest path, here d0 + max(d1, d2) + d3 (+ d4 behind the join)."""
    w = workloads.join_small(4, n=60, shape="guarded")
    w.arrival_us = np.arange(60, dtype=np.int64) * 200_000
    cfg = np.array([[1, 4, 3, 0]] * 5, np.uint8)
    d = w.latency_us[:, 1, 0].astype(np.int64)
    lat = _one(oracle, w, cfg)
    for q in range(60):
        mid = max(d[1], d[2]) if w.branch_bits[q] & 1 else d[1]     # bit 0 clear: stage 2 is skipped
        assert lat[q] == d[0] + mid + d[3] + d[4]


def test_join_guard_that_is_never_true_is_no_join(oracle):
    """If no query follows the second edge the join has one input and the graph is the tree without it."""
    w = workloads.join_small(9, n=300, shape="guarded")
    w.branch_bits[:] &= 0xFE                                        # bit 0 clear everywhere: nobody visits 2
    lin = np.array([-1, 0, 1, 2], np.int32)
    for c in range(4):
        a = _one(oracle, w, w.configs[c])
        _, _, b = oracle.estimate_one(lin, np.full(4, -1, np.int8), np.zeros(4, np.uint8),
                                      w.latency_us[[0, 1, 3, 4]], w.arrival_us, None, w.configs[c][[0, 1, 3, 4]],
                                      0, want_latency=True)
        assert np.array_equal(a, b)


def test_join_rejects_bad_second_parents(oracle):
    w = workloads.join_small(1, n=20)
    for p2 in ([-1, -1, -1, 1], [-1, -1, -1, 3], [-1, -1, -1, 0], [0, -1, -1, 2]):
        with pytest.raises(oracle.OracleError) as e:       # not above the first parent / not below the stage
            oracle.estimate_one(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits,
                                w.configs[0], 0, join=(p2, w.join[1], w.join[2]))
        assert e.value.code == -2
    # a third outgoing edge from stage 0
    with pytest.raises(oracle.OracleError):
        oracle.estimate_one(np.array([-1, 0, 0, 0], np.int32), w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                            w.branch_bits, w.configs[0], 0, join=w.join)
