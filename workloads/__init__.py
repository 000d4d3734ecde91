"""Seeded synthetic inputs for the InferLine Estimator.

This module only draws random inputs and arranges them in arrays.  It holds
none of the Estimator's arithmetic (no queueing, no latency computation, no
percentile): both the CPU oracle's tests and the CUDA path's tests feed on the
same arrays produced here, and nothing else is shared between the two.

The five workloads stand in for the paper's own traces and model profiles,
which are not public.  They keep the shapes the paper describes:

* arrivals are a renewal process whose inter-arrival times are Gamma
  distributed with mean 1/lambda and a given CV, where the paper defines
  CV = sigma^2 / mu^2 (Section 2.1, "Stochastic and Unpredictable Workloads";
  Section 6, "Workload Setup"), so the Gamma shape is 1/CV and its scale is
  CV/lambda;
* a time-varying workload ramps the rate from 150 to 250 qps (Section 7,
  Tuner sensitivity experiment);
* model profiles give a batch latency per (hardware, batch size) that grows
  roughly affinely with the batch, with a CPU-like shape (no gain from
  batching) and accelerator-like shapes (high fixed cost, low per-item cost)
  (Section 2.1, Figure "Example Model Profiles");
* pipelines are linear chains or trees with conditional edges taken by a
  subset of the queries (Section 2, pipeline motifs);
* latency objectives are 150-300 ms (Sections 1 and 7).

All times are integer microseconds.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

BASE_SEED = 181201776

#: il_stage_config field order in the last axis of ``Workload.configs``.
CFG_HW, CFG_MAX_BATCH, CFG_REPLICAS, CFG_RESERVED = 0, 1, 2, 3


@dataclass
class Workload:
    """One benchmark input set.

    parent[s]      parent stage of s (parent[0] = -1, parent[s] < s)
    cond_bit[s]    -1 if the edge parent->s is always taken, else the index of
                   the branch bit that guards it
    cond_val[s]    the edge is taken iff ((bits[q] >> cond_bit[s]) & 1) == cond_val[s]
    latency_us     int32 [S][H][Bmax]; entry (s, h, b-1) is the time stage s
                   needs for a batch of b queries on hardware type h
    arrival_us     int64 [n], non-decreasing
    branch_bits    uint8 [n]
    configs        uint8 [C][S][4] = (hw, max_batch, replicas, 0) per stage
    join           None, or (parent2, cond_bit2, cond_val2): per stage a second incoming
                   edge (parent2[s] = -1: none; else parent[s] < parent2[s] < s) and its guard
    """

    name: str
    parent: np.ndarray
    cond_bit: np.ndarray
    cond_val: np.ndarray
    latency_us: np.ndarray
    arrival_us: np.ndarray
    branch_bits: np.ndarray
    configs: np.ndarray
    slo_us: int
    recipe: Dict[str, object] = field(default_factory=dict)
    join: Optional[tuple] = None

    @property
    def n_stages(self) -> int:
        return int(self.parent.shape[0])

    @property
    def n_hw(self) -> int:
        return int(self.latency_us.shape[1])

    @property
    def max_batch(self) -> int:
        return int(self.latency_us.shape[2])

    @property
    def n_queries(self) -> int:
        return int(self.arrival_us.shape[0])

    @property
    def n_candidates(self) -> int:
        return int(self.configs.shape[0])

    def visits_per_stage(self) -> np.ndarray:
        """n_s: how many queries have stage s on their path (from the bits alone)."""
        S = self.n_stages
        reach = np.zeros((S, self.n_queries), dtype=bool)
        reach[0] = True
        for s in range(1, S):
            r = reach[self.parent[s]]
            if self.cond_bit[s] >= 0:
                r = r & (((self.branch_bits >> self.cond_bit[s]) & 1) == self.cond_val[s])
            reach[s] = r
        return reach.sum(axis=1).astype(np.int64)

    def query_events(self) -> int:
        """E = sum_s n_s: one query-event is one query served at one stage."""
        return int(self.visits_per_stage().sum())


# --------------------------------------------------------------------------
# building blocks
# --------------------------------------------------------------------------

def _rngs(config_id: int):
    ss = np.random.SeedSequence([BASE_SEED, config_id])
    return [np.random.Generator(np.random.PCG64(c)) for c in ss.spawn(4)]


def _to_us(t_seconds: np.ndarray) -> np.ndarray:
    us = np.rint(t_seconds * 1e6).astype(np.int64)
    # cumulative sums are non-decreasing already; rint keeps that
    return us


def gamma_arrivals(rng, n: int, qps: float, cv: float) -> np.ndarray:
    """Renewal arrivals with Gamma inter-arrival times, mean 1/qps, CV = var/mean^2."""
    shape = 1.0 / cv
    scale = cv / qps
    gaps = rng.gamma(shape, scale, size=n)
    return _to_us(np.cumsum(gaps))


def ramp_arrivals(rng, n: int, qps0: float, qps1: float, ramp_s: float) -> np.ndarray:
    """Non-homogeneous Poisson arrivals by thinning.

    Proposals come from a homogeneous Poisson process at max(qps0, qps1); a
    proposal at time t is kept with probability rate(t)/max rate, where rate
    ramps linearly from qps0 to qps1 over ramp_s seconds and then stays.
    Exactly n accepted arrivals are returned.
    """
    top = max(qps0, qps1)
    kept = []
    have = 0
    t0 = 0.0
    while have < n:
        m = max(1024, int((n - have) * 1.6))
        t = t0 + np.cumsum(rng.exponential(1.0 / top, size=m))
        rate = qps0 + (qps1 - qps0) * np.minimum(t, ramp_s) / ramp_s
        keep = rng.random(m) * top < rate
        kept.append(t[keep])
        have += int(keep.sum())
        t0 = float(t[-1])
    return _to_us(np.concatenate(kept)[:n])


def affine_tables(rng, S: int, H: int, Bmax: int, a_range, c_range,
                  jitter: float = 0.0) -> np.ndarray:
    """lat[s][h][b-1] = rint(a + c*b) with a, c drawn per (stage, hardware).

    a_range / c_range are (lo, hi) pairs, or per-hardware lists of pairs.
    With jitter > 0 every entry is scaled by 1 + U[-jitter, jitter] and a
    running maximum over b keeps each row non-decreasing in the batch size.
    """
    def per_hw(r):
        if isinstance(r[0], (tuple, list)):
            assert len(r) == H
            return [tuple(x) for x in r]
        return [tuple(r)] * H

    a_r, c_r = per_hw(a_range), per_hw(c_range)
    b = np.arange(1, Bmax + 1, dtype=np.float64)
    lat = np.empty((S, H, Bmax), dtype=np.float64)
    for s in range(S):
        for h in range(H):
            a = rng.uniform(*a_r[h])
            c = rng.uniform(*c_r[h])
            lat[s, h] = a + c * b
    if jitter > 0.0:
        lat *= 1.0 + rng.uniform(-jitter, jitter, size=lat.shape)
    lat = np.rint(lat)
    if jitter > 0.0:
        lat = np.maximum.accumulate(lat, axis=2)
    return np.maximum(lat, 1.0).astype(np.int32)


def _pow2_upto(m: int) -> np.ndarray:
    return np.array([1 << i for i in range(int(np.log2(m)) + 1)], dtype=np.uint8)


def uniform_candidates(rng, C: int, S: int, H: int, batches: np.ndarray,
                       max_replicas: int) -> np.ndarray:
    """Independent uniform draw per stage over hw x batches x 1..max_replicas."""
    cfg = np.zeros((C, S, 4), dtype=np.uint8)
    cfg[:, :, CFG_HW] = rng.integers(0, H, size=(C, S))
    cfg[:, :, CFG_MAX_BATCH] = batches[rng.integers(0, len(batches), size=(C, S))]
    cfg[:, :, CFG_REPLICAS] = rng.integers(1, max_replicas + 1, size=(C, S))
    return cfg


def product_candidates(rng, S: int, H: int, batches: np.ndarray, max_replicas: int,
                       per_stage: list, limit: Optional[int] = None) -> np.ndarray:
    """Full Cartesian product of seeded per-stage subsets of the grid.

    Stage s keeps per_stage[s] distinct (hw, max_batch, replicas) triples drawn
    without replacement from the grid; candidates enumerate the product with
    stage 0 as the fastest-varying digit.
    """
    grid = np.array([(h, b, r) for h in range(H) for b in batches
                     for r in range(1, max_replicas + 1)], dtype=np.uint8)
    subsets = [grid[rng.choice(len(grid), size=k, replace=False)] for k in per_stage]
    total = int(np.prod(per_stage))
    C = total if limit is None else min(limit, total)
    idx = np.arange(C, dtype=np.int64)
    cfg = np.zeros((C, S, 4), dtype=np.uint8)
    for s in range(S):
        digit = idx % per_stage[s]
        idx = idx // per_stage[s]
        cfg[:, s, :3] = subsets[s][digit]
    return cfg


def bernoulli_bits(rng, n: int, probs) -> np.ndarray:
    """bit i of branch_bits[q] is 1 with probability probs[i], independently."""
    bits = np.zeros(n, dtype=np.uint8)
    for i, p in enumerate(probs):
        bits |= (rng.random(n) < p).astype(np.uint8) << np.uint8(i)
    return bits


# --------------------------------------------------------------------------
# the five workloads
# --------------------------------------------------------------------------

_LINEAR = lambda S: (np.arange(-1, S - 1, dtype=np.int32),
                     np.full(S, -1, dtype=np.int8), np.zeros(S, dtype=np.uint8))

FULL_SIZES = {1: (2_000, 64), 2: (50_000, 4_096), 3: (200_000, 65_536),
              4: (1_000_000, 262_144), 5: (100_000, 1_048_576)}


def make(config_id: int, n_queries: Optional[int] = None,
         n_candidates: Optional[int] = None) -> Workload:
    """Build workload ``config_id`` (1..5).

    n_queries / n_candidates shrink the trace or the candidate set (a prefix of
    the same seeded draw for the candidates; a fresh, shorter draw of the same
    process for the trace).
    """
    n_full, c_full = FULL_SIZES[config_id]
    n = n_full if n_queries is None else int(n_queries)
    C = c_full if n_candidates is None else int(n_candidates)
    r_prof, r_arr, r_bits, r_cand = _rngs(config_id)

    if config_id == 1:
        S, H, B = 2, 2, 16
        parent, cbit, cval = _LINEAR(S)
        lat = affine_tables(r_prof, S, H, B, (1000, 20000), (200, 3000))
        arr = gamma_arrivals(r_arr, n, 100.0, 1.0)
        bits = np.zeros(n, dtype=np.uint8)
        cfg = uniform_candidates(r_cand, C, S, H, _pow2_upto(16), 4)
        slo = 150_000
        recipe = dict(topology="linear-2", arrivals="poisson 100 qps")
    elif config_id == 2:
        S, H, B = 4, 3, 32
        parent, cbit, cval = _LINEAR(S)
        lat = affine_tables(r_prof, S, H, B, (1000, 20000), (200, 3000), jitter=0.05)
        arr = gamma_arrivals(r_arr, n, 200.0, 4.0)
        bits = np.zeros(n, dtype=np.uint8)
        cfg = uniform_candidates(r_cand, C, S, H, _pow2_upto(32), 8)
        slo = 200_000
        recipe = dict(topology="linear-4", arrivals="gamma 200 qps CV=4 (shape 0.25)")
    elif config_id == 3:
        S, H, B = 6, 3, 64
        # 0 -> {1 (bit0 = 0), 3 (bit0 = 1)}; 1 -> 2; 3 -> 4 -> 5
        parent = np.array([-1, 0, 1, 0, 3, 4], dtype=np.int32)
        cbit = np.array([-1, 0, -1, 0, -1, -1], dtype=np.int8)
        cval = np.array([0, 0, 0, 1, 0, 0], dtype=np.uint8)
        lat = affine_tables(r_prof, S, H, B,
                            [(1000, 5000), (8000, 20000), (8000, 20000)],
                            [(1500, 3000), (200, 600), (200, 600)])
        arr = gamma_arrivals(r_arr, n, 300.0, 1.0)
        bits = bernoulli_bits(r_bits, n, [0.7])
        cfg = uniform_candidates(r_cand, C, S, H, _pow2_upto(64), 8)
        slo = 250_000
        recipe = dict(topology="tree-6: 0->{1,3} on bit 0 (P=0.7 takes 3); 1->2; 3->4->5",
                      arrivals="gamma 300 qps CV=1")
    elif config_id == 4:
        S, H, B = 10, 4, 64
        parent, cbit, cval = _LINEAR(S)
        lat = affine_tables(r_prof, S, H, B, (1000, 20000), (200, 3000))
        arr = ramp_arrivals(r_arr, n, 150.0, 250.0, 5000.0)
        bits = np.zeros(n, dtype=np.uint8)
        cfg = uniform_candidates(r_cand, C, S, H, _pow2_upto(64), 16)
        slo = 300_000
        recipe = dict(topology="linear-10", arrivals="NHPP ramp 150->250 qps over 5000 s, thinning")
    elif config_id == 5:
        S, H, B = 8, 4, 64
        # 0 -> {1, 2} on bit 0; 1 -> {3, 4} on bit 1; 2 -> {5, 6} on bit 2; 3 -> 7
        parent = np.array([-1, 0, 0, 1, 1, 2, 2, 3], dtype=np.int32)
        cbit = np.array([-1, 0, 0, 1, 1, 2, 2, -1], dtype=np.int8)
        cval = np.array([0, 0, 1, 0, 1, 0, 1, 0], dtype=np.uint8)
        lat = affine_tables(r_prof, S, H, B, (1000, 20000), (200, 3000))
        arr = gamma_arrivals(r_arr, n, 500.0, 2.0)
        bits = bernoulli_bits(r_bits, n, [0.5, 0.3, 0.7])
        cfg = product_candidates(r_cand, S, H, _pow2_upto(64), 32,
                                 [8, 8, 8, 8, 4, 4, 4, 4], limit=C)
        slo = 200_000
        recipe = dict(topology="tree-8: 0->{1,2} bit0; 1->{3,4} bit1; 2->{5,6} bit2; 3->7",
                      arrivals="gamma 500 qps CV=2 (shape 0.5)")
    else:
        raise ValueError("config_id must be 1..5")

    recipe.update(seed=[BASE_SEED, config_id], n_queries=n, n_candidates=int(cfg.shape[0]))
    return Workload(name=f"config{config_id}", parent=parent, cond_bit=cbit, cond_val=cval,
                    latency_us=np.ascontiguousarray(lat), arrival_us=np.ascontiguousarray(arr),
                    branch_bits=np.ascontiguousarray(bits), configs=np.ascontiguousarray(cfg),
                    slo_us=slo, recipe=recipe)


def fan_out_small(seed: int, n: int = 900, C: int = 30, max_replicas: int = 4, Bmax: int = 8,
                  tiny_times: bool = False) -> Workload:
    """A small pipeline with fan-out (Section 2: parallel branches of a DAG): 0 -> {1, 2} both
    unconditional; 1 -> 3; 2 -> {4 if bit 0 is 1, 5 always}.  Every query visits stages 0, 1, 2, 3, 5;
    those with bit 0 set also stage 4."""
    w = random_small(seed, S=6, H=2, Bmax=Bmax, n=n, C=C, max_replicas=max_replicas, tree=False,
                     qps=80_000.0 if tiny_times else 300.0, cv=2.0, lat_lo=1,
                     lat_hi=30 if tiny_times else 9000, equal_stamp_every=(3 if seed % 2 == 0 else 0))
    w.parent = np.array([-1, 0, 0, 1, 2, 2], np.int32)
    w.cond_bit = np.array([-1, -1, -1, -1, 0, -1], np.int8)
    w.cond_val = np.array([0, 0, 0, 0, 1, 0], np.uint8)
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, 98, seed])))
    w.branch_bits = rng.integers(0, 4, n).astype(np.uint8)
    w.name = f"fanout{seed}"
    return w


def join_small(seed: int, n: int = 900, C: int = 30, max_replicas: int = 4, Bmax: int = 8,
               tiny_times: bool = False, shape: str = "diamond") -> Workload:
    """A small pipeline with a join (Section 2: a DAG in which a model consumes two models' outputs).

    diamond     0 -> {1, 2} -> 3: every query runs 1 and 2 in parallel and enters 3 when both are done.
    guarded     0 -> {1, 2 if bit 0 is 1}; 3 joins 1 and 2; 3 -> 4.  A query with bit 0 clear reaches 3
                through stage 1 alone.
    two_joins   0 -> {1, 2}; 3 joins 1 and 2; 1 is a fork as well: 1 -> {3, 4 if bit 1 is 1}; 5 joins 3 and 4
                (the second edge, 4 -> 5, only exists for queries that visited 4).
    skip        0 -> 1 -> 2 with a skip connection 0 -> 2 (guarded by bit 1): stage 2 joins 0 and 1; 2 -> 3."""
    S = {"diamond": 4, "guarded": 5, "two_joins": 6, "skip": 4}[shape]
    w = random_small(seed, S=S, H=2, Bmax=Bmax, n=n, C=C, max_replicas=max_replicas, tree=False,
                     qps=80_000.0 if tiny_times else 300.0, cv=2.0, lat_lo=1,
                     lat_hi=30 if tiny_times else 9000, equal_stamp_every=(3 if seed % 2 == 0 else 0))
    if shape == "diamond":
        w.parent = np.array([-1, 0, 0, 1], np.int32)
        w.cond_bit = np.array([-1, -1, -1, -1], np.int8)
        w.cond_val = np.zeros(4, np.uint8)
        w.join = (np.array([-1, -1, -1, 2], np.int32), np.full(4, -1, np.int8), np.zeros(4, np.uint8))
    elif shape == "guarded":
        w.parent = np.array([-1, 0, 0, 1, 3], np.int32)
        w.cond_bit = np.array([-1, -1, 0, -1, -1], np.int8)
        w.cond_val = np.array([0, 0, 1, 0, 0], np.uint8)
        w.join = (np.array([-1, -1, -1, 2, -1], np.int32), np.full(5, -1, np.int8), np.zeros(5, np.uint8))
    elif shape == "skip":
        w.parent = np.array([-1, 0, 0, 2], np.int32)
        w.cond_bit = np.array([-1, -1, 1, -1], np.int8)
        w.cond_val = np.array([0, 0, 1, 0], np.uint8)
        w.join = (np.array([-1, -1, 1, -1], np.int32), np.full(4, -1, np.int8), np.zeros(4, np.uint8))
    else:
        w.parent = np.array([-1, 0, 0, 1, 1, 3], np.int32)
        w.cond_bit = np.array([-1, -1, -1, -1, 1, -1], np.int8)
        w.cond_val = np.array([0, 0, 0, 0, 1, 0], np.uint8)
        w.join = (np.array([-1, -1, -1, 2, -1, 4], np.int32), np.full(6, -1, np.int8), np.zeros(6, np.uint8))
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, 97, seed])))
    w.branch_bits = rng.integers(0, 4, n).astype(np.uint8)
    w.name = f"join_{shape}{seed}"
    return w


def sub_batch(config_id: int, size: int, seed: int = 0, n_queries: Optional[int] = None):
    """A seeded sample of ``size`` distinct candidates of workload ``config_id``,
    drawn from its WHOLE candidate set (not a prefix of it), in increasing
    candidate order.  Returns the workload restricted to the sample and the
    sampled candidate indices."""
    w = make(config_id, n_queries=n_queries)
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, config_id, 7, seed])))
    idx = np.sort(rng.choice(w.n_candidates, size=min(size, w.n_candidates), replace=False))
    w.configs = np.ascontiguousarray(w.configs[idx])
    w.recipe.update(sub_batch=dict(size=int(idx.shape[0]), seed=seed))
    return w, idx


def random_small(seed: int, S: int = 3, H: int = 2, Bmax: int = 8, n: int = 200,
                 C: int = 16, max_replicas: int = 4, tree: bool = False,
                 qps: float = 200.0, cv: float = 2.0, lat_lo: int = 1, lat_hi: int = 20000,
                 equal_stamp_every: int = 0) -> Workload:
    """A small random workload for property tests: arbitrary (non-monotone)
    integer tables, optional random tree with conditional edges and optional
    runs of equal arrival stamps."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, 99, seed])))
    if tree:
        parent = np.full(S, -1, dtype=np.int32)
        cbit = np.full(S, -1, dtype=np.int8)
        cval = np.zeros(S, dtype=np.uint8)
        kids = {0: []}
        next_bit = 0
        for s in range(1, S):
            # parents may have: no child; one child (unconditional or guarded,
            # i.e. a cascade); two children guarded by the two values of one bit
            cands = [p for p in range(s) if len(kids[p]) == 0
                     or (len(kids[p]) == 1 and cbit[kids[p][0]] >= 0)]
            p = int(rng.choice(cands))
            parent[s] = p
            if len(kids[p]) == 1:
                sib = kids[p][0]
                cbit[s] = cbit[sib]
                cval[s] = 1 - cval[sib]
            elif rng.random() < 0.6 and next_bit < 8:
                cbit[s] = next_bit
                cval[s] = rng.integers(0, 2)
                next_bit += 1
            kids[p].append(s)
            kids[s] = []
        bits = rng.integers(0, 256, size=n).astype(np.uint8)
    else:
        parent, cbit, cval = _LINEAR(S)
        bits = np.zeros(n, dtype=np.uint8)
    lat = rng.integers(lat_lo, lat_hi + 1, size=(S, H, Bmax)).astype(np.int32)
    arr = gamma_arrivals(rng, n, qps, cv)
    if equal_stamp_every > 1:
        arr = arr[(np.arange(n) // equal_stamp_every) * equal_stamp_every]
    cfg = np.zeros((C, S, 4), dtype=np.uint8)
    cfg[:, :, CFG_HW] = rng.integers(0, H, size=(C, S))
    cfg[:, :, CFG_MAX_BATCH] = rng.integers(1, Bmax + 1, size=(C, S))
    cfg[:, :, CFG_REPLICAS] = rng.integers(1, max_replicas + 1, size=(C, S))
    return Workload(name=f"random{seed}", parent=parent, cond_bit=cbit, cond_val=cval,
                    latency_us=lat, arrival_us=arr, branch_bits=bits, configs=cfg,
                    slo_us=int(np.median(lat)) * S * 2, recipe=dict(seed=seed))
