"""Sequential statement of InferLine's planning algorithm -- TEST INFRASTRUCTURE ONLY.

Algorithm 1 (Initialize) and Algorithm 2 (MinimizeCost) of Section 4.3, taken
step by step in the order the paper lists them, asking the Estimator ONE
`Feasible` question at a time.  The product's Planner batches independent
questions into one estimator call; the tests check it against this plain
version (same plan, same sequence of accepted actions).  Nothing here imports
the CUDA package or the product's Planner.

Readings (where the paper is silent or at odds with itself):
* Algorithm 1's printed test returns False when ServiceTime <= SLO; the prose
  says the problem is infeasible when the service time is GREATER than the
  SLO.  The prose is followed.
* BestHardware(model): the hardware with the lowest batch-1 latency (lowest
  index on ties).
* FindMinThru: throughput of a model = replicas x batch / latency[batch],
  divided by the model's scale factor (fraction of queries that visit it);
  the bottleneck is the smallest; a model at 32 replicas cannot grow, the next
  smallest is taken; if none can grow the pipeline is infeasible.
* `new.cost < best.cost` with best = NULL: the first feasible candidate becomes
  best; afterwards strictly cheaper ones replace it, so on equal cost the
  earlier (model, action) pair in listing order wins.
* DowngradeHW(model): the next cheaper hardware is the most expensive one
  among those strictly cheaper than the current (lowest index on equal
  price).  The other models are frozen; the model is initialised on it (batch
  1, one replica, add replicas until feasible or 32), then minimised locally
  (repeat: remove a replica if that stays feasible, else double the batch if
  that stays feasible) and the result is accepted only if it costs less than
  the configuration it started from.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

MAX_REPLICAS = 32


class SequentialPlanner:
    def __init__(self, parent, latency_us, visits, prices: Sequence[float], slo_us: int,
                 feasible_one: Callable[[np.ndarray], bool]):
        """feasible_one(config [S][4] uint8) -> bool: the Estimator's answer (P99 <= objective)."""
        self.parent = [int(x) for x in parent]
        self.lat = np.asarray(latency_us, dtype=np.int64)
        self.S, self.H, self.Bmax = self.lat.shape
        self.scale = [float(v) / float(visits[0]) for v in visits]
        self.prices = [float(x) for x in prices]
        self.slo_us = int(slo_us)
        self.feasible_one = feasible_one
        self.questions = 0
        self.trajectory: List[np.ndarray] = []      # configuration after Initialize and after every accepted action

    # -- pieces the two algorithms name ---------------------------------------

    def feasible(self, cfg) -> bool:
        self.questions += 1
        return bool(self.feasible_one(np.ascontiguousarray(cfg, dtype=np.uint8)))

    def cost(self, cfg) -> float:
        return sum(int(cfg[s][2]) * self.prices[int(cfg[s][0])] for s in range(self.S))

    def service_time(self, cfg) -> int:
        longest = 0
        for leaf in range(self.S):
            t, s = 0, leaf
            while s >= 0:
                t += int(self.lat[s, int(cfg[s][0]), 0])
                s = self.parent[s]
            longest = max(longest, t)
        return longest

    def find_min_thru(self, cfg) -> Optional[int]:
        best, best_thr = None, None
        for s in range(self.S):
            if int(cfg[s][2]) >= MAX_REPLICAS:
                continue
            b = int(cfg[s][1])
            cap = int(cfg[s][2]) * b / float(self.lat[s, int(cfg[s][0]), b - 1])
            thr = cap / self.scale[s] if self.scale[s] > 0 else float("inf")
            if best is None or thr < best_thr:
                best, best_thr = s, thr
        return best

    def best_hardware(self, s: int) -> int:
        best = 0
        for h in range(1, self.H):
            if self.lat[s, h, 0] < self.lat[s, best, 0]:
                best = h
        return best

    def next_cheaper(self, hw: int) -> Optional[int]:
        pick = None
        for h in range(self.H):
            if self.prices[h] < self.prices[hw] and (pick is None or self.prices[h] > self.prices[pick]):
                pick = h
        return pick

    # -- Algorithm 1 ------------------------------------------------------------

    def initialize(self):
        cfg = np.zeros((self.S, 4), dtype=np.uint8)
        for s in range(self.S):
            cfg[s] = (self.best_hardware(s), 1, 1, 0)
        if self.service_time(cfg) > self.slo_us:
            return None
        while not self.feasible(cfg):
            s = self.find_min_thru(cfg)
            if s is None:
                return None
            cfg[s][2] += 1
        return cfg

    # -- the three actions ------------------------------------------------------

    def increase_batch(self, s: int, cfg):
        if int(cfg[s][1]) * 2 > self.Bmax:
            return None
        new = cfg.copy()
        new[s][1] = int(cfg[s][1]) * 2
        return new

    def remove_replica(self, s: int, cfg):
        if int(cfg[s][2]) <= 1:
            return None
        new = cfg.copy()
        new[s][2] -= 1
        return new

    def downgrade_hw(self, s: int, cfg):
        hw = self.next_cheaper(int(cfg[s][0]))
        if hw is None:
            return None
        new = cfg.copy()
        new[s] = (hw, 1, 1, 0)
        while not self.feasible(new):
            if int(new[s][2]) >= MAX_REPLICAS:
                return None
            new[s][2] += 1
        while True:
            if int(new[s][2]) > 1:
                trial = new.copy()
                trial[s][2] -= 1
                if self.feasible(trial):
                    new = trial
                    continue
            if int(new[s][1]) * 2 <= self.Bmax:
                trial = new.copy()
                trial[s][1] = int(new[s][1]) * 2
                if self.feasible(trial):
                    new = trial
                    continue
            break
        return new if self.cost(new) < self.cost(cfg) else None

    # -- Algorithm 2 ------------------------------------------------------------

    def minimize_cost(self):
        cfg = self.initialize()
        if cfg is None:
            return None
        self.trajectory.append(cfg.copy())
        actions = [self.increase_batch, self.remove_replica, self.downgrade_hw]
        while True:
            best = None
            for s in range(self.S):
                for action in actions:
                    new = action(s, cfg)
                    if new is None:
                        continue
                    if self.feasible(new):
                        if best is None or self.cost(new) < self.cost(best):
                            best = new
            if best is None:
                break
            cfg = best
            self.trajectory.append(cfg.copy())
        return cfg
