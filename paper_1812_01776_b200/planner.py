"""InferLine's low-frequency Planner (Section 4.3) on top of the batched Estimator.

The Planner is host control flow; every feasibility question it asks is
answered by the estimator it is given -- in production ``Estimator.estimate``
(the CUDA library), in tests also the CPU oracle, so that the two plans can be
compared.  Where the paper's loops ask one question at a time and the answers
do not depend on each other, the questions are put to the estimator as ONE
batch of candidates:

* Algorithm 2 evaluates, per iteration, three actions for every model.  The
  hardware downgrade re-initialises one model on the next cheaper hardware (add
  replicas until feasible) and then minimises that model's cost locally; both
  loops walk a small grid (replicas x batch sizes of that one model).  The
  grids of all models and the two simple actions of all models go out in ONE
  call per iteration (a few hundred to a few thousand configurations, which
  cost the GPU the same one wave as a single configuration) and are then walked
  on the host;
* Algorithm 1 adds a replica to the throughput bottleneck until the Estimator
  says feasible.  Which model is the bottleneck follows from the profiles, not
  from the Estimator's answers, so the next configurations of that sequence are
  known in advance: they are evaluated a run at a time, and the first feasible
  one is taken.

Rules taken from the paper:

* Initialize (Algorithm 1): batch 1, one replica, lowest-latency hardware for
  every model.  If the service time (sum of batch-1 latencies along the longest
  path) exceeds the objective, no configuration is feasible (the prose of
  Section 4.3; the printed test in Algorithm 1 has the comparison the other way
  round).  Otherwise add a replica to the throughput bottleneck until the
  Estimator says feasible.
* Feasible: P99 <= objective.
* MinimizeCost (Algorithm 2): repeat { among the feasible results of
  IncreaseBatch (x2), RemoveReplica and DowngradeHW over all models, take the
  cheapest } until no action is feasible.  Increasing the batch never changes
  the cost, so it is taken only when nothing cheaper is feasible; it still
  makes progress (the batch grows), which is what later lets a replica go.
* Cost: sum over models of replicas x price of the model's hardware
  (Section 6, cost model).
* Throughput of a model: replicas x batch / latency[batch], divided by the
  model's scale factor s (the fraction of queries that visit it, Section 4.1),
  i.e. the pipeline input rate the model can sustain.

Ties (equal cost) are broken by model index, then by action order (remove
replica, downgrade hardware, increase batch), so that a plan is a deterministic
function of the estimator's answers.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

MAX_REPLICAS = 32

EstimateFn = Callable[[np.ndarray], Tuple[np.ndarray, np.ndarray]]


@dataclass
class PlanResult:
    feasible: bool
    config: Optional[np.ndarray]          # [S][4] uint8 (hw, max_batch, replicas, 0)
    cost: float
    p99_us: int
    estimator_calls: int                  # batched calls made
    candidates_evaluated: int             # configurations simulated in total
    steps: List[str]                      # what was done, in order
    trajectory: List[np.ndarray] = None   # configuration after Initialize and after every accepted action


class Planner:
    def __init__(self, parent, latency_us, visits, prices: Sequence[float], slo_us: int,
                 estimate: EstimateFn, feasible: Optional[Callable[[np.ndarray], np.ndarray]] = None):
        """
        parent       [S] parent stage of every stage (-1 for the root)
        latency_us   [S][H][Bmax] model profiles
        visits       [S] queries visiting each stage (il_stage_visits); visits / visits[0] is the scale factor
        prices       [H] cost per replica-hour of each hardware type
        estimate     configs [n][S][4] uint8 -> (p99_us[n], miss[n]) for the bound trace and this objective
        feasible     optional: configs -> bool[n], the same answer as p99_us <= slo_us but cheaper to get
                     (Estimator.feasible drops a candidate as soon as it is decided); the search then asks
                     only this, and `estimate` is called once, for the P99 of the final plan
        """
        self.parent = np.asarray(parent, dtype=np.int64)
        self.lat = np.asarray(latency_us, dtype=np.int64)
        self.S, self.H, self.Bmax = self.lat.shape
        self.scale = np.asarray(visits, dtype=np.float64) / float(visits[0])
        self.prices = np.asarray(prices, dtype=np.float64)
        assert self.prices.shape == (self.H,)
        self.slo_us = int(slo_us)
        self._estimate = estimate
        self._feasible = feasible
        self.calls = 0
        self.evaluated = 0
        self.batches = [b for b in (1 << np.arange(7)) if b <= self.Bmax]

    # ---- helpers -----------------------------------------------------------

    def feasible_many(self, configs: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
        configs = np.ascontiguousarray(configs, dtype=np.uint8)
        if configs.shape[0] == 0:
            return np.zeros(0, bool), np.zeros(0, np.int64)
        self.calls += 1
        self.evaluated += configs.shape[0]
        if self._feasible is not None:
            return np.asarray(self._feasible(configs), dtype=bool), np.full(configs.shape[0], -1, np.int64)
        p99, _ = self._estimate(configs)
        p99 = np.asarray(p99, dtype=np.int64)
        return p99 <= self.slo_us, p99

    def cost(self, cfg: np.ndarray) -> float:
        return float((cfg[:, 2].astype(np.float64) * self.prices[cfg[:, 0]]).sum())

    def service_time(self, cfg: np.ndarray) -> int:
        """Sum of batch-1 latencies along the longest root-to-leaf path."""
        best = np.zeros(self.S, dtype=np.int64)
        for s in range(self.S):
            own = int(self.lat[s, cfg[s, 0], 0])
            best[s] = own + (best[self.parent[s]] if self.parent[s] >= 0 else 0)
        return int(best.max())

    def throughput(self, cfg: np.ndarray) -> np.ndarray:
        """Pipeline input rate (queries per microsecond) each model can sustain."""
        b = cfg[:, 1].astype(np.int64)
        lat = self.lat[np.arange(self.S), cfg[:, 0], b - 1].astype(np.float64)
        cap = cfg[:, 2].astype(np.float64) * b / lat
        with np.errstate(divide="ignore"):
            return np.where(self.scale > 0, cap / self.scale, np.inf)

    def best_hardware(self, s: int) -> int:
        return int(np.argmin(self.lat[s, :, 0]))

    def next_cheaper(self, hw: int) -> Optional[int]:
        cheaper = [h for h in range(self.H) if self.prices[h] < self.prices[hw]]
        if not cheaper:
            return None
        return max(cheaper, key=lambda h: (self.prices[h], -h))   # the next price level down

    # ---- Algorithm 1 -------------------------------------------------------

    def initialize(self, steps: List[str]) -> Optional[np.ndarray]:
        cfg = np.zeros((self.S, 4), dtype=np.uint8)
        for s in range(self.S):
            cfg[s] = (self.best_hardware(s), 1, 1, 0)
        if self.service_time(cfg) > self.slo_us:
            steps.append("initialize: service time exceeds the objective")
            return None
        while True:
            # the next configurations of the sequence "add a replica to the bottleneck", this one first
            run = [cfg.copy()]
            stuck = False
            while len(run) < self.INIT_RUN:
                nxt = self._grow_bottleneck(run[-1])
                if nxt is None:
                    stuck = True
                    break
                run.append(nxt)
            ok, _ = self.feasible_many(np.stack(run))
            hit = np.nonzero(ok)[0]
            if hit.size:
                cfg = run[int(hit[0])]
                steps.append(f"initialize: feasible with replicas {cfg[:, 2].tolist()}")
                return cfg
            nxt = None if stuck else self._grow_bottleneck(run[-1])
            if nxt is None:
                steps.append("initialize: every model at the replica limit, still infeasible")
                return None
            cfg = nxt

    INIT_RUN = 32      # configurations of the Initialize sequence evaluated per call

    def _grow_bottleneck(self, cfg: np.ndarray) -> Optional[np.ndarray]:
        """cfg with one more replica for the throughput bottleneck among the models that can still grow."""
        thr = self.throughput(cfg)
        for s in np.argsort(thr, kind="stable"):
            if cfg[s, 2] < MAX_REPLICAS:
                new = cfg.copy()
                new[s, 2] += 1
                return new
        return None

    # ---- Algorithm 2 -------------------------------------------------------

    def _downgrade_grid(self, cfg: np.ndarray, s: int) -> Optional[Tuple[int, np.ndarray]]:
        """Every (batch, replicas) of model s on the next cheaper hardware, other models as in cfg."""
        hw = self.next_cheaper(int(cfg[s, 0]))
        if hw is None:
            return None
        grid = np.repeat(cfg[None], len(self.batches) * MAX_REPLICAS, axis=0)
        k = 0
        for b in self.batches:
            for r in range(1, MAX_REPLICAS + 1):
                grid[k, s] = (hw, b, r, 0)
                k += 1
        return hw, grid

    def _downgrade_pick(self, cfg: np.ndarray, s: int, hw: int, ok: np.ndarray) -> Optional[np.ndarray]:
        """Model s on hardware hw, other models frozen: initialise (batch 1, add
        replicas until feasible), then minimise locally (increase batch / remove
        replica while feasible), walking the grid's answers.  Accepted only if cheaper."""
        ok = ok.reshape(len(self.batches), MAX_REPLICAS)
        # initialise: batch 1, replicas 1, 2, ... until feasible
        feas_r = np.nonzero(ok[0])[0]
        if feas_r.size == 0:
            return None
        bi, r = 0, int(feas_r[0]) + 1
        # local minimisation: remove a replica if that stays feasible, else double the batch if that does
        while True:
            if r > 1 and ok[bi, r - 2]:
                r -= 1
            elif bi + 1 < len(self.batches) and ok[bi + 1, r - 1]:
                bi += 1
            else:
                break
        new = cfg.copy()
        new[s] = (hw, self.batches[bi], r, 0)
        return new if self.cost(new) < self.cost(cfg) else None

    def _downgrade(self, cfg: np.ndarray, s: int) -> Optional[np.ndarray]:
        """The downgrade action of model s, with a call of its own."""
        g = self._downgrade_grid(cfg, s)
        if g is None:
            return None
        ok, _ = self.feasible_many(g[1])
        return self._downgrade_pick(cfg, s, g[0], ok)

    def minimize_cost(self) -> PlanResult:
        steps: List[str] = []
        cfg = self.initialize(steps)
        if cfg is None:
            return PlanResult(False, None, float("inf"), -1, self.calls, self.evaluated, steps, [])
        trajectory = [cfg.copy()]
        while True:
            # one call per iteration: the simple actions of every model and every model's downgrade grid
            simple, simple_labels, simple_model, grids = [], [], [], {}
            for s in range(self.S):
                if cfg[s, 2] > 1:
                    new = cfg.copy(); new[s, 2] -= 1
                    simple.append(new); simple_labels.append(f"remove replica of model {s}"); simple_model.append((s, 0))
                if int(cfg[s, 1]) * 2 <= self.Bmax:
                    new = cfg.copy(); new[s, 1] = int(cfg[s, 1]) * 2
                    simple.append(new); simple_labels.append(f"double batch of model {s} to {int(new[s, 1])}")
                    simple_model.append((s, 2))
                g = self._downgrade_grid(cfg, s)
                if g is not None:
                    grids[s] = g
            if not simple and not grids:
                break
            parts = ([np.stack(simple)] if simple else []) + [grids[s][1] for s in sorted(grids)]
            ok, _ = self.feasible_many(np.concatenate(parts))
            # candidates in the order (model, remove replica, downgrade, double batch), as ties are broken
            cands = []
            at = len(simple)
            downs = {}
            for s in sorted(grids):
                n_grid = grids[s][1].shape[0]
                downs[s] = self._downgrade_pick(cfg, s, grids[s][0], ok[at:at + n_grid])   # feasible by construction
                at += n_grid
            for s in range(self.S):
                for i, (m, kind) in enumerate(simple_model):
                    if m == s and kind == 0 and ok[i]:
                        cands.append((simple[i], simple_labels[i]))
                if downs.get(s) is not None:
                    d = downs[s]
                    cands.append((d, f"downgrade model {s} to hw {int(d[s, 0])} "
                                     f"(batch {int(d[s, 1])}, replicas {int(d[s, 2])})"))
                for i, (m, kind) in enumerate(simple_model):
                    if m == s and kind == 2 and ok[i]:
                        cands.append((simple[i], simple_labels[i]))
            best = None
            for i in range(len(cands)):
                if best is None or self.cost(cands[i][0]) < self.cost(cands[best][0]):
                    best = i
            if best is None:
                break
            cfg = cands[best][0]
            trajectory.append(cfg.copy())
            steps.append(f"{cands[best][1]} -> cost {self.cost(cfg):.4f}")
        p99, _ = self._estimate(np.ascontiguousarray(cfg[None], dtype=np.uint8))
        self.calls += 1
        self.evaluated += 1
        assert int(p99[0]) <= self.slo_us
        return PlanResult(True, cfg, self.cost(cfg), int(p99[0]), self.calls, self.evaluated, steps, trajectory)

    def single_actions(self, cfg: np.ndarray) -> List[np.ndarray]:
        """All configurations one action away (used to check the termination guarantee)."""
        out = []
        for s in range(self.S):
            if cfg[s, 2] > 1:
                new = cfg.copy(); new[s, 2] -= 1; out.append(new)
            if int(cfg[s, 1]) * 2 <= self.Bmax:
                new = cfg.copy(); new[s, 1] = int(cfg[s, 1]) * 2; out.append(new)
            down = self._downgrade(cfg, s)
            if down is not None:
                out.append(down)
        return out


def envelope_windows(service_time_us: int, longest_us: int = 60_000_000) -> np.ndarray:
    """Window lengths of the traffic envelope as Section 5 discretises them: the
    smallest is the pipeline's service time, then doubling up to 60 seconds."""
    out, w = [], max(1, int(service_time_us))
    while w < longest_us:
        out.append(w)
        w *= 2
    return np.array(out + [longest_us], dtype=np.int64)


def tuner_handoff(planner: Planner, cfg: np.ndarray, n_queries: int, span_us: int,
                  envelope_fn: Callable[[np.ndarray], np.ndarray]) -> dict:
    """What the Planner gives the Tuner (Section 5, "Initialization"): the
    traffic envelope of the sample trace, and per model the single-replica
    throughput mu_m and the max-provisioning ratio rho_m = lambda_m / (replicas
    x mu_m), lambda_m being the trace's mean arrival rate times the model's
    scale factor.  envelope_fn is Estimator.traffic_envelope (or the oracle's)."""
    windows = envelope_windows(planner.service_time(cfg))
    counts = np.asarray(envelope_fn(windows), dtype=np.int64)
    lam = n_queries / float(span_us)                       # queries per microsecond
    b = cfg[:, 1].astype(np.int64)
    lat = planner.lat[np.arange(planner.S), cfg[:, 0], b - 1].astype(np.float64)
    mu = b / lat                                           # one replica, queries per microsecond
    rho = lam * planner.scale / (cfg[:, 2].astype(np.float64) * mu)
    return {"window_us": windows, "max_count": counts, "rate_per_us": counts / windows.astype(np.float64),
            "mu_per_us": mu, "rho": rho, "scale_factor": planner.scale.copy()}
