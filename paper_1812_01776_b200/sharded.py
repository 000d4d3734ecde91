"""Candidate sharding over the GPUs of one node.

Candidates are independent of each other (every candidate is its own Estimator
run, Section 4.3), so several GPUs share a batch by taking disjoint slices of
it: profiles and trace are bound on every device, each device evaluates its
slice, and the 16 bytes per candidate come back in candidate order.  There is
no collective and no peer access on the data path.

``ShardedEstimator`` does this inside one process, one host thread per device
(the library call blocks until its device is done).  A multi-process job
(one rank per GPU, e.g. under torchrun) uses ``shard_range`` with its rank to
pick its slice and ``Estimator`` on its own device.
"""
from __future__ import annotations

import threading
from typing import List, Optional, Sequence, Tuple

import numpy as np

from .estimator import Estimator


def shard_range(total: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slice [lo, hi) of `total` units owned by `rank` of `world`:
    sizes differ by at most one, earlier ranks take the larger slices."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    base, rem = divmod(int(total), world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


class ShardedEstimator:
    """One Estimator handle per device; `estimate` splits the candidates over them."""

    def __init__(self, parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits=None,
                 devices: Optional[Sequence[int]] = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the Estimator needs a CUDA device (sm_100a); there is no CPU path")
        self.devices: List[int] = list(range(torch.cuda.device_count())) if devices is None else list(devices)
        if not self.devices:
            raise ValueError("no device given")
        self.shards = [Estimator(parent, cond_bit, cond_val, latency_us, arrival_us, branch_bits, device=d)
                       for d in self.devices]
        self.n_stages = self.shards[0].n_stages
        self.visits = self.shards[0].visits

    @classmethod
    def from_workload(cls, w, devices: Optional[Sequence[int]] = None) -> "ShardedEstimator":
        return cls(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us, w.branch_bits, devices=devices)

    def close(self) -> None:
        for est in self.shards:
            est.close()
        self.shards = []

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def estimate(self, configs: np.ndarray, slo_us: int):
        """Host arrays in and out, as Estimator.estimate: configs [n][S][4] uint8 ->
        (p99_us [n], miss [n]) int64, in the order of `configs`."""
        configs = np.ascontiguousarray(configs, dtype=np.uint8)
        n, world = configs.shape[0], len(self.shards)
        p99 = np.empty(n, dtype=np.int64)
        miss = np.empty(n, dtype=np.int64)
        errors: List[BaseException] = []

        def run(rank: int):
            lo, hi = shard_range(n, rank, world)
            if hi == lo:
                return
            try:
                a, b = self.shards[rank].estimate(configs[lo:hi], slo_us)
                p99[lo:hi] = a
                miss[lo:hi] = b
            except BaseException as exc:      # handed to the caller below
                errors.append(exc)

        if world == 1:
            run(0)
        else:
            threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
            for t in threads:
                t.start()
            for t in threads:
                t.join()
        if errors:
            raise errors[0]
        return p99, miss

    def stats(self) -> List[dict]:
        return [est.stats() for est in self.shards]
