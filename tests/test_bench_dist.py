"""Host logic of the multi-GPU bench path, on CPU with the gloo backend and two
ranks: candidate sharding covers the set exactly once, and the timing
aggregation takes the max (and the sum) over ranks."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_dir):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import bench
    import workloads
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        r, w_, _ = bench.dist_env()
        assert (r, w_) == (rank, world)
        w = workloads.make(1, n_candidates=37 * world)
        lo, hi = bench.shard_range(w.n_candidates, rank, world)
        # each rank "evaluates" its slice: here just a checksum of the configs it owns
        local = float(w.configs[lo:hi].astype(np.int64).sum())
        tot = bench.reduce_sum([local, hi - lo], dist)
        mx = bench.reduce_max([10.0 + rank, 5.0 - rank], dist)
        np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([lo, hi, tot[0], tot[1], mx[0], mx[1]]))
    finally:
        dist.destroy_process_group()


def test_shard_range_partitions():
    import bench
    for total in (0, 1, 7, 4096, 4097):
        for world in (1, 2, 3, 8):
            parts = [bench.shard_range(total, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == total
            for a, b in zip(parts, parts[1:]):
                assert a[1] == b[0]
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_gloo(tmp_path):
    import torch.multiprocessing as mp
    import workloads
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [np.load(tmp_path / f"r{r}.npy") for r in range(world)]
    w = workloads.make(1, n_candidates=37 * world)
    assert res[0][0] == 0 and res[0][1] == res[1][0] and res[1][1] == w.n_candidates
    for r in res:
        assert r[2] == float(w.configs.astype(np.int64).sum())   # slices cover the set once
        assert r[3] == w.n_candidates
        assert r[4] == 11.0 and r[5] == 5.0                      # max over ranks


def test_reduce_helpers_without_process_group():
    import bench
    assert bench.reduce_max([1.0, 2.0]) == [1.0, 2.0]
    assert bench.reduce_sum([3.0]) == [3.0]


def test_shard_range_partitions_exactly():
    from paper_1812_01776_b200 import shard_range
    for total in (0, 1, 7, 64, 4096, 1_048_577):
        for world in (1, 2, 3, 8):
            cuts = [shard_range(total, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == total
            assert all(cuts[r][1] == cuts[r + 1][0] for r in range(world - 1))
            sizes = [hi - lo for lo, hi in cuts]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        shard_range(10, 2, 2)


@pytest.mark.gpu
def test_sharded_estimator_on_the_visible_devices(oracle):
    """The package's sharded call on however many devices this process sees (one is fine):
    results in candidate order, equal to the oracle's."""
    import torch
    import workloads
    import paper_1812_01776_b200 as il
    w = workloads.make(3, n_queries=2500, n_candidates=101)
    exp = oracle.estimate_workload(w)
    with il.ShardedEstimator.from_workload(w) as sh:
        assert len(sh.shards) == torch.cuda.device_count()
        p99, miss = sh.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])
        assert sum(s["candidates"] for s in sh.stats()) == 101
    # the same through two handles on one device: the split and the reassembly are what is tested
    with il.ShardedEstimator.from_workload(w, devices=[0, 0]) as sh:
        p99, miss = sh.estimate(w.configs, w.slo_us)
        assert np.array_equal(p99, exp[0]) and np.array_equal(miss, exp[1])
        assert [s["candidates"] for s in sh.stats()] == [51, 50]
