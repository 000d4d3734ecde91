"""Inputs that put a chosen multiset of latencies in front of the P99 / miss step, with the
multiset known by construction (no simulation needed to state it).  Shared by the oracle's pins
(CPU) and the CUDA parity tests."""
import numpy as np

import workloads


def grouped_workload(group_sizes, lat_by_size, S):
    """A linear S-stage pipeline, one replica and max batch 64 everywhere, whose queries arrive in
    simultaneous groups spaced further apart than any group takes: a group of b queries is one batch
    of b at every stage, so each of its queries has latency sum_s table[s][b] = lat_by_size[b],
    split over the stages.  This puts chosen latency multisets in front of the percentile kernel."""
    B = 64
    lat = np.ones((S, 1, B), dtype=np.int64)
    for b, v in lat_by_size.items():
        per = [v // S] * S
        per[0] += v - sum(per)
        lat[:, 0, b - 1] = per
    assert lat.min() >= 1 and lat.max() < 2 ** 31
    gap = int(lat.sum(axis=0).max()) + 7
    arr = np.concatenate([np.full(b, (g + 1) * gap, dtype=np.int64) for g, b in enumerate(group_sizes)])
    parent = np.arange(-1, S - 1, dtype=np.int32)
    cfg = np.zeros((1, S, 4), dtype=np.uint8)
    cfg[0, :, 1] = B
    cfg[0, :, 2] = 1
    want = np.concatenate([np.full(b, lat_by_size[b], dtype=np.int64) for b in group_sizes])
    w = workloads.Workload(name="groups", parent=parent, cond_bit=np.full(S, -1, np.int8),
                           cond_val=np.zeros(S, np.uint8), latency_us=lat.astype(np.int32),
                           arrival_us=arr, branch_bits=np.zeros(arr.shape[0], np.uint8), configs=cfg, slo_us=0)
    return w, want


SELECT_CASES = {
    # name: (group sizes, latency of a query in a group of b, stages)
    "n1": ([1], {1: 5}, 1),
    "all_equal_n100": ([4] * 25, {4: 777}, 1),
    "n100_k99": ([1] * 98 + [2], {1: 10, 2: 999}, 1),          # the two largest are equal: p99 = 999
    "n101_k100": ([1] * 99 + [2], {1: 10, 2: 999}, 2),
    "n100_distinct_tail": ([1] * 97 + [3], {1: 50, 3: 60}, 1),
    "duplicates": [[1 + (g * 7) % 9 for g in range(300)], {b: 1000 + 13 * (b % 4) for b in range(1, 10)}, 2],
    "above_2_32_among_small": ([1] * 180 + [5, 3, 2], {1: 40, 5: 3 * 2 ** 31 - 9, 3: 2 ** 32 + 1, 2: 2 ** 32}, 3),
    "p99_above_2_32": ([1] * 90 + [5, 3, 2], {1: 40, 5: 3 * 2 ** 31 - 9, 3: 2 ** 32 + 1, 2: 2 ** 32}, 3),
    "byte_boundaries": ([1 + g % 8 for g in range(400)], {1: 255, 2: 256, 3: 65535, 4: 65536, 5: 2 ** 24 - 1,
                                                           6: 2 ** 24, 7: 2 ** 31 - 1, 8: 257}, 1),
    # more than 4,096 latencies that agree in their bit length and the seven bits below the leading one (what a
    # radix select with a logarithmic first digit must narrow down before it can finish on a short list):
    # all equal; the rank among 1,280 equal values 2^14 above 4,640 others; the rank inside those 4,640
    "all_equal_n6400": ([64] * 100, {64: 1000003}, 1),
    "crowded_then_few": ([64] * 70 + [32] * 40 + [16] * 10,
                         {64: 2 ** 33 + 5, 32: 2 ** 33 + 5 + 2 ** 14, 16: 2 ** 33 + 8}, 6),
    "crowded_twice": ([64] * 70 + [32] + [16] * 10, {64: 2 ** 33 + 5, 32: 2 ** 33 + 5 + 2 ** 14, 16: 2 ** 33 + 8}, 6),
}
