#!/usr/bin/env python
"""Benchmark of the batched Estimator: candidate configurations evaluated per second.

One step = one pass of the whole hot path (simulation kernel + percentile
kernel) over one batch of candidates of the image-pipeline workload
(4 stages, 50,000 gamma arrivals at 200 qps with CV 4, 4,096 candidates).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (under torchrun) every rank evaluates its own 4,096-candidate slice
of an N x 4,096 seeded candidate set against the same trace; there is no
data-path collective, only a barrier and a max over ranks of the timings.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

WORKLOAD_ID = 2          # the benchmark workload; --workload picks another one for side measurements
WORKLOADS = {
    1: "config1: linear 2-stage pipeline, 2,000 Poisson arrivals (100 qps), 64 candidates",
    2: "config2: linear 4-stage image pipeline, 50,000 gamma arrivals (200 qps, CV 4), 4,096 candidates",
    3: "config3: 6-stage tree with one branch point, 200,000 gamma arrivals (300 qps, CV 1), 65,536 candidates",
    4: "config4: linear 10-stage pipeline, 1,000,000 arrivals ramping 150->250 qps, 262,144 candidates",
    5: "config5: 8-stage tree with three branch points, 100,000 gamma arrivals (500 qps, CV 2), 1,048,576 candidates",
}
# DRAM bytes (read + write) of a simulation kernel per query-event, from an ncu capture of a reduced case
# (1,024 candidates x 20,000 queries; traffic is proportional to the query-events processed).
# An entry is None whenever its kernel has changed since the capture.
NCU_DRAM_BYTES_PER_QUERY_EVENT = {"des_packed_kernel": 12.24, "des_lane_kernel": 7.37}
# Warp instructions executed per query-event (smsp__inst_executed.sum of the same captures): how many issue slots
# the kernel spends, next to the algorithmic operation count of the roofline.
NCU_WARP_INST_PER_QUERY_EVENT = {"des_packed_kernel": 32.9, "des_lane_kernel": 6.53}
METRIC = "candidate_configs_per_s"
UNIT = "candidates/s"


# ----------------------------------------------------------------------------
# helpers that hold no GPU work (covered by CPU tests)
# ----------------------------------------------------------------------------

def shard_range(total: int, rank: int, world: int):
    """Contiguous slice [lo, hi) of `total` units owned by `rank`."""
    base, rem = divmod(total, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", str(rank)))
    return rank, world, local


def reduce_max(values, dist=None, device=None):
    """Max over ranks of a list of floats (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return list(values)
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def reduce_sum(values, dist=None, device=None):
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return list(values)
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t.tolist()


def load_measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.gpu_index)],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------
# the oracle arm (CPU); also used for the cpu_baseline object
# ----------------------------------------------------------------------------

def time_oracle(w, n_sample: int, processes: int, pool=None):
    """Times the CPU oracle, as it stands, on the first n_sample candidates.
    With a pool (already started, see oracle.make_pool) the timed region holds
    only the simulation and the hand-over of inputs and results."""
    import oracle
    oracle.build()
    cfg = w.configs[:n_sample]
    t0 = time.perf_counter()
    if processes == 1:
        oracle.estimate_many(w.parent, w.cond_bit, w.cond_val, w.latency_us, w.arrival_us,
                             w.branch_bits, cfg, w.slo_us)
    else:
        oracle.estimate_many_parallel(w.parent, w.cond_bit, w.cond_val, w.latency_us,
                                      w.arrival_us, w.branch_bits, cfg, w.slo_us,
                                      processes=processes, pool=pool)
    return time.perf_counter() - t0


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    w = workloads.make(args.workload, n_queries=args.queries,
                       n_candidates=min(args.candidates or 10**9, 4096, workloads.FULL_SIZES[args.workload][1]))
    cores = os.cpu_count() or 1
    import oracle
    per_step = max(cores, min(w.n_candidates, 8 * cores))
    pool = oracle.make_pool(cores) if cores > 1 else None
    for _ in range(min(args.warmup, 1)):
        time_oracle(w, cores, cores, pool)
    times = [time_oracle(w, per_step, cores, pool) for _ in range(args.steps)]
    if pool is not None:
        pool.terminate()
    sec = sum(times) / len(times)
    value = per_step / sec
    sample = (f"first {per_step} of {workloads.FULL_SIZES[args.workload][1]} candidates per step, "
              f"{w.n_queries}-query trace, "
              f"{cores} processes each running the single-threaded oracle on a disjoint slice")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload], "sampled_candidates_per_step": per_step},
        "query_events_per_s": value * w.query_events(),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------

def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_1812_01776_b200 as il

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the Estimator")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    per_rank = args.candidates or workloads.FULL_SIZES[args.workload][1]
    w = workloads.make(args.workload, n_queries=args.queries, n_candidates=per_rank * world)
    lo, hi = shard_range(w.n_candidates, rank, world)
    cfg_host = np.ascontiguousarray(w.configs[lo:hi])
    n_cand = hi - lo
    events_per_cand = w.query_events()

    est = il.Estimator.from_workload(w, device=local)
    est.set_variant(args.variant)
    kernel = est.kernel_name()
    ws_bytes = est.reserve_workspace(n_cand)
    stream = torch.cuda.Stream(device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # > 126 MB of L2
    cfg_pinned = torch.from_numpy(cfg_host).pin_memory()
    out_pinned = torch.empty((2, n_cand), dtype=torch.int64).pin_memory()

    with torch.cuda.stream(stream):
        est.use_current_stream()
        d_cfg = cfg_pinned.to(dev, non_blocking=True)
        d_p99 = torch.empty(n_cand, dtype=torch.int64, device=dev)
        d_miss = torch.empty(n_cand, dtype=torch.int64, device=dev)

        def barrier():
            torch.cuda.synchronize(dev)
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize(dev)

        def one_step():
            """Device-resident step, timed on the library's stream; returns ms and stats."""
            flush.fill_(1)                      # evict L2 between steps (not timed)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            est.estimate_device(d_cfg, w.slo_us, d_p99, d_miss)
            b.record(stream)
            b.synchronize()
            return a.elapsed_time(b), est.stats()

        def one_step_e2e():
            """Host buffers through il_estimate: H2D of configs and D2H of results inside."""
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(dev)
            a.record(stream)
            p99, miss = il.il_estimate(est._h, cfg_pinned.numpy(), w.slo_us)
            b.record(stream)
            b.synchronize()
            return a.elapsed_time(b), p99, miss

        for _ in range(args.warmup):
            one_step()
        barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        step_ms, sim_ms, sel_ms, launches, batches, alg_ops = [], [], [], 0, 0, 0
        for _ in range(args.steps):
            ms, st = one_step()
            step_ms.append(ms); sim_ms.append(st["sim_ms"]); sel_ms.append(st["select_ms"])
            launches += st["kernel_launches"]; batches = st["batches"]; alg_ops = st["algorithmic_ops"]
        barrier()
        clocks = sampler.stop() if rank == 0 else {}
        total_ms = sum(step_ms)

        # end to end through host buffers
        one_step_e2e()
        barrier()
        e2e_ms = []
        for _ in range(1 if args.no_e2e else args.steps):
            ms, p99_h, miss_h = one_step_e2e()
            e2e_ms.append(ms)
        barrier()
        e2e_total = sum(e2e_ms)
        same = bool(np.array_equal(p99_h, d_p99.cpu().numpy()) and np.array_equal(miss_h, d_miss.cpu().numpy()))
        feasible = float((p99_h <= w.slo_us).mean())

        issue_rate, _ = il.il_measure_int_issue(stream.cuda_stream)

    total_ms, e2e_total = reduce_max([total_ms, e2e_total], dist if world > 1 else None, dev)
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    K = args.steps
    cand_total = n_cand * world
    value = cand_total * K / (total_ms * 1e-3)
    e2e_value = cand_total * (1 if args.no_e2e else K) / (e2e_total * 1e-3)
    peaks, peaks_kind = load_measured_peaks()
    sim_avg_s = (sum(sim_ms) / K) * 1e-3
    # integer-issue roofline of the simulation kernel (the dominant one)
    alu_peak = issue_rate * 32.0                     # thread-level integer ops/s, measured in this run
    alu_achieved = alg_ops / sim_avg_s
    # HBM view of the same kernel: slab written once, streams written and read once, trace once per CTA wave
    n, S = w.n_queries, w.n_stages
    rec_bytes = 12 if kernel == "des_kernel" else 8  # wide: int64 time + int32 query; else one 64-bit record
    stream_bytes = (events_per_cand - n) * 2 * rec_bytes
    hbm_bytes_per_cand = 8 * n + stream_bytes + 4 * S
    hbm_achieved = hbm_bytes_per_cand * n_cand / sim_avg_s / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": total_ms / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload] + " per GPU"
                               + ("" if not (args.candidates or args.queries) else " [candidates/queries overridden]"),
                   "candidates_per_gpu": n_cand, "queries": n, "stages": S,
                   "query_events_per_candidate": events_per_cand,
                   "l2": "256 MiB buffer written between steps; working set "
                         f"{ws_bytes / 2**30:.1f} GiB > L2",
                   "workspace_bytes": ws_bytes, "kernel_variant": args.variant, "kernel": kernel, "parallelism": f"candidates sharded over {world} GPU(s)"},
        "query_events_per_s": value * events_per_cand,
        "batches_per_s": batches * world * K / (total_ms * 1e-3) if batches else None,
        "mean_batch": events_per_cand * n_cand / batches if batches else None,
        "feasible_fraction": feasible,
        "kernel_ms": {"simulate": sum(sim_ms) / K, "select": sum(sel_ms) / K},
        "roofline": {"bound": "alu", "achieved": alu_achieved / 1e12, "peak": alu_peak / 1e12,
                     "unit": "Tinteger-op/s", "frac": alu_achieved / alu_peak,
                     "traffic": (NCU_DRAM_BYTES_PER_QUERY_EVENT[kernel] * events_per_cand * n_cand
                                 if NCU_DRAM_BYTES_PER_QUERY_EVENT.get(kernel) and args.workload == 2
                                 else None),
                     "traffic_unit": "DRAM bytes per launch (ncu capture of a reduced case, scaled by query-events)",
                     "kernel": kernel,
                     "peak_source": "integer-issue probe of this run (warp-inst/s x 32 lanes)",
                     "issue_peak_warp_inst_per_s": issue_rate,
                     "issue_slots_used": (NCU_WARP_INST_PER_QUERY_EVENT[kernel] * events_per_cand * n_cand
                                          / sim_avg_s / issue_rate
                                          if NCU_WARP_INST_PER_QUERY_EVENT.get(kernel) and args.workload == 2 else None)},
        "roofline_hbm": {"bound": "hbm", "achieved": hbm_achieved, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": hbm_achieved / peaks["hbm_gbs"],
                         "peak_source": f"{peaks_kind} copy bandwidth",
                         "kernel": kernel},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(cfg_host.nbytes),
                "d2h_bytes_per_step": int(16 * n_cand), "matches_device_path": same},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        per_cand_s = w.query_events() / 4.5e6            # the oracle does a few million query-events/s/core
        n_sample = int(max(cores, min(w.n_candidates, 16 * cores, 12.0 * cores / per_cand_s)))
        n_one = int(max(1, min(64, w.n_candidates, 4.0 / per_cand_s)))
        import oracle
        pool = oracle.make_pool(cores) if cores > 1 else None
        sec = time_oracle(w, n_sample, cores, pool)
        if pool is not None:
            pool.terminate()
        sec1 = time_oracle(w, n_one, 1)
        line["cpu_baseline"] = {
            "value": n_sample / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n_sample} of {w.n_candidates} candidates, full trace, {cores} "
                      f"processes x single-threaded oracle; 1 core on {n_one} candidates: "
                      f"{n_one / sec1:.1f} candidates/s",
            "one_core_value": n_one / sec1}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", type=int, default=WORKLOAD_ID, choices=[1, 2, 3, 4, 5],
                    help="which of the five workloads (default 2, the one the metric is quoted on)")
    ap.add_argument("--candidates", type=int, default=None,
                    help="candidates per GPU (default: the workload's 4,096); smaller values are "
                         "for profiler captures, not for reported numbers")
    ap.add_argument("--queries", type=int, default=None,
                    help="trace length (default: the workload's 50,000); for profiler captures")
    ap.add_argument("--variant", type=int, default=0,
                    help="simulation kernel (IL_VARIANT_*): 0 the library's choice, 1 wide streams, "
                         "2 packed records with the trace staged through shared memory, 3 lane kernel, "
                         "4 packed records, one candidate per warp")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer timing (profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
