#!/usr/bin/env python
"""Benchmark of the batched Estimator: candidate configurations evaluated per second.

One step = one pass of the whole hot path (simulation kernel + percentile
kernel) over one batch of candidates.  The headline workload is the largest
one: the 10-stage pipeline on its full 1,000,000-query trace with a seeded
16,384-candidate sample of its 262,144 candidates (drawn from the whole set).
The same JSON line carries, under "per_workload", a short measurement of each
of the other four workloads at full size.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (under torchrun) every rank evaluates its own seeded 16,384-candidate
sample against the same trace; there is no data-path collective, only a barrier
and a max over ranks of the timings.  Prints one JSON line on rank 0.
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

WORKLOAD_ID = 4          # the headline workload (the largest); --workload picks another one
SUB_BATCH = {4: 16384}   # workloads timed on a seeded sample of their candidates (full sweep: --candidates 0)
WORKLOADS = {
    1: "config1: linear 2-stage pipeline, 2,000 Poisson arrivals (100 qps), 64 candidates",
    2: "config2: linear 4-stage image pipeline, 50,000 gamma arrivals (200 qps, CV 4), 4,096 candidates",
    3: "config3: 6-stage tree with one branch point, 200,000 gamma arrivals (300 qps, CV 1), 65,536 candidates",
    4: "config4: linear 10-stage pipeline, 1,000,000 arrivals ramping 150->250 qps, 262,144 candidates",
    5: "config5: 8-stage tree with three branch points, 100,000 gamma arrivals (500 qps, CV 2), 1,048,576 candidates",
}
# Counters of the simulation kernels from ncu captures of a reduced case (traffic and instructions grow in
# proportion to the query-events processed).  Each entry names the SHA-256 of the kernel source it was taken
# from; when the source in the tree differs, the figures that depend on the capture are reported as null.
NCU_CAPTURES = {
    # whole streams (workloads 1, 2, 3, 5): 16,384 candidates x 8,000 queries of workload 2, all warp slots busy
    "des_lane_kernel": {
        "source": "paper_1812_01776_b200/csrc/des_lane_kernel.cu",
        "source_sha256": "7ced5906c1a2907bed48cee1217576a44e88a55664f1015da071eca0aecef96a",
        "dram_bytes_per_query_event": 8.84, "warp_inst_per_query_event": 6.89,
        "summary": "profiles/des_lane_kernel_config2.md"},
    # stream rings (workload 4): 3,552 candidates x 20,000 queries of workload 4, all warp slots busy
    "des_lane_kernel:rings": {
        "source": "paper_1812_01776_b200/csrc/des_lane_kernel.cu",
        "source_sha256": "7ced5906c1a2907bed48cee1217576a44e88a55664f1015da071eca0aecef96a",
        "dram_bytes_per_query_event": 8.99, "warp_inst_per_query_event": 7.68,
        "summary": "profiles/des_lane_kernel_config4_rings.md"},
    # pipelines with branch points (workloads 3, 5; a lane idles while its stage has no query): 5,920 candidates x
    # 20,000 queries of workload 3, all warp slots busy
    "des_lane_kernel:tree": {
        "source": "paper_1812_01776_b200/csrc/des_lane_kernel.cu",
        "source_sha256": "7ced5906c1a2907bed48cee1217576a44e88a55664f1015da071eca0aecef96a",
        "dram_bytes_per_query_event": 8.84, "warp_inst_per_query_event": 12.74,
        "summary": "profiles/des_lane_kernel_config3_branch_bits.md"},
    "des_packed_kernel": {
        "source": "paper_1812_01776_b200/csrc/des_packed_kernel.cu",
        "source_sha256": "",       # not captured again since the kernel got its node-stage entry and checks
        "dram_bytes_per_query_event": 12.24, "warp_inst_per_query_event": 32.9,
        "summary": "profiles/des_packed_kernel_config2.md"},
}
LANE_CTAS = None         # --lane-ctas: resident CTAs per SM of the lane kernel, for side measurements
RING_LOG2 = None         # --ring-log2: ring length of the lane kernel's streams, for side measurements
BITS_LOOKUP = False      # --bits-lookup: stages look the branch bits up instead of finding them in the records
METRIC = "candidate_configs_per_s"
UNIT = "candidates/s"


# ----------------------------------------------------------------------------
# helpers that hold no GPU work (covered by CPU tests)
# ----------------------------------------------------------------------------

from paper_1812_01776_b200.sharded import shard_range  # noqa: E402  (the package's sharding rule)


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


def ncu_capture(kernel: str, rings: bool = False, tree: bool = False):
    """The capture record of `kernel` if it still describes the source in the tree, else None."""
    import hashlib
    name = kernel.split("<")[0]
    cap = NCU_CAPTURES.get(name + ":rings") if rings else (NCU_CAPTURES.get(name + ":tree") if tree else None)
    cap = cap or NCU_CAPTURES.get(name)
    if not cap:
        return None
    try:
        with open(os.path.join(ROOT, cap["source"]), "rb") as f:
            now = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return cap if now == cap["source_sha256"] else None


def load_workload(workload_id: int, candidates, queries, seed: int = 0):
    """The workload a step runs on and the text that names it.  candidates: None = the default
    (a seeded sample for the workloads listed in SUB_BATCH, else the full set), 0 = the full set."""
    full_n, full_c = workloads.FULL_SIZES[workload_id]
    if candidates is None and queries is None and workload_id in SUB_BATCH:
        w, _ = workloads.sub_batch(workload_id, SUB_BATCH[workload_id], seed=seed)
        text = (f"{WORKLOADS[workload_id]}; timed on a seeded sample of {w.n_candidates:,} candidates "
                f"drawn from the whole set, full {w.n_queries:,}-query trace")
        return w, text
    w = workloads.make(workload_id, n_queries=queries, n_candidates=candidates or None)
    text = WORKLOADS[workload_id]
    if w.n_candidates != full_c or w.n_queries != full_n:
        text += f" [overridden: first {w.n_candidates:,} candidates, {w.n_queries:,} queries]"
    return w, text


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


def oracle_sample(w, cores: int, seconds: float = 12.0):
    """How many candidates of w the oracle is timed on per step: about `seconds` of work on
    `cores` cores (it does a few million query-events per second and core), at least one per core."""
    per_cand_s = w.query_events() / 4.5e6
    return int(max(cores, min(w.n_candidates, seconds * cores / per_cand_s)))


def run_reference(args):
    """The oracle, as it stands, on the host cores: the same workload, metric and unit as the CUDA
    arm; each step is the first oracle_sample() candidates of the batch the CUDA arm times."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    w, text = load_workload(args.workload, args.candidates, args.queries)
    cores = os.cpu_count() or 1
    import oracle
    per_step = oracle_sample(w, cores, seconds=6.0)
    pool = oracle.make_pool(cores) if cores > 1 else None
    for _ in range(min(args.warmup, 1)):
        time_oracle(w, cores, cores, pool)
    times = [time_oracle(w, per_step, cores, pool) for _ in range(args.steps)]
    if pool is not None:
        pool.terminate()
    sec = sum(times) / len(times)
    value = per_step / sec
    sample = (f"first {per_step} of the {w.n_candidates} candidates of the batch per step, "
              f"{w.n_queries}-query trace, "
              f"{cores} processes each running the single-threaded oracle on a disjoint slice")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": workload_config(w, text, world),
        "query_events_per_s": value * w.query_events(),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, text: str, world: int):
    """The `config` object: names the workload only, so that both arms print the same one."""
    return {"workload": text + (" per GPU" if world > 1 else ""),
            "candidates_per_gpu": w.n_candidates, "queries": w.n_queries, "stages": w.n_stages,
            "query_events_per_candidate": w.query_events(),
            "l2": "256 MiB buffer written between steps (L2 is 126 MB)",
            "parallelism": f"candidates sharded over {world} GPU(s), no data-path collective"}


# ----------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------

def measure(il, torch, w, dev, stream, flush, steps, warmup, e2e_steps, variant, issue_rate, peaks,
            barrier=lambda: None, sampler=None):
    """Times `steps` device-resident steps (after `warmup`) and `e2e_steps` host-buffer steps of
    workload w on this rank's GPU.  Returns the per-workload record; times are per-rank."""
    n_cand = w.n_candidates
    cfg_host = np.ascontiguousarray(w.configs)
    events_per_cand = w.query_events()
    est = il.Estimator.from_workload(w, device=dev.index)
    est.set_variant(variant)
    if RING_LOG2 is not None:
        est.set_test_knob(1, RING_LOG2)
    if LANE_CTAS is not None:
        est.set_test_knob(4, LANE_CTAS)
    if BITS_LOOKUP:
        est.set_test_knob(5, 0)
    kernel = est.kernel_name()
    ws_bytes = est.reserve_workspace(n_cand)
    cfg_pinned = torch.from_numpy(cfg_host).pin_memory()
    with torch.cuda.stream(stream):
        est.use_current_stream()
        d_cfg = cfg_pinned.to(dev, non_blocking=True)
        d_p99 = torch.empty(n_cand, dtype=torch.int64, device=dev)
        d_miss = torch.empty(n_cand, dtype=torch.int64, device=dev)

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

        for _ in range(warmup):
            one_step()
        barrier()
        if sampler is not None:
            sampler.start()
        step_ms, sim_ms, sel_ms, launches = [], [], [], 0
        st = {}
        for _ in range(steps):
            ms, st = one_step()
            step_ms.append(ms); sim_ms.append(st["sim_ms"]); sel_ms.append(st["select_ms"])
            launches += st["kernel_launches"]
        barrier()
        clocks = sampler.stop() if sampler is not None else None
        one_step_e2e()
        barrier()
        e2e_ms = []
        p99_h = miss_h = None
        for _ in range(e2e_steps):
            ms, p99_h, miss_h = one_step_e2e()
            e2e_ms.append(ms)
        barrier()
        same = bool(np.array_equal(p99_h, d_p99.cpu().numpy()) and np.array_equal(miss_h, d_miss.cpu().numpy()))
        feasible = float((p99_h <= w.slo_us).mean())
    est.close()

    n, S = w.n_queries, w.n_stages
    shared = bool(st.get("stage_runs")) and st["stage_runs"] < n_cand * S
    if shared:
        kernel = ("shared configuration prefixes: a covering set of whole candidates on des_lane_kernel "
                  "(des_node_stage_kernel, node by node, where that does not apply)")
    sim_s = statistics.mean(sim_ms) * 1e-3
    sel_s = statistics.mean(sel_ms) * 1e-3
    total_events = events_per_cand * n_cand
    rec_bytes = 12 if kernel == "des_kernel" else 8  # separate time/query streams, else one 64-bit record
    slab_bytes = 8 * n * n_cand                       # written once by the simulation, read once by the select
    stream_bytes = (events_per_cand - n) * 2 * rec_bytes * n_cand   # written once, read once
    # the lane kernel keeps its streams in rings when whole streams of all resident candidates pass 48 GiB
    rings = kernel == "des_lane_kernel" and (events_per_cand - n) * 8 * 148 * 8 * (32 // S) > 48 * 2**30
    cap = None if shared else ncu_capture(kernel, rings, tree=bool((w.cond_bit >= 0).any()))
    alu_peak = issue_rate * 32.0
    hbm_note = ("latency slab written once + every inter-stage stream record written once "
                "and read once (the streams are this design's, not the method's)")
    if shared:
        # only the simulated stage runs move data: per run its arrival stream read and its output written
        # (about 16 B per simulated query-event); the method's own count does not apply
        simulated_events = total_events * st["stage_runs"] / float(n_cand * S)
        stream_bytes = 16.0 * simulated_events
        slab_bytes = 0
        hbm_note = ("shared prefixes: about 16 B per SIMULATED query-event (stage_runs_simulated / "
                    "stage_runs_of_the_method of the method's count)")
    rec = {
        "candidates": n_cand, "queries": n, "stages": S, "query_events_per_candidate": events_per_cand,
        "kernel": kernel, "workspace_bytes": ws_bytes, "steps": steps, "warmup": warmup,
        "ms_per_step": {"mean": statistics.mean(step_ms), "median": statistics.median(step_ms),
                        "best": min(step_ms)},
        "step_ms_sum": sum(step_ms), "e2e_ms_sum": sum(e2e_ms), "e2e_steps": e2e_steps,
        "candidates_per_s": n_cand / (statistics.mean(step_ms) * 1e-3),
        "candidates_per_s_best": n_cand / (min(step_ms) * 1e-3),
        "query_events_per_s": total_events / (statistics.mean(step_ms) * 1e-3),
        "batches": st.get("batches"), "mean_batch": total_events / st["batches"] if st.get("batches") else None,
        "stage_runs_simulated": st.get("stage_runs"), "stage_runs_of_the_method": n_cand * S,
        "feasible_fraction": feasible,
        "kernel_ms": {"simulate": statistics.mean(sim_ms), "select": statistics.mean(sel_ms)},
        "gpu_launches": int(launches),
        "e2e": {"candidates_per_s": n_cand * e2e_steps / (sum(e2e_ms) * 1e-3),
                "h2d_bytes_per_step": int(cfg_host.nbytes), "d2h_bytes_per_step": int(16 * n_cand),
                "matches_device_path": same},
        "roofline": {"bound": "alu", "achieved": st["algorithmic_ops"] / sim_s / 1e12, "peak": alu_peak / 1e12,
                     "unit": "Tinteger-op/s", "frac": st["algorithmic_ops"] / sim_s / alu_peak,
                     "traffic": cap["dram_bytes_per_query_event"] * total_events if cap else None,
                     "traffic_unit": "DRAM bytes per launch (ncu capture of a reduced case, scaled by query-events)",
                     "capture": ({"summary": cap["summary"], "source_sha256": cap["source_sha256"]} if cap else
                                 "none that matches the kernel source in the tree"),
                     "kernel": kernel,
                     "peak_source": "integer-issue probe of this run (warp-inst/s x 32 lanes)",
                     "issue_peak_warp_inst_per_s": issue_rate,
                     "issue_slots_used": (cap["warp_inst_per_query_event"] * total_events / sim_s / issue_rate
                                          if cap else None)},
        "roofline_hbm": {"bound": "hbm", "kernel": kernel, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "achieved": (slab_bytes + stream_bytes) / sim_s / 1e9,
                         "frac": (slab_bytes + stream_bytes) / sim_s / 1e9 / peaks["hbm_gbs"],
                         "bytes": hbm_note,
                         "slab_only_achieved": slab_bytes / sim_s / 1e9,
                         "slab_only_frac": slab_bytes / sim_s / 1e9 / peaks["hbm_gbs"]},
        "roofline_select": {"bound": "hbm", "kernel": "select_kernel", "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "achieved": slab_bytes / sel_s / 1e9 if sel_s > 0 and not shared else None,
                            "frac": slab_bytes / sel_s / 1e9 / peaks["hbm_gbs"] if sel_s > 0 and not shared else None,
                            "bytes": "8 n per candidate, read once" if not shared else
                                     "shared prefixes: per-node top lists and a per-candidate combine instead"},
    }
    if clocks is not None:
        rec["clocks"] = clocks
    return rec


def measure_feasibility(il, torch, dev, stream, flush):
    """Feasibility-only mode against the full estimate on workload 2's shape (device-resident, best of 3
    each): its 4,096 candidates (one wave of warps: a dropped candidate leaves its lanes idle) and
    16,384 candidates of the same draw (dropped candidates make room for the next ones); and a Planner
    run on workload 2's trace whose questions are answered either way."""
    from paper_1812_01776_b200.planner import Planner
    out = {"workload": WORKLOADS[2], "batches": []}
    for n_cand in (4096, 16384):
        w = workloads.make(2, n_candidates=n_cand)
        with il.Estimator.from_workload(w, device=dev.index) as est, torch.cuda.stream(stream):
            est.reserve_workspace(w.n_candidates)
            est.use_current_stream()
            d_cfg = torch.from_numpy(w.configs).to(dev)
            d_flag = torch.empty(w.n_candidates, dtype=torch.uint8, device=dev)

            def timed(fn):
                best = None
                for _ in range(3):
                    flush.fill_(1)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream); fn(); b.record(stream); b.synchronize()
                    best = a.elapsed_time(b) if best is None else min(best, a.elapsed_time(b))
                return best
            full_ms = timed(lambda: est.estimate_device(d_cfg, w.slo_us))
            feas_ms = timed(lambda: est.feasible_device(d_cfg, w.slo_us, d_flag))
            st = est.stats()
            out["batches"].append(dict(candidates=w.n_candidates, estimate_ms=full_ms, feasible_ms=feas_ms,
                                       speedup=full_ms / feas_ms,
                                       infeasible_fraction=1.0 - float(d_flag.float().mean().item()),
                                       dropped_early=st["early_exits"]))
    w = workloads.make(2)
    with il.Estimator.from_workload(w, device=dev.index) as est, torch.cuda.stream(stream):
        est.reserve_workspace(w.n_candidates)
        est.use_current_stream()
        prices = np.array([0.90, 0.35, 0.10])
        plans = {}
        for name, feas in (("estimate", None), ("feasible", lambda c: est.feasible(c, w.slo_us))):
            pl = Planner(w.parent, w.latency_us, est.visits, prices, w.slo_us,
                         lambda c: est.estimate(c, w.slo_us), feasible=feas)
            t0 = time.perf_counter()
            res = pl.minimize_cost()
            plans[name] = {"seconds": time.perf_counter() - t0, "estimator_calls": res.estimator_calls,
                           "candidates_evaluated": res.candidates_evaluated, "cost": res.cost}
        out["planner"] = plans
        out["planner"]["same_plan"] = plans["estimate"]["cost"] == plans["feasible"]["cost"]
    return out


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

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    peaks, peaks_kind = load_measured_peaks()
    stream = torch.cuda.Stream(device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # > 126 MB of L2
    issue_rate, _ = il.il_measure_int_issue(stream.cuda_stream)
    torch.cuda.synchronize(dev)

    # every rank takes its own seeded sample (or, for a workload timed in full, its own slice)
    if args.candidates is None and args.queries is None and args.workload in SUB_BATCH:
        w, text = load_workload(args.workload, None, None, seed=rank)
    else:
        w, text = load_workload(args.workload, (args.candidates or workloads.FULL_SIZES[args.workload][1]) * world
                                if args.candidates != 0 else 0, args.queries)
        lo, hi = shard_range(w.n_candidates, rank, world)
        w.configs = np.ascontiguousarray(w.configs[lo:hi])
    e2e_steps = 1 if args.no_e2e else max(1, min(args.steps, args.e2e_steps))
    main = measure(il, torch, w, dev, stream, flush, args.steps, args.warmup, e2e_steps, args.variant,
                   issue_rate, peaks, barrier, ClockSampler(local) if rank == 0 else None)
    total_ms, e2e_total = reduce_max([main["step_ms_sum"], main["e2e_ms_sum"]], dist if world > 1 else None, dev)

    per_workload = []
    if world == 1 and not args.no_per_workload:
        for wid in (1, 2, 3, 5):
            if wid == args.workload:
                continue
            wk, tk = load_workload(wid, None, None)
            r = measure(il, torch, wk, dev, stream, flush, 3, 2, 1, args.variant, issue_rate, peaks)
            r["workload"] = tk
            for k in ("step_ms_sum", "e2e_ms_sum"):
                r.pop(k)
            per_workload.append(r)
    feas = None
    if world == 1 and not args.no_per_workload:
        feas = measure_feasibility(il, torch, dev, stream, flush)
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    K = args.steps
    n_cand = w.n_candidates
    cand_total = n_cand * world
    value = cand_total * K / (total_ms * 1e-3)
    e2e_value = cand_total * e2e_steps / (e2e_total * 1e-3)
    cfg = workload_config(w, text, world)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": args.warmup, "ms_per_step": total_ms / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": cfg,
        "launch": {"workspace_bytes": main["workspace_bytes"], "kernel_variant": args.variant,
                   "kernel": main["kernel"]},
        "ms_per_step_stats": main["ms_per_step"],
        "query_events_per_s": value * main["query_events_per_candidate"],
        "batches_per_s": main["batches"] * world / (total_ms / K * 1e-3) if main["batches"] else None,
        "mean_batch": main["mean_batch"],
        "stage_runs_simulated": main["stage_runs_simulated"],
        "stage_runs_of_the_method": main["stage_runs_of_the_method"],
        "feasible_fraction": main["feasible_fraction"],
        "kernel_ms": main["kernel_ms"],
        "roofline": main["roofline"],
        "roofline_hbm": dict(main["roofline_hbm"], peak_source=f"{peaks_kind} copy bandwidth"),
        "roofline_select": dict(main["roofline_select"], peak_source=f"{peaks_kind} copy bandwidth"),
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps,
                "h2d_bytes_per_step": main["e2e"]["h2d_bytes_per_step"],
                "d2h_bytes_per_step": main["e2e"]["d2h_bytes_per_step"],
                "matches_device_path": main["e2e"]["matches_device_path"]},
        "gpu_launches": main["gpu_launches"],
        "clocks": main.get("clocks", {}),
        "per_workload": per_workload,
        "feasible_only": feas,
    }
    if world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        n_sample = oracle_sample(w, cores)
        n_one = int(max(1, min(64, w.n_candidates, 4.0 / (w.query_events() / 4.5e6))))
        import oracle
        pool = oracle.make_pool(cores) if cores > 1 else None
        sec = time_oracle(w, n_sample, cores, pool)
        if pool is not None:
            pool.terminate()
        sec1 = time_oracle(w, n_one, 1)
        line["cpu_baseline"] = {
            "value": n_sample / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n_sample} of the {w.n_candidates} candidates of the batch, full trace, {cores} "
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
                    help="which of the five workloads the headline numbers are taken on (default 4, the largest)")
    ap.add_argument("--candidates", type=int, default=None,
                    help="candidates per GPU: the first N of the workload's draw (0: all of them); default: the "
                         "full set, or for workload 4 a seeded sample of 16,384 drawn from the whole set")
    ap.add_argument("--queries", type=int, default=None,
                    help="trace length (default: the workload's own); shorter traces are for profiler captures")
    ap.add_argument("--variant", type=int, default=0,
                    help="simulation kernel (IL_VARIANT_*): 0 the library's choice, 1 wide streams, "
                         "2 packed records with the trace staged through shared memory, 3 lane kernel, "
                         "4 packed records, one candidate per warp")
    ap.add_argument("--no-e2e", action="store_true", help="one host-buffer step only (profiler captures)")
    ap.add_argument("--e2e-steps", type=int, default=5, help="host-buffer steps timed (at most --steps)")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip the short measurements of the other workloads")
    ap.add_argument("--lane-ctas", type=int, default=None,
                    help="resident CTAs per SM of the lane kernel (side measurements; default 4)")
    ap.add_argument("--ring-log2", type=int, default=None,
                    help="largest stream ring of the lane kernel, log2 records (side measurements; default 13)")
    ap.add_argument("--bits-lookup", action="store_true",
                    help="lane kernel: stages look the queries' branch bits up by index instead of carrying them "
                         "in the stream records (side measurements)")
    args = ap.parse_args()
    global RING_LOG2, LANE_CTAS, BITS_LOOKUP
    RING_LOG2 = args.ring_log2
    LANE_CTAS = args.lane_ctas
    BITS_LOOKUP = args.bits_lookup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
