#!/usr/bin/env python
"""Benchmark of the segmented-gossip synchronization round on B200.

One STEP = a workload's whole round sequence (peer selection + segment-wise
aggregation, `rounds` times, ping-pong buffers) over one batch of synthetic
parameters.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|1..5] [--impl reference]

Default (`--workload all`): the headline (`value`, `roofline`, `e2e`,
`cpu_baseline`) is the largest workload (5, BERT-large sized, fused local
step), timed over exactly K steps, and `per_workload` holds an entry for each of
the five workloads, every one timed in this same run with its own CUDA events,
clock samples and roofline fraction.  `--workload k` times workload k alone.

N > 1 (launched with torch.distributed.run): every rank runs an independent
federation replica on its own GPU (Eq. 3 needs no exchange between column
shards or replicas), times are the max over ranks, the value is the sum of all
ranks' worker-parameters over that time.
"""
from __future__ import annotations

import argparse
import datetime
import gc
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "worker_params_aggregated_per_s"
UNIT = "worker-params/s"
FALLBACK_HBM_GBS = 6650.0
NCU_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")
HEADLINE_WORKLOAD = "5"
# a per-workload timed region is stretched (by repeating the step) to at least this long, so
# that the 50 ms clock poll lands several samples inside it
MIN_REGION_S = 0.5


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="all",
                    help="all (default: headline on workload 5, per_workload entries for 1..5), "
                         "1..5 or a workload name")
    ap.add_argument("--impl", default="combo", choices=["combo", "reference"])
    ap.add_argument("--op", default="round", choices=["round", "divergence", "pull"],
                    help="round: the synchronization round (default); divergence: the Eq. 7 diagnostic alone; "
                         "pull: the worker-sharded round (workers spread over the ranks' GPUs, segments "
                         "pulled from peer memory) beside an all-reduce of the same vectors")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graphs", action="store_true", help="never replay short steps from CUDA graphs")
    ap.add_argument("--path", type=int, default=0,
                    help="0 auto, 1 direct gather, 2 staged (persistent CTAs), 5 staged (one tile per CTA); "
                         "with --op pull: 3 = nothing staged")
    ap.add_argument("--P", type=int, default=0, help="override the vector length (scaled-down runs)")
    ap.add_argument("--N", type=int, default=0, help="override the number of workers")
    ap.add_argument("--rounds", type=int, default=0, help="override the rounds per step")
    ap.add_argument("--S", type=int, default=0, help="override the number of segments")
    ap.add_argument("--R", type=int, default=-1, help="override the number of replicas (peers per segment)")
    ap.add_argument("--tile", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--warm", action="store_true",
                    help="one buffer pair only: a working set smaller than L2 stays there between steps "
                         "(the default rotates over enough pairs that every step reads HBM)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="ordinary launches instead of programmatic stream serialization")
    return ap.parse_args()


def elem_bytes(wl):
    return 4 if wl.dtype == "f32" else 2


def algorithmic_bytes_per_launch(wl):
    """Compulsory HBM traffic of one aggregation launch: every worker-parameter
    read once and written once (and its gradient read once when the local step
    is fused)."""
    e = elem_bytes(wl)
    return wl.N * wl.P * e * 2 + (wl.N * wl.P * 4 if wl.fused_sgd else 0)


def hbm_peak():
    mp = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(mp):
        try:
            return float(json.load(open(mp))["hbm_gbs"]), "measured"
        except (ValueError, KeyError):
            pass
    return FALLBACK_HBM_GBS, "fallback"


def pair_bytes_of(wl):
    return 2 * wl.N * wl.P * elem_bytes(wl)


def l2_note(wl, warm=False):
    """How the timed steps are kept from being served by the 126 MB L2 (a fact of the
    workload's size, so both arms of the benchmark print the same string)."""
    pb = pair_bytes_of(wl)
    if pb >= 512e6:
        return "inputs larger than L2 (%.2f GB in + out per round)" % (pb / 1e9)
    if warm:
        return "WARM: one buffer pair of %.0f MB, served from L2 where it fits" % (pb / 1e6)
    nsets = int(-(-512e6 // pb))
    return "rotating over %d buffer pairs (%.0f MB) so that each step reads HBM" % (nsets, nsets * pb / 1e6)


def config_of(wl, world, warm=False):
    return {"workload": wl.name, "N": wl.N, "P": wl.P, "S": wl.S, "R": wl.R, "rounds_per_step": wl.rounds,
            "weights": "sample counts" if wl.weighted else "equal", "fused_sgd": wl.fused_sgd,
            "parallelism": "replicas x%d" % world, "l2": l2_note(wl, warm)}


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """nvidia-smi polled every 50 ms in the background; samples are kept with
    their wall-clock time so that those inside a timed region can be picked."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def wait_first_sample(self, timeout=5.0):
        t0 = time.time()
        while self.proc is not None and time.time() - t0 < timeout:
            if os.path.getsize(self.tmp.name) > 0:
                return
            time.sleep(0.05)

    def _rows(self):
        rows = []
        try:
            text = open(self.tmp.name).read()
        except OSError:
            return rows
        for line in text.splitlines():
            parts = [q.strip() for q in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]),
                             [q.lower().startswith("active") for q in parts[4:8]]))
            except ValueError:
                continue
        return rows

    def window(self, t_begin: float, t_end: float):
        """Summary of the samples taken between two wall-clock times."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "power_w_max": None}
        if self.proc is None:
            return out
        time.sleep(0.12)                      # let the poller write the samples of the region's end
        rows = self._rows()
        inside = [r for r in rows if t_begin - 0.03 <= r[0] <= t_end + 0.03]
        if not inside:           # region shorter than the polling period: nearest samples
            inside = sorted(rows, key=lambda r: abs(r[0] - 0.5 * (t_begin + t_end)))[:3]
        if inside:
            out["sm_mhz"] = statistics.median(r[1] for r in inside)
            out["sm_max_mhz"] = max(r[2] for r in inside)
            out["power_w_max"] = max(r[3] for r in inside)
            out["samples"] = len(inside)
            reasons = set()
            for r in inside:
                for name, on in zip(self.NAMES, r[4]):
                    if on:
                        reasons.add(name)
            out["reasons"] = sorted(reasons)
        return out

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.close()
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        self.proc = None


# ------------------------------------------------------------------ reference arm (CPU oracle)
def oracle_inputs(wl, width):
    import numpy as np
    import torch

    from paper_1908_07782_b200 import synth

    small = wl.scaled(width)
    x = synth.make_params(small, "cpu")
    xb = x.view(torch.int16).numpy().view(np.uint16) if wl.dtype == "bf16" else x.numpy()
    grads = synth.make_grads(small, 0, "cpu").numpy() if (wl.fused_sgd and wl.dtype != "bf16") else None
    w = synth.make_weights(wl, "cpu")
    return xb, grads, (w.numpy() if w is not None else None)


def oracle_sample(wl, target_wp, threads=1):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: all N rows of
    a column slab, `reps` rounds.  With threads > 1 the slab is cut into that many column
    ranges (Eq. 3 couples workers only at equal column) and the same single-threaded oracle
    function runs on each of them at once, from a thread pool (the foreign call releases the
    interpreter lock).  Returns (worker-params/s, description, worker-params, seconds)."""
    import concurrent.futures

    import oracle

    # a slab of at most 4 M columns (memory stays bounded), repeated for as many rounds as
    # the target amount of work asks for
    width = int(min(wl.P, 4 << 20, max(1024, target_wp // wl.N)))
    xb, grads, wn = oracle_inputs(wl, width)
    reps = max(1, int(round(target_wp / float(wl.N * width))))
    oracle.select_peers(wl.sampler_seed, 0, wl.N, wl.S, wl.R)        # loads the library
    threads = max(1, min(threads, width // 1024))
    cuts = [width * i // threads for i in range(threads + 1)]
    pool = concurrent.futures.ThreadPoolExecutor(threads) if threads > 1 else None
    slabs = [(cuts[i], cuts[i + 1], xb[:, cuts[i]:cuts[i + 1]].copy() if threads > 1 else xb,
              None if grads is None else (grads[:, cuts[i]:cuts[i + 1]].copy() if threads > 1 else grads))
             for i in range(threads)]

    def run_slab(idx, sl):
        a, b, xs, gs = sl
        oracle.segment_aggregate(xs, idx, wl.S, wl.R, weights=wn, grads=gs, lr=wl.lr, P=wl.P, p_begin=a, p_end=b)

    t0 = time.perf_counter()
    for t in range(reps):
        idx = oracle.select_peers(wl.sampler_seed, t, wl.N, wl.S, wl.R)
        if pool is None:
            run_slab(idx, slabs[0])
        else:
            list(pool.map(lambda sl: run_slab(idx, sl), slabs))
    dt = time.perf_counter() - t0
    if pool is not None:
        pool.shutdown()
    wp = wl.N * width * reps
    desc = "%d round(s), all %d workers, columns [0,%d) of %d (%d worker-params)" % (
        reps, wl.N, width, wl.P, wp)
    return wp / dt, desc, wp, dt


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    per_step = 1.0e8
    for _ in range(args.warmup):
        oracle_sample(wl, per_step / 4)
    total_wp, total_t, desc = 0, 0.0, ""
    for _ in range(args.steps):
        v, desc, wp, dt = oracle_sample(wl, per_step)
        total_wp += wp
        total_t += dt
    value = total_wp / total_t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype,
        "data": "synthetic",
        "config": config_of(wl, max(args.gpus, 1)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": "each step a bounded sample: " + desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------ divergence diagnostic (extra line)
def run_divergence(args, wl):
    """Times combo_aggregation_divergence (Eq. 7) on the workload's vectors: aggregated
    models against the mean of the models the round started from (two arrays read)."""
    import torch

    import paper_1908_07782_b200 as combo
    from paper_1908_07782_b200 import synth

    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    e = elem_bytes(wl)
    x = synth.make_params(wl, dev)
    out = torch.empty_like(x)
    weights = synth.make_weights(wl, dev)
    idx = torch.empty((wl.N, wl.S, wl.R), dtype=torch.int32, device=dev)
    combo.combo_select_peers(wl.sampler_seed, 0, wl.N, wl.S, wl.R, idx)
    if wl.dtype == "bf16":
        combo.combo_segment_aggregate_bf16(x, out, weights, idx, wl.N, wl.P, wl.S, wl.R)
    else:
        combo.combo_segment_aggregate(x, out, weights, idx, wl.N, wl.P, wl.S, wl.R)
    combo.combo_set_tuning(args.tile, args.stages)
    combo.combo_set_kernel_path(args.path)
    rho = torch.empty(wl.N, dtype=torch.float64, device=dev)
    scratch = torch.empty(combo.combo_divergence_scratch_bytes(wl.N) // 8, dtype=torch.float64, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        combo.combo_aggregation_divergence(out, x, e, weights, wl.N, wl.P, rho, scratch)
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        combo.combo_aggregation_divergence(out, x, e, weights, wl.N, wl.P, rho, scratch)
    b.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    alg = 2 * wl.N * wl.P * e
    peak, src = hbm_peak()
    ach = alg / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "worker_params_measured_per_s", "op": "aggregation_divergence", "value": wl.N * wl.P / (ms * 1e-3),
        "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "P": wl.P, "arrays_read": 2,
                   "kernel_path": {1: "direct", 2: "staged"}.get(combo.combo_last_kernel_path(), "?")},
        "roofline": {"bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                     "traffic": None, "peak_source": src, "kernel": "k_divergence_staged + k_divergence_finish",
                     "algorithmic_bytes_per_launch": alg},
        "gpu_launches": 2 * args.steps, "rho_mean": float(rho.mean())}))
    return 0


# ------------------------------------------------------------------ worker-sharded round (extra line)
def run_pull(args, wl):
    """Times ShardedFederation.round: every rank hosts N/world workers in symmetric memory and
    forms their new models with combo_segment_aggregate_rows, loading the pulled segments
    from the owning GPU (Section 3).  With one rank every pull is a local load.  Beside it,
    timed the same way, the scheme the paper says Combo degrades to at R = n-1 (Section 4.3):
    an NCCL all-reduce of the same hosted vectors, each scaled by |D_j| first, which leaves
    every rank with the global weighted sum."""
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_1908_07782_b200 as combo
    from paper_1908_07782_b200 import sharding, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    e = elem_bytes(wl)
    dtype = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    weights = synth.make_weights(wl, dev)
    combo.combo_set_kernel_path(args.path)             # 3 forces the unstaged pull kernel
    combo.combo_set_tuning(args.tile, args.stages)
    fed = sharding.ShardedFederation(wl.N, wl.P, wl.S, wl.R, dtype, weights=weights)
    x = synth.make_params(wl, dev)                     # same seeds on every rank: take the hosted rows
    fed.rows().copy_(x[fed.w_begin:fed.w_end])
    del x
    stream = torch.cuda.current_stream()
    for t in range(max(args.warmup, 3)):
        fed.round(wl.sampler_seed, t)
    torch.cuda.synchronize()
    dist.barrier()
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record(stream)
    steps = args.steps
    for t in range(steps):
        fed.round(wl.sampler_seed, 100 + t)
    b.record(stream)
    torch.cuda.synchronize()
    dist.barrier()
    ms = torch.tensor([a.elapsed_time(b) / steps], device=dev, dtype=torch.float64)
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms = float(ms)
    kernel_path = combo.combo_last_kernel_path()
    combo.combo_device_status()

    # ---- the pull kernel alone (no barrier, no peer selection), for the roofline figure
    nxt = 1 - fed.cur
    def pull_only():
        combo.combo_segment_aggregate_rows(fed.row_tables[fed.cur], fed.bufs[nxt], fed.pitch, fed.elem_bytes,
                                           fed.weights, fed.idx, fed.N, fed.P, fed.S, fed.R, fed.w_begin,
                                           fed.n_local, stream=stream)
    for _ in range(3):
        pull_only()
    torch.cuda.synchronize()
    dist.barrier()
    ka = torch.cuda.Event(enable_timing=True)
    kb = torch.cuda.Event(enable_timing=True)
    ka.record(stream)
    for _ in range(steps):
        pull_only()
    kb.record(stream)
    torch.cuda.synchronize()
    dist.barrier()
    ms_k = torch.tensor([ka.elapsed_time(kb) / steps], device=dev, dtype=torch.float64)
    dist.all_reduce(ms_k, op=dist.ReduceOp.MAX)
    ms_k = float(ms_k)

    # ---- comparison arm: all-reduce of the same hosted vectors (the R = n-1 limit, Section 4.3)
    hosted = fed.rows()
    n_loc = hosted.shape[0]
    wsc = (weights[fed.w_begin:fed.w_end] if weights is not None
           else torch.ones(n_loc, device=dev)).to(hosted.dtype)
    hosted_t = hosted.t()                              # [P][n_local] view

    def allreduce_step():
        # local weighted sum of the hosted rows (in the models' storage type), then the sum over ranks
        acc = torch.mv(hosted_t, wsc)
        dist.all_reduce(acc, op=dist.ReduceOp.SUM)
        return acc

    for _ in range(3):
        allreduce_step()
    torch.cuda.synchronize()
    dist.barrier()
    a2 = torch.cuda.Event(enable_timing=True)
    b2 = torch.cuda.Event(enable_timing=True)
    a2.record(stream)
    for _ in range(steps):
        allreduce_step()
    b2.record(stream)
    torch.cuda.synchronize()
    dist.barrier()
    ms_ar = torch.tensor([a2.elapsed_time(b2) / steps], device=dev, dtype=torch.float64)
    dist.all_reduce(ms_ar, op=dist.ReduceOp.MAX)
    ms_ar = float(ms_ar)

    if rank == 0:
        idx_np = fed.idx.cpu().numpy()
        traffic = sharding.pull_traffic(idx_np, world, wl.P, e)
        link = int((traffic.sum(axis=1) - np.diag(traffic)).max())      # most any one rank pulls over NVLink
        n_local_max = -(-wl.N // world)
        if kernel_path == 4:
            # staged: the hosted rows and every distinct pulled row read once, results written once
            rows_local, rows_remote = sharding.distinct_rows_read(idx_np, world, 0, wl.P)
            alg = int((rows_local + rows_remote + n_local_max) * wl.P * e)
        else:
            alg = (wl.R + 2) * n_local_max * wl.P * e                    # per GPU: R+1 reads (no reuse), 1 write
        peak, src = hbm_peak()
        ach = alg / (ms_k * 1e-3) / 1e9
        line = {
            "metric": METRIC, "op": "worker_sharded_round", "value": wl.N * wl.P / (ms * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "strong", "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "N": wl.N, "P": wl.P, "S": wl.S, "R": wl.R,
                       "workers_per_gpu": n_local_max, "parallelism": "workers sharded x%d" % world,
                       "step": "barrier + peer selection + pull aggregation (1 round)"},
            "roofline": {"bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                         "traffic": None, "peak_source": src,
                         "kernel": {3: "k_pull_aggregate", 4: "k_pull_staged"}.get(kernel_path, "?"),
                         "avg_launch_ms": ms_k, "algorithmic_bytes_per_launch": alg,
                         "nvlink_bytes_per_round_max_rank": link,
                         "nvlink_gbs_max_rank": link / (ms_k * 1e-3) / 1e9},
            "allreduce_arm": {"what": "weighted sum of the hosted rows + NCCL all-reduce of the [P] result "
                                      "-- the R = n-1 limit of Section 4.3",
                              "ms_per_step": ms_ar, "pull_round_over_allreduce": ms / ms_ar,
                              "bytes_reduced_per_rank": e * wl.P},
            "gpu_launches": 2 * steps,
        }
        print(json.dumps(line))
    dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------ our arm
def time_workload(wl, args, dev, rank, world, sampler, steps, want_e2e):
    """Runs `steps` timed steps of one workload with device-resident inputs (CUDA events on the
    launching stream, every aggregation launch also bracketed on its own where steps are
    launched from the host), optionally the end-to-end arm, and returns the figures.  All
    device buffers are released before returning."""
    import torch
    import torch.distributed as dist

    import paper_1908_07782_b200 as combo
    from paper_1908_07782_b200 import synth

    combo.combo_set_kernel_path(args.path)
    combo.combo_set_tuning(args.tile, args.stages)
    combo.combo_set_launch_overlap(not args.no_overlap)

    # every rank: an independent replica of the workload (seed offset by rank)
    seed = 1000 * rank
    e = elem_bytes(wl)
    x0 = synth.make_params(wl, dev, seed=seed)
    # A working set that fits in L2 would be served from it on repeated steps: rotate over
    # enough independent buffer pairs that every step reads its inputs from HBM.
    pair_bytes = pair_bytes_of(wl)
    nsets = 1 if (pair_bytes >= 512e6 or args.warm) else int(-(-512e6 // pair_bytes))
    sets = [[x0, torch.empty_like(x0)]]
    for _ in range(nsets - 1):
        sets.append([x0.clone(), torch.empty_like(x0)])
    if args.warm and pair_bytes < 512e6:
        # the same pair eight times over, so that a replayed graph holds as many launches as
        # in the rotating case (a graph of one short kernel would time the graph launch)
        nsets = 8
        sets = sets * 8
    weights = synth.make_weights(wl, dev)
    grads = synth.make_grads(wl, 0, dev, seed=1000 + seed) if wl.fused_sgd else None
    idx = torch.empty((wl.N, wl.S, wl.R), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def aggregate(src, dst, st=None):
        if wl.dtype == "bf16":
            combo.combo_segment_aggregate_bf16(src, dst, weights, idx, wl.N, wl.P, wl.S, wl.R, stream=st)
        elif wl.fused_sgd:
            combo.combo_segment_aggregate_sgd(src, grads, wl.lr, dst, weights, idx, wl.N, wl.P, wl.S, wl.R,
                                              stream=st)
        else:
            combo.combo_segment_aggregate(src, dst, weights, idx, wl.N, wl.P, wl.S, wl.R, stream=st)

    agg_events = []
    step_no = [0]

    def step(record):
        bufs = sets[step_no[0] % nsets]
        step_no[0] += 1
        cur = 0
        for t in range(wl.rounds):
            combo.combo_select_peers(wl.sampler_seed + rank, t, wl.N, wl.S, wl.R, idx)
            if record:
                a = torch.cuda.Event(enable_timing=True)
                b = torch.cuda.Event(enable_timing=True)
                a.record(stream)
                aggregate(bufs[cur], bufs[1 - cur])
                b.record(stream)
                agg_events.append((a, b))
            else:
                aggregate(bufs[cur], bufs[1 - cur])
            cur = 1 - cur

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step(False)
    torch.cuda.synchronize()
    # A step that takes less than the CPU needs to launch it (workload 1: two kernels of a
    # few microseconds) is replayed from CUDA graphs, one graph per buffer pair.
    probe0 = torch.cuda.Event(enable_timing=True)
    probe1 = torch.cuda.Event(enable_timing=True)
    probe0.record(stream)
    for _ in range(3):
        step(False)
    probe1.record(stream)
    torch.cuda.synchronize()
    step_ms_est = probe0.elapsed_time(probe1) / 3.0
    use_graphs = step_ms_est < 0.3 and not args.no_graphs
    if steps is None:
        # a per-workload entry: as many steps as fill MIN_REGION_S (at least the --steps asked for)
        steps = max(args.steps, int(math.ceil(MIN_REGION_S * 1e3 / max(step_ms_est, 1e-3))))
        if use_graphs:
            steps = -(-steps // nsets) * nsets
    group_ms = None
    if use_graphs:
        gs = torch.cuda.Stream()

        def capture(body):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(gs):
                body(gs)
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=gs):
                    body(gs)
            return g

        def whole(st, pair):
            cur = 0
            for t in range(wl.rounds):
                combo.combo_select_peers(wl.sampler_seed + rank, t, wl.N, wl.S, wl.R, idx, stream=st)
                aggregate(pair[cur], pair[1 - cur], st)
                cur = 1 - cur

        def only_agg(st, pair):
            cur = 0
            for t in range(wl.rounds):
                aggregate(pair[cur], pair[1 - cur], st)
                cur = 1 - cur

        # one graph holding a step on every buffer pair (nsets steps), single-step graphs for
        # the remainder, and the same with the aggregation launches alone
        all_steps = capture(lambda st: [whole(st, pr) for pr in sets])
        all_aggs = capture(lambda st: [only_agg(st, pr) for pr in sets])
        graphs, agg_graphs = [], []
        if steps % nsets:
            for pair in sets[: steps % nsets]:
                graphs.append(capture(lambda st, pair=pair: whole(st, pair)))
                agg_graphs.append(capture(lambda st, pair=pair: only_agg(st, pair)))
        torch.cuda.synchronize()
        all_steps.replay()

        def replay_steps(big, singles):
            for _ in range(steps // nsets):
                big.replay()
            for k in range(steps % nsets):
                singles[k].replay()
    if sampler:
        sampler.wait_first_sample()
    barrier()
    t_begin = time.time()
    ev0 = torch.cuda.Event(enable_timing=True)
    ev1 = torch.cuda.Event(enable_timing=True)
    if use_graphs:
        with torch.cuda.stream(gs):
            ev0.record(gs)
            replay_steps(all_steps, graphs)
            ev1.record(gs)
            # the aggregation launches alone, same buffers, for the roofline figure: one event
            # pair per replay of the all-pairs graph (nsets * rounds launches each)
            marks = [torch.cuda.Event(enable_timing=True)]
            marks[0].record(gs)
            for _ in range(max(steps // nsets, 1)):
                all_aggs.replay()
                m = torch.cuda.Event(enable_timing=True)
                m.record(gs)
                marks.append(m)
        barrier()
        per_group = nsets * wl.rounds
        group_ms = [marks[i].elapsed_time(marks[i + 1]) / per_group for i in range(len(marks) - 1)]
        agg_ms = group_ms
    else:
        ev0.record(stream)
        for _ in range(steps):
            step(True)
        ev1.record(stream)
        barrier()
        agg_ms = [a.elapsed_time(b) for a, b in agg_events]
    ms_total = ev0.elapsed_time(ev1)
    t_end = time.time()
    clocks = sampler.window(t_begin, t_end) if sampler else None
    kernel_path = combo.combo_last_kernel_path()
    combo.combo_device_status()

    # ---- end to end: host buffers, copies inside the timed region
    e2e = None
    if want_e2e:
        bufs = sets[0]
        nbytes = wl.N * wl.P * e
        h_in = torch.empty((wl.N, wl.P), dtype=x0.dtype).pin_memory()
        h_in.copy_(x0)
        h_out = torch.empty_like(h_in).pin_memory()
        h_w = weights.cpu() if weights is not None else None
        h_g = None
        if grads is not None:
            h_g = torch.empty((wl.N, wl.P), dtype=torch.float32).pin_memory()
            h_g.copy_(grads)
        d_w = torch.empty(wl.N, device=dev) if weights is not None else None
        e2e_steps = max(1, min(steps, 5))

        def e2e_step():
            combo.combo_round_host(h_in, h_g, wl.lr, h_out, e, h_w, wl.sampler_seed + rank, 0, wl.rounds,
                                   wl.N, wl.P, wl.S, wl.R, bufs[0], grads, bufs[1], d_w, idx)
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        a = torch.cuda.Event(enable_timing=True)
        b = torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        b.record(stream)
        barrier()
        e2e_ms = max(a.elapsed_time(b), 1e3 * (time.perf_counter() - t0) if world == 1 else 0.0)
        e2e = {"ms": e2e_ms, "steps": e2e_steps,
               "h2d": nbytes * (2 if h_g is not None else 1) + (4 * wl.N if h_w is not None else 0),
               "d2h": nbytes}
        del h_in, h_out, h_g

    avg_launch_ms = sum(agg_ms) / len(agg_ms)
    # ---- max over ranks
    if world > 1:
        t = torch.tensor([ms_total, e2e["ms"] if e2e else 0.0, avg_launch_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t[0])
        if e2e:
            e2e["ms"] = float(t[1])
        avg_launch_ms = float(t[2])

    del sets, x0, grads, idx, weights
    torch.cuda.empty_cache()

    peak, peak_src = hbm_peak()
    alg = algorithmic_bytes_per_launch(wl)
    achieved = alg / (avg_launch_ms * 1e-3) / 1e9
    traffic = None
    if os.path.exists(NCU_TRAFFIC_FILE):
        try:
            rec = json.load(open(NCU_TRAFFIC_FILE)).get(wl.name)
            if rec and rec.get("valid"):
                traffic = rec["dram_bytes_per_launch"]
        except ValueError:
            pass
    wp_per_step = wl.N * wl.P * wl.rounds * world
    kernel = {1: "k_direct", 2: "k_staged", 5: "k_tile"}.get(kernel_path, "?")
    res = {
        "wl": wl, "steps": steps, "ms_total": ms_total, "value": wp_per_step * steps / (ms_total * 1e-3),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                     "kernel": kernel, "avg_launch_ms": avg_launch_ms,
                     "median_launch_ms": statistics.median(agg_ms), "min_launch_ms": min(agg_ms),
                     "launch_samples": len(agg_ms),
                     "sample_is": ("mean over one graph replay of %d launches" % (nsets * wl.rounds)) if use_graphs
                     else "one launch",
                     "algorithmic_bytes_per_launch": alg,
                     "launch": "CUDA graph replay (step shorter than its CPU launch cost)" if use_graphs
                     else "stream launches"},
        "gpu_launches": 2 * wl.rounds * steps,
        "e2e": None,
    }
    if e2e:
        res["e2e"] = {"value": wp_per_step * e2e["steps"] / (e2e["ms"] * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                      "ms_per_step": e2e["ms"] / e2e["steps"]}
    return res


def per_workload_entry(res, world):
    wl = res["wl"]
    return {"workload": wl.name, "dtype": wl.dtype, "config": config_of(wl, world), "steps": res["steps"],
            "ms_per_step": res["ms_total"] / res["steps"], "value": res["value"], "unit": UNIT,
            "roofline": res["roofline"], "clocks": res["clocks"], "gpu_launches": res["gpu_launches"]}


def main():
    args = parse_args()
    from paper_1908_07782_b200 import synth
    run_all = args.workload == "all"
    wl = synth.get_workload(HEADLINE_WORKLOAD if run_all else args.workload)
    if args.P or args.N or args.rounds or args.S or args.R >= 0:
        import dataclasses
        wl = dataclasses.replace(wl, P=args.P or wl.P, N=args.N or wl.N, rounds=args.rounds or wl.rounds,
                                 S=args.S or wl.S, R=args.R if args.R >= 0 else wl.R,
                                 name="%s@N=%d,P=%d,S=%d,R=%d" % (wl.name, args.N or wl.N, args.P or wl.P,
                                                                 args.S or wl.S, args.R if args.R >= 0 else wl.R))
        run_all = False
    if args.impl == "reference":
        return run_reference(args, wl)
    if args.op == "divergence":
        return run_divergence(args, wl)
    if args.op == "pull":
        return run_pull(args, wl)

    import torch
    import torch.distributed as dist

    import paper_1908_07782_b200 as combo

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    combo.load()
    sampler = ClockSampler(local_rank) if rank == 0 else None

    per_workload = []
    if run_all:
        # the four smaller workloads first, each in a region of its own; their buffers are
        # released before the next one starts
        for key in synth.WORKLOAD_ORDER:
            if synth.WORKLOADS[key].name == wl.name:
                continue
            r = time_workload(synth.WORKLOADS[key], args, dev, rank, world, sampler, None, False)
            per_workload.append(per_workload_entry(r, world))
            del r
            gc.collect()
            torch.cuda.empty_cache()
    head = time_workload(wl, args, dev, rank, world, sampler, args.steps, not args.no_e2e)
    if run_all:
        per_workload.append(per_workload_entry(head, world))
        order = {name: i for i, name in enumerate(synth.WORKLOAD_ORDER)}
        per_workload.sort(key=lambda d: order[d["workload"]])
    if sampler:
        sampler.stop()

    if rank == 0:
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_total"] / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": config_of(wl, world, args.warm),
            "roofline": head["roofline"],
            "gpu_launches": head["gpu_launches"],
            "clocks": head["clocks"],
        }
        if head["e2e"]:
            line["e2e"] = head["e2e"]
        if per_workload:
            line["per_workload"] = per_workload
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            v, desc, wp, dt = oracle_sample(wl, 1.0e9)
            cores = os.cpu_count() or 1
            va, desca, wpa, dta = oracle_sample(wl, 1.0e9 * min(cores, 8), threads=cores)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": desc + ", %.1f s" % dt,
                                    "all_cores": {"value": va, "unit": UNIT, "cores": cores,
                                                  "how": "the same single-threaded oracle function on %d column "
                                                         "ranges at once (thread pool)" % cores,
                                                  "sample": desca + ", %.1f s" % dta}}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
