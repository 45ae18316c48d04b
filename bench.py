#!/usr/bin/env python
"""Benchmark of the PowerGossip hot path: gossip rounds per second.

    python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]

One "step" is one gossip round (all power steps, every layer, every edge of the
round's graph) of the workload, by default the largest one: the LSTM-shaped
stack (46.5 M fp32 parameters per worker) on 32 workers with a perfect matching
re-drawn every round.  Inputs are synthetic and seeded; they are far larger
than L2, so nothing is flushed between steps.

value      rounds/s with the parameters already resident in HBM (CUDA events on
           the launching stream, max over ranks).
e2e        the same round driven through the C ABI with host buffers: every step
           uploads all parameters from pinned host memory, runs the round and
           reads all parameters back, all inside the timed region.
roofline   the kernel with the largest share of the timed region: its algorithmic
           bytes per launch (4 B per parameter it covers for every time it has
           to read or write X once) over its average launch time, measured with
           CUDA events on the launching stream inside the timed region, against
           the measured HBM copy bandwidth of this machine.
cpu_baseline the fp64 CPU checker, as it stands, on a bounded sample of the same
           workload on the host cores (reported for context only).

With --gpus N > 1 (launched under torchrun, one process per GPU) every rank runs
an independent replica of the network; there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "gossip_rounds_per_s"
UNIT = "rounds/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="lstm_matching32")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--cpu-sample-workers", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workers", type=int, default=0,
                    help="override the number of workers (smaller captures for profiling)")
    return ap.parse_args()


# ----------------------------------------------------------------------------
# machine peaks and clocks
# ----------------------------------------------------------------------------
def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ts, line in self.lines:
            if ts < t0 - 0.05 or ts > t1 + 0.15:
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# replicas: every rank runs its own network; the job's time is the slowest rank's
# ----------------------------------------------------------------------------
def max_over_ranks(ms_local: float, dist, device) -> float:
    """Largest device time over all ranks (identity without a process group)."""
    if dist is None:
        return float(ms_local)
    import torch

    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, steps: int, ms_total: float) -> float:
    """Rounds per second of all replicas together: world x steps over the slowest rank's time."""
    return world * steps / (ms_total / 1e3)


# ----------------------------------------------------------------------------
# the CPU checker as a timed baseline (bounded sample)
# ----------------------------------------------------------------------------
def time_oracle_sample(w, sample_workers: int, rounds: int, warmup: int = 1, target_seconds: float = 0.0):
    """Times the fp64 CPU checker on `sample_workers` workers of the workload.

    The cost of a round is proportional to the number of workers (every worker
    takes part in `degree` edges whatever N is), so rounds/s of the full
    workload = rounds/s of the sample x sample_workers / n_workers.
    With `target_seconds`, the number of timed rounds is chosen from the warm-up
    rounds' pace so that about that much CPU time is measured (at least `rounds`).
    Returns (scaled rounds/s, seconds timed, workers in the sample, threads, rounds timed).
    """
    from oracle import pg_oracle as po
    from paper_2008_01425_b200 import workloads as wl

    n = min(sample_workers, w.n_workers)
    if w.kind == wl.TORUS:
        sample = w.replace(n_workers=n, torus_rows=2, torus_cols=n // 2)
    else:
        sample = w.replace(n_workers=n)
    o = po.Oracle(kind=sample.kind, n_workers=sample.n_workers, layer_shapes=sample.layer_shapes,
                  rank=sample.rank, power_steps=sample.power_steps, seed=sample.seed,
                  torus_rows=sample.torus_rows, torus_cols=sample.torus_cols,
                  weight_rule=sample.weight_rule, W=wl.mixing_matrix(sample))
    for i in range(sample.n_workers):
        for l in range(len(sample.layer_shapes)):
            o.set_params(i, l, wl.initial_params(sample, i, l))
    t0 = time.perf_counter()
    o.round(max(warmup, 1))         # includes the first touch of every per-pair vector
    if target_seconds > 0.0:
        pace = (time.perf_counter() - t0) / max(warmup, 1)
        rounds = int(min(max(rounds, target_seconds / max(pace, 1e-6)), 1000))
    t0 = time.perf_counter()
    o.round(rounds)
    dt = time.perf_counter() - t0
    o.close()
    scaled = (rounds / dt) * (sample.n_workers / w.n_workers)
    return scaled, dt, sample.n_workers, po.num_threads(), rounds


# ----------------------------------------------------------------------------
def run_reference(args, w):
    """--impl reference: the CPU checker on the host cores.  Every step is one
    round on a bounded sample (4 workers) of the workload; the result is scaled
    to the full worker count."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    value, dt, n_sample, cores, _ = time_oracle_sample(w, 4, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "n_workers": w.n_workers, "rank": w.rank,
                   "power_steps": w.power_steps, "params_per_worker": w.params_per_worker},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "%d of %d workers of %s, %d timed rounds in %.1f s, scaled by workers"
                                   % (n_sample, w.n_workers, w.name, args.steps, dt)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
def main():
    args = parse_args()
    from paper_2008_01425_b200 import workloads as wl

    w = wl.by_name(args.workload)
    if args.workers:
        w = w.replace(name="%s_%dworkers" % (w.name, args.workers), n_workers=args.workers)
    if args.impl == "reference":
        run_reference(args, w)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import numpy as np
    import torch

    from paper_2008_01425_b200 import binding as pg
    from paper_2008_01425_b200 import build as pg_build

    if rank == 0:
        pg_build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    device = "cuda:%d" % local_rank
    torch.cuda.set_device(local_rank)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs: seeded synthetic stack in pinned host memory ----------------
    L = len(w.layer_shapes)
    total = w.total_params
    host = torch.empty(total, dtype=torch.float32, pin_memory=True)
    views, off = [], 0
    for i in range(w.n_workers):
        row = []
        for l, (n, m) in enumerate(w.layer_shapes):
            v = host[off:off + n * m].view(n, m)
            v.numpy()[...] = wl.initial_params(w, i, l)
            row.append(v)
            off += n * m
        views.append(row)
    back = torch.empty(total, dtype=torch.float32, pin_memory=True)
    back_views, off = [], 0
    for i in range(w.n_workers):
        row = []
        for l, (n, m) in enumerate(w.layer_shapes):
            row.append(back[off:off + n * m].view(n, m))
            off += n * m
        back_views.append(row)

    net = pg.PowerGossip(kind=w.kind, n_workers=w.n_workers, layer_shapes=w.layer_shapes, rank=w.rank,
                         power_steps=w.power_steps, seed=w.seed, torus_rows=w.torus_rows,
                         torus_cols=w.torus_cols, custom_edges=w.custom_edges,
                         weight_rule=w.weight_rule, W=wl.mixing_matrix(w), device=device)
    stream = torch.cuda.current_stream()

    def upload():
        for i in range(w.n_workers):
            for l in range(L):
                net.pg_write_params(i, l, views[i][l], stream)

    def download():
        for i in range(w.n_workers):
            for l in range(L):
                net.pg_read_params(i, l, back_views[i][l], stream)

    # ---- device-resident timing ------------------------------------------------
    upload()
    for _ in range(max(args.warmup, 3)):
        net.pg_round(stream)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = net.pg_kernel_launches()
    net.pg_timing_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        net.pg_round(stream)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    net.pg_timing_enable(False)
    ms_total = e0.elapsed_time(e1)
    ms_total_local = ms_total
    launches = net.pg_kernel_launches() - launches0
    kernel_times = net.pg_timing_read()
    status = net.pg_device_status(stream)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_total = max_over_ranks(ms_total, dist, device)
    ms_step = ms_total / args.steps
    value = whole_job_rate(world, args.steps, ms_total)

    # ---- end to end through the C ABI with host buffers -------------------------
    # Every step uploads the whole stack from pinned memory, runs one round and reads the
    # whole result back.  The read-back of step s runs on one stream beside the upload of
    # step s + 1 on another (both directions of the link at once); a matrix is overwritten
    # only after its own read-back has finished, and a round starts after all uploads.
    e2e_steps = max(1, args.e2e_steps)
    upload()
    net.pg_round(stream)
    download()
    up_stream, down_stream = torch.cuda.Stream(), torch.cuda.Stream()
    read_done = [[torch.cuda.Event() for _ in range(L)] for _ in range(w.n_workers)]
    barrier()
    e0.record(stream)
    up_stream.wait_stream(stream)
    for step in range(e2e_steps):
        for i in range(w.n_workers):
            for l in range(L):
                if step > 0:
                    up_stream.wait_event(read_done[i][l])
                net.pg_write_params(i, l, views[i][l], up_stream)
        stream.wait_stream(up_stream)
        net.pg_round(stream)
        down_stream.wait_stream(stream)
        for i in range(w.n_workers):
            for l in range(L):
                net.pg_read_params_async(i, l, back_views[i][l], down_stream)
                read_done[i][l].record(down_stream)
    stream.wait_stream(down_stream)
    e1.record(stream)
    barrier()
    status = status or net.pg_device_status(stream)
    ms_e2e = e0.elapsed_time(e1)
    ms_e2e = max_over_ranks(ms_e2e, dist, device)
    e2e_value = whole_job_rate(world, e2e_steps, ms_e2e)
    finite = bool(torch.isfinite(back[: min(total, 1 << 22)]).all())

    if rank != 0:
        net.close()
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ------------------------------------------
    # per kernel kind: total ms, launches and algorithmic bytes of the launches in the
    # timed region (the library counts 4 B per parameter a launch covers for every
    # time it has to read or write X once)
    peak, peak_kind = hbm_peak()
    names = {"update_forward": "row_sweep_kernel<update+forward>", "transposed": "col_sweep_kernel<transposed>",
             "pair_sweep": "pair_sweep_kernel<pending update + X q + X^T p>", "forward": "row_sweep_kernel<forward>",
             "edge_left": "edge_left_kernel", "edge_right": "edge_right_kernel", "pair_edge": "pair_edge_kernel",
             "update_only": "row_sweep_kernel<update>"}
    kinds = {}
    for kind, (ms, n, nbytes) in kernel_times.items():
        if n:
            kinds[names[kind]] = {"launches": n, "total_ms": ms, "share": ms / ms_total_local,
                                  "avg_launch_ms": ms / n,
                                  "algorithmic_bytes_per_launch": nbytes / n,
                                  "achieved_gbs": (nbytes / (ms * 1e-3) / 1e9) if nbytes else None}
    top = max(kinds, key=lambda k: kinds[k]["total_ms"])
    traffic = None
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            rec = json.load(f)
        src = open(os.path.join(ROOT, "paper_2008_01425_b200", "csrc", "pg_kernels.cu"), "rb").read()
        if (rec.get("kernel_source_sha256") == hashlib.sha256(src).hexdigest()
                and rec.get("workload") == w.name and rec.get("kernel") == top):
            traffic = rec.get("dram_bytes_per_launch")
    except Exception:
        traffic = None
    roofline = {
        "bound": "hbm", "kernel": top, "achieved": kinds[top]["achieved_gbs"], "peak": peak,
        "unit": "GB/s", "frac": kinds[top]["achieved_gbs"] / peak, "peak_source": peak_kind,
        "algorithmic_bytes_per_launch": kinds[top]["algorithmic_bytes_per_launch"],
        "avg_launch_ms": kinds[top]["avg_launch_ms"], "traffic": traffic,
        "kernels": kinds,
    }
    bytes_round = 12.0 * total * w.power_steps
    eff = bytes_round / (ms_step * 1e-3) / 1e9

    cpu = None
    if not args.no_cpu_baseline:
        try:
            v, dt, n_sample, cores, n_timed = time_oracle_sample(w, args.cpu_sample_workers, 2, 2, target_seconds=12.0)
            cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": "%d of %d workers of %s, %d timed rounds in %.1f s, scaled by workers"
                             % (n_sample, w.n_workers, w.name, n_timed, dt)}
        except Exception as exc:  # the baseline never decides the run
            cpu = {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": "failed: %r" % (exc,)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "n_workers": w.n_workers, "layers": L,
                   "params_per_worker": w.params_per_worker, "rank": w.rank,
                   "power_steps": w.power_steps, "graph": ["ring", "torus", "matching", "custom"][w.kind],
                   "l2": "inputs (%.2f GB) larger than L2, no flush" % (4.0 * total / 1e9),
                   "parallelism": "replicas x%d (no data-path collective)" % world if world > 1 else "1 gpu",
                   "effective_hbm_gbs_12B_per_param_step": eff,
                   "effective_frac_of_8TBs_nominal": eff / 8000.0,
                   "effective_frac_of_measured_copy": eff / peak},
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps,
                "h2d_bytes_per_step": 4 * total, "d2h_bytes_per_step": 4 * total,
                "ms_per_step": ms_e2e / e2e_steps, "result_finite": finite},
        "gpu_launches": int(launches),
        "device_status": int(status),
        "clocks": clocks,
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    net.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
