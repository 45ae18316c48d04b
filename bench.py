#!/usr/bin/env python
"""Benchmark of the PowerGossip hot path: gossip rounds per second.

    python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]

One "step" is one gossip round (all power steps, every layer, every edge of the
round's graph) of the workload, by default the largest one: the LSTM-shaped
stack (46.5 M fp32 parameters per worker) on 32 workers with a perfect matching
re-drawn every round.  Inputs are synthetic and seeded; they are far larger
than L2, so nothing is flushed between steps.

value      rounds/s with the parameters already resident in HBM: K rounds between
           two CUDA events on the launching stream, repeated (at least five times,
           and until half a second has been timed), the median repetition, max over
           ranks.  No per-kernel events are recorded in these repetitions.
e2e        the same round driven through the C ABI with host buffers: every step
           uploads all parameters from pinned host memory, runs the round and
           reads all parameters back, all inside the timed region.
roofline   a separate pass of K rounds with one event pair around every kernel:
           the kernel kind with the largest share, its algorithmic bytes per launch
           (4 B per parameter it covers for every time it has to read or write X
           once) over its average launch time, against the measured HBM copy
           bandwidth of this machine; and the same for the whole round on the
           bytes the round really moves (8 B per parameter and step on pair-sweep
           layers, 12 B on three-sweep layers).
per_config the five workloads of the task (the torus at 1, 2 and 4 power steps, the
           VGG-shaped ring at rank 1 and 2), each with its own clock sample.
parity     the CUDA path against the fp64 CPU checker on a 4-worker slice of the
           workload after 3 rounds, and the drift of the worker average.
cpu_baseline the fp64 CPU checker, as it stands, on a bounded sample of the same
           workload on the host cores (reported for context only).

With --gpus N > 1 (launched under torchrun, one process per GPU) every rank runs
an independent replica of the network; there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
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
NOMINAL_HBM_GBS = 8000.0
ORACLE_SAMPLE_WORKERS = 8       # both CPU legs time the checker on this many workers
MIN_REPETITIONS = 5
MIN_TIMED_MS = 500.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="lstm_matching32")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
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
    """Samples nvidia-smi clocks and throttle reasons while a timed region runs (read-only)."""

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

    def window(self, t0: float, t1: float):
        """Summary of the samples taken between two wall-clock times."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        sm, smax, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ts, line in list(self.lines):
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

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()


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


def repetitions_for(ms_region: float) -> int:
    """At least MIN_REPETITIONS, and as many as bring the timed total to MIN_TIMED_MS."""
    return int(min(max(MIN_REPETITIONS, math.ceil(MIN_TIMED_MS / max(ms_region, 1e-3))), 2000))


def median(values):
    v = sorted(values)
    return v[len(v) // 2] if len(v) % 2 else 0.5 * (v[len(v) // 2 - 1] + v[len(v) // 2])


def config_of(w, world: int):
    """What both arms report about the workload."""
    return {"workload": w.name, "n_workers": w.n_workers, "layers": len(w.layer_shapes),
            "params_per_worker": w.params_per_worker, "rank": w.rank, "power_steps": w.power_steps,
            "graph": ["ring", "torus", "matching", "custom"][w.kind],
            "l2": "inputs (%.2f GB) larger than L2, no flush" % (4.0 * w.total_params / 1e9)
                  if 4.0 * w.total_params > 126e6 else "inputs (%.3f GB) fit in L2: latency-bound" % (4.0 * w.total_params / 1e9),
            "parallelism": "replicas x%d (no data-path collective)" % world if world > 1 else "1 gpu"}


# ----------------------------------------------------------------------------
# the CPU checker as a timed baseline (bounded sample)
# ----------------------------------------------------------------------------
def oracle_sample(w, sample_workers: int):
    """The checker on `sample_workers` workers of the workload, parameters loaded."""
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
    return o, sample


def time_oracle(o, rounds: int):
    t0 = time.perf_counter()
    o.round(rounds)
    return time.perf_counter() - t0


def cpu_baseline(w, warmup: int = 2, target_seconds: float = 12.0):
    """The fp64 checker on ORACLE_SAMPLE_WORKERS workers: all host threads for about
    `target_seconds`, then two rounds on one thread.  A round costs in proportion to the
    number of workers (every worker takes part in `degree` edges whatever N is), so the
    full workload's rate is the sample's x sample workers / N: an extrapolation."""
    from oracle import pg_oracle as po

    o, sample = oracle_sample(w, ORACLE_SAMPLE_WORKERS)
    threads = po.num_threads()
    pace = time_oracle(o, max(warmup, 1)) / max(warmup, 1)     # includes the first touch of every vector
    rounds = int(min(max(2, target_seconds / max(pace, 1e-6)), 1000))
    dt = time_oracle(o, rounds)
    scale = sample.n_workers / w.n_workers
    value = rounds / dt * scale
    po.set_num_threads(1)
    rounds_1 = int(min(max(1, 4.0 / max(pace * threads, 1e-6)), rounds))
    dt_1 = time_oracle(o, rounds_1)
    po.set_num_threads(threads)
    o.close()
    return {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
            "one_thread_value": rounds_1 / dt_1 * scale,
            "sample": "%d of %d workers of %s, %d timed rounds in %.1f s on %d threads (%d rounds in %.1f s on one), "
                      "extrapolated to %d workers in proportion to the worker count"
                      % (sample.n_workers, w.n_workers, w.name, rounds, dt, threads, rounds_1, dt_1, w.n_workers)}


def run_reference(args, w):
    """--impl reference: the CPU checker on the host cores.  Every step is one round on a
    bounded sample (ORACLE_SAMPLE_WORKERS workers) of the workload; `value` is extrapolated
    to the full worker count, `ms_per_step` is the time a sample step really took."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import pg_oracle as po

    o, sample = oracle_sample(w, ORACLE_SAMPLE_WORKERS)
    time_oracle(o, max(args.warmup, 1))
    dt = time_oracle(o, args.steps)
    o.close()
    scale = sample.n_workers / w.n_workers
    value = args.steps / dt * scale
    world = int(os.environ.get("WORLD_SIZE", "1"))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 * dt / args.steps,
        "ms_per_step_extrapolated": 1000.0 / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_of(w, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": po.num_threads(), "kind": "oracle",
                         "sample": "%d of %d workers of %s, %d timed rounds in %.1f s, extrapolated to %d workers "
                                   "in proportion to the worker count"
                                   % (sample.n_workers, w.n_workers, w.name, args.steps, dt, w.n_workers)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------
def make_network(w, device):
    from paper_2008_01425_b200 import binding as pg
    from paper_2008_01425_b200 import workloads as wl

    return pg.PowerGossip(kind=w.kind, n_workers=w.n_workers, layer_shapes=w.layer_shapes, rank=w.rank,
                          power_steps=w.power_steps, seed=w.seed, torus_rows=w.torus_rows,
                          torus_cols=w.torus_cols, custom_edges=w.custom_edges,
                          weight_rule=w.weight_rule, W=wl.mixing_matrix(w), device=device)


def time_rounds(net, stream, steps: int, reps: int, barrier, batched: bool = False):
    """`reps` repetitions of `steps` rounds, each between two events on `stream` with a
    synchronisation on both sides; returns the list of milliseconds."""
    import torch

    out = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(reps):
        barrier()
        e0.record(stream)
        if batched:
            net.pg_rounds(steps, stream)
        else:
            for _ in range(steps):
                net.pg_round(stream)
        e1.record(stream)
        barrier()
        out.append(e0.elapsed_time(e1))
    return out


def measure_config(w, device, sampler, peak, steps_hint_ms: float = 100.0):
    """One line of per_config: the workload uploaded, warmed up, timed as the median of
    repetitions of about `steps_hint_ms` each, with the clocks seen meanwhile."""
    import torch

    from paper_2008_01425_b200 import workloads as wl

    net = make_network(w, device)
    stream = torch.cuda.current_stream()
    for i in range(w.n_workers):
        for l in range(len(w.layer_shapes)):
            net.pg_write_params(i, l, wl.initial_params(w, i, l), stream)
    for _ in range(5):
        net.pg_round(stream)
    sync = torch.cuda.synchronize
    sync()
    probe = time_rounds(net, stream, 10, 1, sync)[0] / 10.0
    steps = int(min(max(10, steps_hint_ms / max(probe, 1e-4)), 20000))
    reps = repetitions_for(steps * probe)
    t0 = time.time()
    times = time_rounds(net, stream, steps, reps, sync)
    t1 = time.time()
    ms = median(times) / steps
    bytes_round, pair_share = net.pg_round_bytes()
    per_param = bytes_round / (w.total_params * w.power_steps)
    gbs = bytes_round / (ms * 1e-3) / 1e9
    resident = 4.0 * w.total_params <= 126e6
    entry = {"workload": w.name, "rank": w.rank, "power_steps": w.power_steps, "n_workers": w.n_workers,
             "ms_per_round": ms, "rounds_per_s": 1000.0 / ms, "steps_per_repetition": steps, "repetitions": reps,
             "bytes_per_param_and_step": per_param, "share_of_params_on_pair_sweep": pair_share,
             "algorithmic_bytes_per_round": bytes_round,
             "clocks": sampler.window(t0, t1) if sampler else None, "device_status": net.pg_device_status(stream)}
    if resident:
        entry["us_per_round"] = 1000.0 * ms
        entry["note"] = "stack resident in L2: latency-bound, no HBM fraction"
        if w.kind != wl.MATCHING:
            net.pg_rounds(2 * steps, stream)          # warm-up rounds and the graph capture happen here
            sync()
            entry["us_per_round_pg_rounds"] = 1000.0 * median(time_rounds(net, stream, steps, reps, sync, True)) / steps
    else:
        entry["effective_gbs"] = gbs
        entry["frac_of_measured_copy"] = gbs / peak
        entry["frac_of_8TBs_nominal"] = gbs / NOMINAL_HBM_GBS
    net.close()
    return entry


def parity_slice(w, device):
    """CUDA path against the fp64 checker on a 4-worker slice of the workload after 3 rounds:
    max over (worker, layer) of ||X_gpu - X_ref||_F / ||X_ref||_F, and the relative drift of
    the worker average on the GPU (Lemma 1)."""
    import numpy as np

    from paper_2008_01425_b200 import workloads as wl

    o, sample = oracle_sample(w, 4)
    net = make_network(sample, device)
    L = len(sample.layer_shapes)
    avg0 = []
    for l in range(L):
        acc = np.zeros(sample.layer_shapes[l], dtype=np.float64)
        for i in range(sample.n_workers):
            x = wl.initial_params(sample, i, l)
            net.pg_write_params(i, l, x)
            acc += x
        avg0.append(acc / sample.n_workers)
    rounds = 3
    for _ in range(rounds):
        net.pg_round()
    o.round(rounds)
    worst, drift = 0.0, 0.0
    for l in range(L):
        acc = np.zeros(sample.layer_shapes[l], dtype=np.float64)
        for i in range(sample.n_workers):
            got = net.pg_read_params(i, l).astype(np.float64)
            ref = o.get_params(i, l)
            worst = max(worst, float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)))
            acc += got
        drift = max(drift, float(np.linalg.norm(acc / sample.n_workers - avg0[l]) / max(np.linalg.norm(avg0[l]), 1e-300)))
    d_ref = o.consensus_distance()
    status = net.pg_device_status()
    net.close()
    o.close()
    return {"max_relative_error": worst, "average_drift": drift, "tolerance": 1e-4, "rounds": rounds,
            "consensus_distance_checker": d_ref, "device_status": status,
            "sample": "%d of %d workers of %s against the fp64 CPU checker" % (sample.n_workers, w.n_workers, w.name)}


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

    import torch

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

    net = make_network(w, device)
    stream = torch.cuda.current_stream()

    def upload():
        for i in range(w.n_workers):
            for l in range(L):
                net.pg_write_params(i, l, views[i][l], stream)

    def download():
        for i in range(w.n_workers):
            for l in range(L):
                net.pg_read_params(i, l, back_views[i][l], stream)

    # ---- device-resident timing: repetitions of exactly K rounds, no per-kernel events ----
    warmup = max(args.warmup, 3)
    upload()
    for _ in range(warmup):
        net.pg_round(stream)
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    probe = time_rounds(net, stream, args.steps, 1, barrier)[0]
    reps = repetitions_for(max_over_ranks(probe, dist, device))
    launches0 = net.pg_kernel_launches()
    t_wall0 = time.time()
    times = time_rounds(net, stream, args.steps, reps, barrier)
    t_wall1 = time.time()
    launches_all = net.pg_kernel_launches() - launches0
    status = net.pg_device_status(stream)
    clocks = sampler.window(t_wall0, t_wall1) if sampler else None
    ms_total_local = median(times)
    ms_total = max_over_ranks(ms_total_local, dist, device)
    ms_step = ms_total / args.steps
    value = whole_job_rate(world, args.steps, ms_total)

    # ---- a separate pass of K rounds with an event pair around every kernel ------------
    net.pg_timing_enable(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        net.pg_round(stream)
    e1.record(stream)
    barrier()
    net.pg_timing_enable(False)
    ms_timing_pass = e0.elapsed_time(e1)
    kernel_times = net.pg_timing_read()
    bytes_round, pair_share = net.pg_round_bytes()

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
    net.close()
    del net, host, back, views, back_views
    torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel and of the whole round -------------------
    peak, peak_kind = hbm_peak()
    names = {"update_forward": "row_sweep_kernel<update+forward>", "transposed": "col_sweep_kernel<transposed>",
             "pair_sweep": "pair_sweep kernels<pending update + X q + X^T p>", "forward": "row_sweep_kernel<forward>",
             "edge_left": "edge_left_kernel", "edge_right": "edge_right_kernel", "pair_edge": "pair_edge_kernel",
             "update_only": "row_sweep_kernel<update>"}
    kinds = {}
    for kind, (ms, n, nbytes) in kernel_times.items():
        if n:
            kinds[names[kind]] = {"launches": n, "total_ms": ms, "share": ms / ms_timing_pass,
                                  "avg_launch_ms": ms / n,
                                  "algorithmic_bytes_per_launch": nbytes / n,
                                  "achieved_gbs": (nbytes / (ms * 1e-3) / 1e9) if nbytes else None}
    top = max(kinds, key=lambda k: kinds[k]["total_ms"])
    traffic, traffic_note = None, None
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            rec = json.load(f)
        digest = hashlib.sha256()
        for name in ("pg_kernels.cu", "pg_api.cu", "pg_device.h"):      # kernels, tile shapes, layout
            digest.update(open(os.path.join(ROOT, "paper_2008_01425_b200", "csrc", name), "rb").read())
        if (rec.get("kernel_source_sha256") == digest.hexdigest()
                and rec.get("workload") == w.name and rec.get("kernel") == top):
            traffic = rec.get("dram_bytes_per_launch")
            traffic_note = rec.get("note")
    except Exception:
        traffic = None
    round_gbs = bytes_round / (ms_step * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": top, "achieved": kinds[top]["achieved_gbs"], "peak": peak,
        "unit": "GB/s", "frac": kinds[top]["achieved_gbs"] / peak, "peak_source": peak_kind,
        "algorithmic_bytes_per_launch": kinds[top]["algorithmic_bytes_per_launch"],
        "avg_launch_ms": kinds[top]["avg_launch_ms"], "traffic": traffic, "traffic_note": traffic_note,
        "timing_pass_ms_per_step": ms_timing_pass / args.steps,
        "round": {"algorithmic_bytes": bytes_round,
                  "bytes_per_param_and_step": bytes_round / (total * w.power_steps),
                  "share_of_params_on_pair_sweep": pair_share,
                  "achieved_gbs": round_gbs, "frac_of_measured_copy": round_gbs / peak,
                  "frac_of_8TBs_nominal": round_gbs / NOMINAL_HBM_GBS,
                  "rounds_per_s_of_the_three_sweep_method_at_this_rate": round_gbs * 1e9 / (12.0 * total * w.power_steps)},
        "kernels": kinds,
    }

    parity = None
    if not args.no_parity:
        try:
            parity = parity_slice(w, device)
        except Exception as exc:
            parity = {"max_relative_error": None, "sample": "failed: %r" % (exc,)}

    per_config = None
    if world == 1 and not args.no_per_config:
        per_config = []
        for cfg in (wl.tiny_ring(), wl.resnet20_ring8(), wl.torus8x8(1), wl.torus8x8(2), wl.torus8x8(4),
                    wl.vgg16_ring16(1), wl.vgg16_ring16(2)):
            try:
                per_config.append(measure_config(cfg, device, sampler, peak))
            except Exception as exc:
                per_config.append({"workload": cfg.name, "failed": repr(exc)})
            torch.cuda.empty_cache()
        per_config.append({"workload": w.name, "rank": w.rank, "power_steps": w.power_steps, "n_workers": w.n_workers,
                           "ms_per_round": ms_step, "rounds_per_s": 1000.0 / ms_step,
                           "steps_per_repetition": args.steps, "repetitions": reps,
                           "bytes_per_param_and_step": bytes_round / (total * w.power_steps),
                           "share_of_params_on_pair_sweep": pair_share, "algorithmic_bytes_per_round": bytes_round,
                           "effective_gbs": round_gbs, "frac_of_measured_copy": round_gbs / peak,
                           "frac_of_8TBs_nominal": round_gbs / NOMINAL_HBM_GBS, "clocks": clocks,
                           "device_status": int(status), "note": "the headline measurement"})
    if sampler:
        sampler.stop()

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        try:
            cpu = cpu_baseline(w)
        except Exception as exc:  # the baseline never decides the run
            cpu = {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": "failed: %r" % (exc,)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(w, world),
        "repetitions": reps, "ms_per_repetition": {"median": ms_total_local, "min": min(times), "max": max(times)},
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps,
                "h2d_bytes_per_step": 4 * total, "d2h_bytes_per_step": 4 * total,
                "ms_per_step": ms_e2e / e2e_steps, "result_finite": finite},
        "gpu_launches": int(round(launches_all / reps)),
        "gpu_launches_all_repetitions": int(launches_all),
        "device_status": int(status),
        "clocks": clocks,
        "roofline": roofline,
        "parity": parity,
        "per_config": per_config,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
