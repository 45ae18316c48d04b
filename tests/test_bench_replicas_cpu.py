"""bench.py's multi-GPU mode runs independent replicas (no data-path collective);
the only cross-rank step is taking the slowest rank's time.  Checked here with
two gloo ranks on the CPU, plus the reference arm's rank handling."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    rate = bench.whole_job_rate(world, 20, ms)
    dist.barrier()
    dist.destroy_process_group()
    with open(out % rank, "w") as f:
        json.dump({"ms": ms, "rate": rate}, f)


def test_slowest_rank_sets_the_time(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    out = str(tmp_path / "r%d.json")
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for r in range(world):
        got = json.load(open(out % r))
        assert got["ms"] == 15.0                       # the slower rank's time, on every rank
        assert abs(got["rate"] - 2 * 20 / 0.015) < 1e-6   # both replicas' rounds over that time


def test_without_a_process_group_it_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.whole_job_rate(1, 10, 5.0) == 2000.0


def test_reference_arm_prints_one_line_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                        "tiny_ring4_64x32", "--steps", "3", "--warmup", "1", "--gpus", "2"],
                       env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == b""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                        "tiny_ring4_64x32", "--steps", "3", "--warmup", "1", "--gpus", "2"],
                       env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.decode().strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
