"""The N > 1 path on CPU (gloo, world size 2): the schedule is replicated, so every rank must build the
same trees from the same timeline; timings are combined as the maximum over ranks and the value as the
sum over ranks; the oracle arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import paper_2002_05814_b200 as hpl
    import workloads as wl

    # (1) timings: max over ranks; value: whole job
    tot, wall = bench.max_over_ranks([10.0 * (rank + 1), 7.0 - rank], dist, torch.device("cpu"))
    assert (tot, wall) == (20.0, 7.0)
    assert abs(bench.whole_job_value(1_000_000_000, 4, world, tot) - 2 * 4 * 1.0 / 20e-3) < 1e-6

    # (2) replicated schedules: every rank feeds the same timeline to its own (schedule-only) context
    w = wl.workload("cfg3")
    c = hpl.Context(w.chunk_bytes, w.degree, w.degree)
    for i in range(16):
        c.create(i, i, w.object_bytes)
    c.reduce(100, list(range(16)), 8)
    arr = wl.exponential_arrivals_ns(w.seed, 16, w.extra["mean_arrival_ns"])
    for i in sorted(range(16), key=lambda i: (arr[i], i)):
        c.advance(arr[i])
        c.put(i, 4096 * (i + 1), w.object_bytes)
    c.advance(max(arr) + 1)
    c.fail(sorted(range(16), key=lambda i: (arr[i], i))[2])
    words = torch.tensor(c.schedule_dump(100), dtype=torch.int64)
    gathered = [torch.zeros_like(words) for _ in range(world)]
    dist.all_gather(gathered, words)
    assert all(torch.equal(g, words) for g in gathered)
    c.shutdown()
    dist.barrier()
    with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
        f.write("ok")
    dist.destroy_process_group()


def test_two_ranks_on_gloo(tmp_path):
    from paper_2002_05814_b200 import build
    build.build()
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok0").exists() and (tmp_path / "ok1").exists()


def test_oracle_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "cfg1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0", "--workload", "cfg1"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
