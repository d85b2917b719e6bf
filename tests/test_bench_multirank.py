"""The benchmark's N > 1 path on CPU: two `gloo` ranks (replicas - the layer has no exchange step on
one node) reduce their step times with MAX and report the whole-job aggregate; the reference arm
runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")        # rank 1 is the slow one
    value = bench.aggregate_throughput(1000, world, ms)
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"ms": ms, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_aggregate(tmp_path):
    out = str(tmp_path / "r0.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    got = json.load(open(out))
    assert got["ms"] == 15.0                                  # the maximum over ranks, not rank 0's own
    assert got["value"] == 2 * 1000 / 15e-3                   # both replicas' tokens over that time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.aggregate_throughput(131072, 1, 13.1072) == 131072 / 13.1072e-3


def test_reference_arm_other_ranks_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
