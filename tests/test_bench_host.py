"""Host-side logic of bench.py: the N > 1 path (max over ranks, whole-job throughput) on CPU with gloo."""
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


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank "measured" a different time: the job time is the slowest rank's
    ms = 10.0 + 5.0 * rank
    worst = bench.reduce_max(ms)
    value = bench.aggregate_throughput(units_per_rank=1000.0, world=world, max_seconds=worst / 1e3)
    dist.barrier()
    if rank == 0:
        json.dump({"worst": worst, "value": value}, open(out, "w"))
    dist.destroy_process_group()


def test_two_rank_aggregation(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["worst"] == 15.0
    assert abs(r["value"] - 2 * 1000.0 / 0.015) < 1e-6


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5) == 3.5
    assert bench.aggregate_throughput(10.0, 4, 2.0) == 20.0
    peaks = bench.load_peaks()
    assert peaks["hbm_gbs"] > 1000 and peaks["source"] in ("measured", "fallback")
    assert bench.dist_env() == (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
                                int(os.environ.get("WORLD_SIZE", 1)))


def test_reference_arm_other_ranks_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
