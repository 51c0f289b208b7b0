"""Host logic of the multi-rank benchmark path on CPU (gloo, world size 2): the path shards as
independent replicas, so the only exchange is the MAX of the ranks' timings, and the reference arm
runs on rank 0 alone."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 2.0 + 3.0 * rank                       # rank 1 is the slow one
    worst = bench.max_over_ranks(ms, device="cpu")
    value = bench.whole_job_gflops(world, 1e9, worst)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"worst": worst, "value": value}, f)
    dist.destroy_process_group()


def test_timing_is_the_max_over_ranks_and_value_is_the_aggregate(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    assert got[0] == got[1]
    assert got[0]["worst"] == 5.0
    assert abs(got[0]["value"] - 2 * 1e9 / 5.0 / 1e6) < 1e-9


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(1.25, device="cpu") == 1.25
    assert bench.whole_job_gflops(1, 2e9, 4.0) == 500.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and out.stdout.strip() == ""
