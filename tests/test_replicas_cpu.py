"""N > 1 path on CPU: the step has no exchange between GPUs, so bench.py runs N independent replicas and
only the timing is combined (max over ranks).  Two gloo ranks check that combination and that the
reference arm runs on rank 0 alone."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"ms": ms, "value": bench.job_tokens_per_s(8192, 10, world, ms)}, f)
    dist.destroy_process_group()


def test_two_replicas_report_slowest_rank_time(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["ms"] == 15.0                                   # max over the two ranks
    assert abs(r["value"] - 2 * 8192 * 10 / 15e-3) < 1e-6    # both replicas' tokens over the slowest time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""      # other ranks exit 0 without work


def test_model_flops_match_hand_count():
    import bench
    import workloads as wl
    w = wl.CONFIGS["cfg4"]
    # forward 8 x (75.5 + 6.3) + wgrad 8 x 75.5 + 14 streams x (75.5 + 12.6) + heads 8 x 6 d V  [MF per token]
    assert abs(bench.model_flops_per_token(w, 2) / 1e6 - 4961.6) < 0.5
    assert abs(bench.model_flops_per_token(w, 3) / 1e6 - 5314.0) < 0.5
    w2 = wl.CONFIGS["cfg2"]
    assert abs(bench.model_flops_per_token(w2, 1) / 1e6 - 1492.6) < 0.5
    assert abs(bench.model_flops_per_token(w2, 4) / 1e6 - 1492.6) < 0.5
