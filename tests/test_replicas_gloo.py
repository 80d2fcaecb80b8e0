"""The N > 1 path of the benchmark is "replicas only": no data-path collective, just a barrier and a maximum of
the per-rank times.  These tests run that aggregation with two gloo ranks on CPU, and the reference arm's rule
that only rank 0 works and prints."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    my_ms = 10.0 if rank == 0 else 25.0                # rank 1 is the straggler
    mx = bench.max_over_ranks([my_ms, 2.0 * my_ms], world, "cpu")
    value, ms = bench.aggregate_tokens_per_s(100, my_ms, world, "cpu")
    dist.barrier()
    out[rank] = (mx, value, ms)
    dist.destroy_process_group()


def test_replica_aggregation_takes_the_slowest_rank_and_sums_tokens():
    world, port = 2, 29617
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        mx, value, ms = res[rank]
        assert mx == [25.0, 50.0]                       # max over ranks, seen by every rank
        assert ms == 25.0
        assert value == pytest.approx(2 * 100 / 25e-3)  # whole-job tokens/s over the slowest rank's time


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1, "cpu") == [3.0, 4.0]
    assert bench.aggregate_tokens_per_s(50, 10.0, 1, "cpu") == (5000.0, 10.0)


def test_reference_arm_under_two_ranks_only_rank0_prints():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29618")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2",
           "--warmup", "1", "--workload", "tiny"]
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
