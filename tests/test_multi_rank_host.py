"""Host-side logic of the multi-GPU benchmark path, exercised with two gloo ranks on CPU: shards are
independent, the slowest rank's time counts, and the reference arm runs on rank 0 only."""
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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    # rank r pretends its timed region took 10 + 5 r milliseconds
    total = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"), dist)
    value = bench.whole_job_throughput(4096, world, total / 10)
    out[rank] = (total, value)
    dist.barrier()
    dist.destroy_process_group()


def test_slowest_rank_counts_and_throughput_is_whole_job():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29517, out), nprocs=world, join=True)
    for r in range(world):
        total, value = out[r]
        assert total == 15.0
        assert value == pytest.approx(2 * 4096 / (1.5e-3))


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29518", WORLD_SIZE="2")
    outs = []
    for rank in (0, 1):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                            "--warmup", "0", "--workload", "sweep_c16", "--cpu-seconds", "1"], env=e, capture_output=True, text=True, timeout=300)
        assert p.returncode == 0, p.stderr
        outs.append(p.stdout.strip())
    line = json.loads(outs[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert outs[1] == ""
