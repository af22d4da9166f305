"""The N > 1 path on CPU with gloo, world size 2.  The reshard does not shard across GPUs (replicas only), so
what N > 1 adds is the max-over-ranks time, the summed throughput, and rank 0 alone printing the line."""
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
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 40.0 if rank == 0 else 50.0           # rank 1 is the slow one
    ms_per_step, value = bench.aggregate_over_ranks(local_ms, 10, 32_000_000_000, world, torch.device("cpu"))
    out[rank] = (ms_per_step, value)
    dist.barrier()
    dist.destroy_process_group()


def test_replicas_aggregate_max_time_and_summed_bytes():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    for rank in (0, 1):
        ms, value = out[rank]
        assert ms == pytest.approx(5.0)                               # slowest rank: 50 ms / 10 steps
        assert value == pytest.approx(2 * 32.0 / 5e-3)                # both replicas' bytes over that time


def test_reference_arm_prints_once_under_torchrun():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29612", os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
