"""Host-side logic of the N>1 benchmark path, on CPU with the gloo backend
(world_size 2): units are independent, so ranks run replicas with no data-path
collective; the only exchange is the max over ranks of the device time."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 100.0 if rank == 0 else 250.0          # rank 1 is the slow one
    per_step, value = bench.job_throughput(local_ms, steps=50, world=world, dist=dist, device="cpu")
    out[rank] = (per_step, value)
    dist.barrier()
    dist.destroy_process_group()


def test_job_throughput_takes_the_slowest_rank_and_counts_all_replicas():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29617, out), nprocs=2, join=True)
    for rank in (0, 1):
        per_step, value = out[rank]
        assert abs(per_step - 5.0) < 1e-9             # 250 ms / 50 steps
        assert abs(value - 2 * 1000.0 / 5.0) < 1e-6   # two replicas' worth of steps per second


def test_reference_arm_prints_on_rank_zero_only():
    sys.path.insert(0, ROOT)
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29618")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
           "--steps", "5", "--warmup", "1", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", LOCAL_RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", LOCAL_RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def test_single_process_throughput():
    sys.path.insert(0, ROOT)
    import bench
    per_step, value = bench.job_throughput(30.0, steps=10, world=1)
    assert per_step == 3.0 and abs(value - 1000.0 / 3.0) < 1e-9
    n = bench.live_rows_schedule(bench.wl.CONFIGS["tiny"], first_step=33, count=40)
    assert n[0] == 33 and max(n) == 64 and n[64 - 33 + 1 - 1] == 64 and n[64 - 33 + 1] == 49
