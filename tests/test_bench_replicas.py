"""Host logic of the multi-GPU bench path, on CPU: the path has no exchange step, so N ranks are N
independent replicas; what is shared is a barrier, the max-over-ranks of the timing and the rule
that rank 0 alone reports.  Run as two gloo ranks."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.job_throughput(world, 4096, 32, ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_add_their_units():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, 29731, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 15.0
    assert abs(value - 2 * 4096 * 32 / 15e-3) < 1e-6 * value


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
           "--steps", "1", "--warmup", "0"]
    r0 = subprocess.run(cmd, env=dict(env, RANK="0", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    r1 = subprocess.run(cmd, env=dict(env, RANK="1", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0 and r1.returncode == 0
    assert r1.stdout.strip() == ""
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
