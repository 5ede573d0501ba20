"""The benchmark's multi-process arithmetic (replicas only: max over ranks of the step time, whole-job rate),
run as two gloo ranks on the CPU.  The reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.all_max(3.0 + 2.0 * rank, torch.device("cpu"), world)  # rank 0: 3 ms, rank 1: 5 ms
    out[rank] = (ms, bench.whole_job_value(1000.0, ms, world))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29517, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1] == (5.0, 2 * 1000.0 / 5e-3)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.all_max(4.25, None, 1) == 4.25 and bench.whole_job_value(10.0, 2.0, 1) == 5000.0
    assert bench.compulsory_bytes(10, 100, 8, 2, True) == 400 + 400 + 80 + 2 * 10 * 8 * 2


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
