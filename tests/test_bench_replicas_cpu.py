"""Host logic of `bench.py --gpus N`: N independent replicas, no data-path collective.

Two gloo ranks on CPU check what the multi-GPU run relies on: different seeds per replica, the
job time is the slowest rank's, the reported value is the sum over replicas, and under
`--impl reference` only rank 0 produces a line.
"""
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
    ms_local = 100.0 + 50.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, device="cpu")
    out[rank] = (ms, bench.replica_seed(3, rank), bench.aggregate_frames_per_s(world, 10, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_replicas_report_the_slowest_rank_and_the_summed_throughput():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29571, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 150.0
    assert res[0][1] != res[1][1]
    assert abs(res[0][2] - 2 * 10 / 0.150) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
