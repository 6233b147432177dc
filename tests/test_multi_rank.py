"""The N > 1 path of the benchmark on CPU: two gloo ranks.

The hot path does not shard (one stream's cache lives on one GPU), so N ranks are N
independent replicas: each rank draws its own frames, there is no data-path
collective, and the only exchange is the max-over-ranks of the timed region.  These
tests run that logic as two processes over gloo."""
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
    try:
        ms_local = 10.0 if rank == 0 else 25.0          # rank 1 is the slow replica
        value, ms = bench.job_throughput(ms_local, steps=5, world=world, dist=dist, device="cpu")
        out[rank] = (value, ms, bench.replica_seed(7, rank))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_all_frames_over_the_slowest_rank():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        value, ms, _ = res[rank]
        assert ms == 25.0                               # max over ranks, the same on every rank
        assert abs(value - 2 * 5 / 25e-3) < 1e-9        # whole-job frames/s: both replicas' frames
    assert res[0][2] != res[1][2]                       # the replicas stream different frames


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.job_throughput(20.0, steps=4, world=1)
    assert ms == 20.0 and abs(value - 4 / 20e-3) < 1e-9


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
