"""The multi-rank bookkeeping of bench.py on CPU (gloo, world size 2): the path has no exchange
step, every rank runs its own shard; the job's time is the slowest rank's, its throughput the
sum of all ranks' work over that time; the oracle arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.rank_info() == (rank, world, rank)
        local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
        tags = [bench.shard_tag(i, rank) for i in range(bench.NSETS)]
        out[rank] = (ms, tags, bench.job_throughput(2.0e12, world, ms))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_disjoint_shards():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        (ms0, tags0, tp0), (ms1, tags1, tp1) = out[0], out[1]
    assert ms0 == ms1 == 15.0                             # max over ranks, the same on both
    assert not set(tags0) & set(tags1) and len(set(tags0 + tags1)) == 2 * len(tags0)
    assert tp0 == tp1 == 2 * 2.0e12 / 15.0e-3 / 1e12      # both ranks' work over the slowest time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.job_throughput(1.0e12, 1, 1.0) == 1000.0       # 1 TOP in 1 ms


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
