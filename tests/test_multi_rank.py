"""The N > 1 bench path on CPU: two gloo ranks, timing reduced as the maximum over ranks, whole-job throughput of
independent replicas.  (The LAQ path itself does not shard across GPUs and has no collective: bench.py --gpus N runs
N replicas.)"""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, world, device="cpu")
    dist.barrier()
    value = bench.replicas_throughput(world, 200, ms)
    with open(os.path.join(out_dir, "rank%d.txt" % rank), "w") as f:
        f.write("%r %r" % (ms, value))
    dist.destroy_process_group()


def test_two_ranks_time_is_the_maximum_and_value_is_the_whole_job(tmp_path):
    world, port = 2, 29000 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        ms, value = (float(v) for v in open(tmp_path / ("rank%d.txt" % rank)).read().split())
        assert ms == 15.0                              # every rank sees the slowest rank's time
        assert value == pytest.approx(2 * 200 / 0.015)


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.replicas_throughput(1, 100, 50.0) == pytest.approx(2000.0)
