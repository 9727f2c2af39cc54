"""The multi-GPU path is N independent replicas; its only distributed logic is the max over ranks
of the elapsed time.  Exercised here with two gloo processes on the CPU."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2309_06973_b200 import dist_util


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local = [10.0 + rank, 5.0 - rank]              # rank 1 is slower on the first, faster on the second
    got = dist_util.max_over_ranks(local)
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_figure():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29531, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 5.0]
    # 8 variants per replica, 2 replicas, slowest replica 1.6 ms per step -> 0.1 ms per variant job-wide
    assert abs(dist_util.ms_per_variant(1.6, 8, 2) - 0.1) < 1e-12


def test_single_process_is_identity():
    assert dist_util.max_over_ranks([3.5, 1.0]) == [3.5, 1.0]
