"""N > 1 is N independent replicas: the cross-rank logic (max time over ranks, whole-job rate)
is exercised here with two gloo ranks on CPU."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2106_08301_b200 import replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 2.0 if rank == 0 else 3.5            # rank 1 is the slow one
    agreed = replicas.max_over_ranks(ms, dist)
    dist.barrier()
    out[rank] = agreed
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29541, out), nprocs=world, join=True)
    assert out[0] == 3.5 and out[1] == 3.5
    # two replicas, 7 units each, 3.5 ms -> 4000 units/s
    assert replicas.whole_job_rate(7.0, world, out[0]) == 4000.0


def test_single_process_passthrough():
    assert replicas.max_over_ranks(1.25) == 1.25
    assert replicas.whole_job_rate(10.0, 1, 5.0) == 2000.0
