"""The N > 1 benchmark protocol (independent replicas; barrier + max over ranks) with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2607_06519_b200 import replicas

    replicas.barrier(dist)
    local = 0.010 if rank == 0 else 0.025  # rank 1 is slower: it sets the job's time
    rate, sec = replicas.whole_job_rate(units_per_rank=50, local_seconds=local, dist=dist)
    out[rank] = (rate, sec, replicas.world(dist))
    dist.destroy_process_group()


def test_two_rank_weak_scaling_aggregate():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert len(out) == 2
    for rank in range(world):
        rate, sec, w = out[rank]
        assert w == 2
        assert abs(sec - 0.025) < 1e-12          # max over ranks
        assert abs(rate - 2 * 50 / 0.025) < 1e-6  # all ranks' units over the slowest rank's time


def test_single_process_passthrough():
    from paper_2607_06519_b200 import replicas

    rate, sec = replicas.whole_job_rate(10, 0.5, None)
    assert (rate, sec) == (20.0, 0.5)
    assert replicas.world(None) == 1
