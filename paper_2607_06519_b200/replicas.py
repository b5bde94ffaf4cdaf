"""Host-side logic of the N-GPU benchmark: independent replicas, no collective on the data path.

The hot path has no exchange step (units are independent; the build targets one GPU), so `bench.py --gpus N` runs one
replica per rank.  The only communication is the measurement protocol: a barrier before the timed region and a MAX
over the ranks' device-measured times, from which the whole-job throughput follows.  Works with any
torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch


def world(dist) -> int:
    return dist.get_world_size() if dist is not None and dist.is_initialized() else 1


def barrier(dist) -> None:
    if dist is not None and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The slowest rank's time: every rank gets the same number."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, local_seconds: float, dist, device="cpu"):
    """(aggregate units/s over all ranks, max seconds): every rank processed `units_per_rank` units (weak scaling)."""
    sec = max_over_ranks(local_seconds, dist, device)
    return world(dist) * units_per_rank / sec, sec
