"""Host-side logic for runs on several GPUs (one process per GPU).

Tensors of a model are independent problems: the quantizer couples the elements of one tensor
only (through its global scale), so a multi-GPU job shards by tensor and needs no collective
on the data path.  What the ranks do exchange is bookkeeping: a barrier around the timed
region and the maximum over ranks of a device-side time.  Those go through
``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from dataclasses import replace

import torch
import torch.distributed as dist


def assign_tensors(n_tensors: int, rank: int, world: int) -> list[int]:
    """Indices of the tensors rank ``rank`` quantizes when ``n_tensors`` independent tensors are
    dealt round-robin to ``world`` ranks (strong scaling: the total work is fixed)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    return list(range(rank, n_tensors, world))


def rank_workload(wl, rank: int):
    """The workload rank ``rank`` quantizes under weak scaling: the same shapes and distribution,
    drawn from a seed of its own (a different layer of the same model)."""
    return wl if rank == 0 else replace(wl, name=f"{wl.name}_rank{rank}", seed=wl.seed + 7919 * rank)


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (a time) over all ranks; the value itself on one rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    """Sum of a per-rank scalar (units of work done) over all ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return sum_over_ranks(units_this_rank, device) / max_over_ranks(seconds_this_rank, device)
