"""Host-side logic for running the path on several GPUs of one node.

The (batch, query head) units of the SparQ step are independent, so the path shards by batch with
no data-path collective: every rank owns its own sequences (its own cache) and runs the same
kernels.  The only cross-rank traffic is bookkeeping for measurement: a barrier, and the maximum
over ranks of a device-measured duration.  These helpers are backend-agnostic (NCCL on GPUs, gloo
in the CPU tests).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def env_rank() -> Tuple[int, int, int]:
    """(world_size, rank, local_rank) as torchrun exports them; (1, 0, 0) when run plainly."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def shard_batch(B_total: int, world: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the sequences rank owns when B_total sequences are split as evenly as possible
    (the first B_total % world ranks get one more)."""
    base, extra = divmod(B_total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_seed(base_seed: int, rank: int) -> int:
    """Distinct, reproducible workload seed per rank (weak scaling: every rank draws its own batch)."""
    return base_seed + 1000 * rank


def max_over_ranks(x: float, device: Optional[torch.device] = None) -> float:
    """Maximum of a per-rank scalar (a duration); identity when no process group is up."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device: Optional[torch.device] = None) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_this_rank: int, seconds_this_rank: float, device: Optional[torch.device] = None) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return sum_over_ranks(units_this_rank, device) / max_over_ranks(seconds_this_rank, device)
