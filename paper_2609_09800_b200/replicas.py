"""Multi-GPU use of the library: independent replicas, one per rank (replicas only).

The service model of one package runs on one GPU; nothing is exchanged between ranks on the data path.
What a multi-rank run needs is bookkeeping: every rank serves its own seeded stream, and the job's rate is
the units all ranks served divided by the slowest rank's device time.  These helpers do that reduction over
any ``torch.distributed`` process group (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the stream a rank generates: distinct per rank, reproducible."""
    return int(base_seed) * 1000 + int(rank)


def combine(local_units: float, local_ms: float, device: str = "cpu", group=None):
    """Returns (units summed over ranks, max device time over ranks in ms)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(local_units), float(local_ms)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(u.item()), float(t.item())


def job_rate(local_units: float, local_ms: float, device: str = "cpu", group=None) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    units, ms = combine(local_units, local_ms, device, group)
    return units / (ms * 1e-3) if ms > 0 else 0.0
