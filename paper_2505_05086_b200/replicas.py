"""Host-side bookkeeping for running the ASI path as independent data-parallel replicas.

The method is per-device: every replica compresses its own micro-batch with its own factors, so the
hot path has no collective.  The only cross-rank step is how a multi-GPU measurement is reduced:
the slowest rank's device time bounds the job, and the job's throughput is the units all ranks
processed divided by that time."""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks of the default process group (the value itself without one)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, ms_local: float, device="cpu"):
    """(whole-job units per second, max-over-ranks milliseconds) for replicas that each processed
    `units_per_rank` units in `ms_local` milliseconds of device time."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    ms = max_over_ranks(ms_local, device)
    return world * units_per_rank / (ms * 1e-3), ms
