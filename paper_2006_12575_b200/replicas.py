"""Host-side bookkeeping for replica runs (one process per GPU, no data-path collective).

The convolution path shards only by independent volumes, so N GPUs run N copies of the same work.
The job's throughput is the work of all ranks over the slowest rank's device time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def job_time_ms(local_ms: float, device=None) -> float:
    """Max over ranks of a per-rank device time (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def job_throughput(units_per_rank: float, local_ms: float, device=None) -> float:
    """Units processed by all ranks per second, timed by the slowest rank."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / (job_time_ms(local_ms, device) * 1e-3)
