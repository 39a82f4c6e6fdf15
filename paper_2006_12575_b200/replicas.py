"""Host-side pieces of replica (data-parallel) runs: one process per GPU.

The convolution path shards only by independent volumes, so N GPUs run N copies of the same work and the
job's throughput is the work of all ranks over the slowest rank's device time.  Training adds the one real
exchange of data parallelism (Sec. 1 of the paper): the flat fp32 gradient buffers of a step are averaged over
the replicas before the parameter update, here by bucketed all-reduces of the process group (NCCL on GPUs).
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


def allreduce_mean_(flat: torch.Tensor, bucket_elems: int = 16 << 20) -> torch.Tensor:
    """Averages a flat gradient buffer over all replicas, in place, bucket by bucket.

    Every bucket is its own asynchronous all-reduce, so that the first buckets travel while the later ones are
    still being enqueued; the division by the world size follows once all have completed.  Without a process
    group (or with one rank) the buffer is returned untouched.  The training step hands back all gradients at
    once, so the exchange starts after the backward pass; overlapping it with the backward pass would need the
    step split at layer boundaries and is not built.
    """
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return flat
    if flat.dim() != 1 or not flat.is_contiguous():
        raise ValueError("allreduce_mean_ wants a flat contiguous buffer")
    works = []
    for start in range(0, flat.numel(), bucket_elems):
        works.append(dist.all_reduce(flat[start:start + bucket_elems], op=dist.ReduceOp.SUM, async_op=True))
    for w in works:
        w.wait()
    flat.mul_(1.0 / dist.get_world_size())
    return flat


def shard_patches(num_patches: int, rank: int, world: int) -> range:
    """Contiguous share of a sliding-window patch list for one replica (the first ranks take the remainder)."""
    base, rem = divmod(num_patches, world)
    start = rank * base + min(rank, rem)
    return range(start, start + base + (1 if rank < rem else 0))
