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
    group (or with one rank) the buffer is returned untouched.  This form starts after the backward pass;
    OverlappedGradientAverage starts each bucket while the backward pass is still running.
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


def plan_buckets(layer_offsets, total: int, bucket_elems: int):
    """Cuts a flat gradient buffer of `total` elements into buckets that end on layer boundaries.

    layer_offsets: ascending start offsets of the layers (the first is 0).  The backward pass finishes the layers
    last to first, so the buckets are grown from the END of the buffer: a bucket is closed as soon as it holds at
    least bucket_elems elements (a shorter leftover at the front joins its neighbour).  Returns the ascending list of bucket start offsets (the first is 0); bucket b
    covers [start[b], start[b + 1]) and the last one ends at `total`.
    """
    offs = sorted(set(int(o) for o in layer_offsets))
    if not offs or offs[0] != 0 or offs[-1] >= total:
        raise ValueError("layer offsets must start at 0 and lie inside the buffer")
    starts, end = [], total
    for o in reversed(offs):
        if end - o >= bucket_elems or o == 0:
            starts.append(o)
            end = o
    starts = starts[::-1]
    if len(starts) > 1 and starts[1] < bucket_elems:          # a short leftover at the front joins its neighbour
        del starts[1]
    return starts


class OverlappedGradientAverage:
    """Average of a flat gradient buffer over the replicas, bucket by bucket, each bucket started as soon as the
    backward pass has finished it (Sec. 1 of the paper: data parallelism; the exchange hides behind the rest of
    the backward pass instead of following it).

    The producer reports progress with bucket_ready(b) - buckets become final from the last to the first - and
    calls finish() after the step.  On GPUs the all-reduces run on a communication stream that waits for the event
    the training step recorded for the bucket (lamp_unet_train_step_buckets); on CPU tensors (gloo, used by the
    tests) a bucket is reduced when it is reported.  The data of a peer only ever lands in this rank's own buffer
    through the collective library; no kernel of the library is given a peer's memory.
    """

    def __init__(self, flat: torch.Tensor, bucket_start, comm_stream=None):
        if flat.dim() != 1 or not flat.is_contiguous():
            raise ValueError("OverlappedGradientAverage wants a flat contiguous buffer")
        self.flat = flat
        self.starts = [int(v) for v in bucket_start]
        self.ends = self.starts[1:] + [flat.numel()]
        self.world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
        self.comm_stream = comm_stream
        self.works = []
        self.order = []                       # buckets in the order their exchange was started

    def bucket_ready(self, b: int, event=None):
        """Bucket b of the buffer is final (event: the CUDA event that says so on the device)."""
        self.order.append(b)
        if self.world == 1:
            return
        view = self.flat[self.starts[b]:self.ends[b]]
        if self.comm_stream is not None:
            if event is not None:
                self.comm_stream.wait_event(event)
            with torch.cuda.stream(self.comm_stream):
                self.works.append(dist.all_reduce(view, op=dist.ReduceOp.SUM, async_op=True))
        else:
            self.works.append(dist.all_reduce(view, op=dist.ReduceOp.SUM, async_op=True))

    def finish(self):
        """Waits for every bucket and divides by the number of replicas; the buffer then holds the average."""
        if sorted(self.order) != list(range(len(self.starts))):
            raise RuntimeError("not every bucket was reported ready exactly once")
        for w in self.works:
            w.wait()
        if self.comm_stream is not None:
            torch.cuda.current_stream().wait_stream(self.comm_stream)
        if self.world > 1:
            self.flat.mul_(1.0 / self.world)
        self.works, self.order = [], []
        return self.flat


def train_step_overlapped(binding, net, weights, biases, x, labels, loss, grad_w, grad_b, probs, ws, bucket_start,
                          events, comm_stream):
    """One data-parallel training step on this rank: lamp_unet_train_step_buckets, with the all-reduce of every
    gradient bucket started on comm_stream behind the event the step records for it; the bias gradients (small)
    follow at the end.  Returns after enqueueing; grad_w and grad_b hold the averages in stream order."""
    avg = OverlappedGradientAverage(grad_w, bucket_start, comm_stream)
    binding.lamp_unet_train_step_buckets(net, weights, biases, x, labels, loss, grad_w, grad_b, probs, ws, bucket_start, events)
    for b in range(len(bucket_start) - 1, -1, -1):           # the order in which the step finishes them
        avg.bucket_ready(b, events[b])
    avg.finish()
    allreduce_mean_(grad_b)
    return avg


def sliding_window_sharded(binding, net, weights, biases, volume, patch, overlap, sw_batch, window, sums_planar,
                           weight_sums, argmax, ws, write_probs=False):
    """Sliding-window inference with the patches split over the replicas: this rank runs its share
    (shard_patches), the un-normalised class sums and weight totals are added over the ranks, and every rank
    divides and takes the arg max.  sums_planar [K][D][H][W] and weight_sums [D][H][W] are fp32 buffers of this
    rank; with write_probs the former ends up holding the blended probabilities."""
    _, D, H, W, _ = volume.shape
    K = sums_planar.shape[0]
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    rank = dist.get_rank() if world > 1 else 0
    n = binding.lamp_sliding_window_num_patches(D, H, W, patch, overlap)
    mine = shard_patches(n, rank, world)
    binding.lamp_sliding_window_partial(net, weights, biases, volume, patch, overlap, sw_batch, window, mine.start, len(mine),
                                        sums_planar, weight_sums, ws)
    if world > 1:
        dist.all_reduce(sums_planar, op=dist.ReduceOp.SUM)
        dist.all_reduce(weight_sums, op=dist.ReduceOp.SUM)
    binding.lamp_sliding_window_finish(sums_planar, weight_sums, K, D * H * W, write_probs, argmax)
