"""The multi-GPU path is independent replicas: the timing reduction, the gradient average of data-parallel
training and the patch split of sliding-window inference.  Checked with two gloo ranks on CPU."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2006_12575_b200 import replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 12.5            # rank 1 is the slow one
    out[rank] = (replicas.job_time_ms(local_ms), replicas.job_throughput(1000.0, local_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_job_time_is_the_slowest_rank_and_work_adds_up():
    assert replicas.job_time_ms(3.0) == 3.0 and replicas.job_throughput(6.0, 3.0) == 2000.0     # no process group
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29517 + os.getpid() % 200, out), nprocs=2, join=True)
    for rank in (0, 1):
        t, thr = out[rank]
        assert t == 12.5
        assert abs(thr - 2 * 1000.0 / 12.5e-3) < 1e-6


def _grad_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.arange(1000, dtype=torch.float32) * (rank + 1)          # rank 0: i, rank 1: 2 i
    replicas.allreduce_mean_(g, bucket_elems=96)                      # 11 buckets, the last one short
    out[rank] = g.tolist()
    dist.barrier()
    dist.destroy_process_group()


def test_gradient_average_over_two_replicas_in_buckets():
    g = torch.ones(5)
    assert replicas.allreduce_mean_(g) is g and g.tolist() == [1.0] * 5                          # no process group
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_grad_worker, args=(2, 29817 + os.getpid() % 200, out), nprocs=2, join=True)
    want = [1.5 * i for i in range(1000)]
    assert out[0] == want and out[1] == want


def test_patch_shards_cover_the_list_once():
    for n, world in ((363, 8), (27, 4), (5, 8), (0, 2)):
        seen = []
        for r in range(world):
            seen += list(replicas.shard_patches(n, r, world))
        assert seen == list(range(n))
        sizes = [len(replicas.shard_patches(n, r, world)) for r in range(world)]
        assert max(sizes) - min(sizes) <= 1


def test_bucket_plan_ends_on_layer_boundaries_and_grows_from_the_end():
    assert replicas.plan_buckets([0, 10, 30, 60, 100, 150], 200, 60) == [0, 100]       # [30, 100) and the short [0, 30) are one bucket
    assert replicas.plan_buckets([0], 5, 60) == [0]
    assert replicas.plan_buckets([0, 4, 8], 12, 1) == [0, 4, 8]
    starts = replicas.plan_buckets(list(range(0, 1000, 7)), 1000, 100)
    ends = starts[1:] + [1000]
    assert starts[0] == 0 and all(s % 7 == 0 for s in starts) and all(b - a >= 100 for a, b in zip(starts, ends))


def _overlap_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    layer_offsets = [0, 100, 250, 400, 700, 900]
    total = 1000
    starts = replicas.plan_buckets(layer_offsets, total, 300)
    g = torch.full((total,), float("nan"))
    avg = replicas.OverlappedGradientAverage(g, starts)
    ends = starts[1:] + [total]
    # the backward pass: layers finish last to first; a bucket is reported once its first layer has been written
    layer_ends = layer_offsets[1:] + [total]
    reported = []
    for lo, hi in reversed(list(zip(layer_offsets, layer_ends))):
        g[lo:hi] = torch.arange(lo, hi, dtype=torch.float32) * (rank + 1)
        for b in range(len(starts) - 1, -1, -1):
            if starts[b] >= lo and b not in reported:
                assert not torch.isnan(g[starts[b]:ends[b]]).any()       # nothing is exchanged before it is final
                avg.bucket_ready(b)
                reported.append(b)
    avg.finish()
    out[rank] = (g.tolist(), starts, reported)
    dist.barrier()
    dist.destroy_process_group()


def test_overlapped_gradient_average_starts_buckets_from_the_end_and_gives_the_mean():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_overlap_worker, args=(2, 30117 + os.getpid() % 200, out), nprocs=2, join=True)
    want = [1.5 * i for i in range(1000)]
    for rank in (0, 1):
        g, starts, reported = out[rank]
        assert g == want
        assert starts == [0, 400, 700] and reported == [2, 1, 0]
    # a bucket that is never reported is an error, not a silent partial average
    avg = replicas.OverlappedGradientAverage(torch.zeros(10), [0, 5])
    avg.bucket_ready(1)
    try:
        avg.finish()
        raise AssertionError("finish() accepted a missing bucket")
    except RuntimeError:
        pass


class _FakeSlidingWindow:
    """Stands in for the library's three sliding-window calls on CPU tensors: every patch predicts a constant
    class distribution that depends on its index, blended with the oracle's window."""

    def __init__(self, K):
        import numpy as np
        from oracle import unet as O
        self.np, self.O, self.K = np, O, K

    def _grid(self, D, H, W, patch, overlap):
        sd, sh, sw = (self.O.window_starts(n, p, overlap) for n, p in zip((D, H, W), patch))
        return [(a, b, c) for a in sd for b in sh for c in sw]

    def probs_of(self, i):
        v = self.np.arange(1, self.K + 1, dtype=self.np.float64) + (i % 5) * self.np.arange(self.K)[::-1]
        return v / v.sum()

    def lamp_sliding_window_num_patches(self, D, H, W, patch, overlap):
        return len(self._grid(D, H, W, patch, overlap))

    def lamp_sliding_window_partial(self, net, w, b, volume, patch, overlap, sw_batch, window, first, count, sums, wsum, ws):
        _, D, H, W, _ = volume.shape
        win = self.O.gaussian_window(patch) if window else self.np.ones(tuple(patch))
        acc = self.np.zeros((self.K, D, H, W))
        tot = self.np.zeros((D, H, W))
        for i, (a, b_, c) in enumerate(self._grid(D, H, W, patch, overlap)):
            if first <= i < first + count:
                sl = (slice(a, a + patch[0]), slice(b_, b_ + patch[1]), slice(c, c + patch[2]))
                acc[(slice(None),) + sl] += win[None] * self.probs_of(i)[:, None, None, None]
                tot[sl] += win
        sums.copy_(torch.from_numpy(acc))
        wsum.copy_(torch.from_numpy(tot))

    def lamp_sliding_window_finish(self, sums, wsum, K, V, write_probs, argmax):
        a = sums / wsum[None]
        if write_probs:
            sums.copy_(a)
        if argmax is not None:
            argmax.copy_(a.reshape(K, -1).argmax(0).to(torch.uint8))


def _sw_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    K, D, H, W, patch = 3, 12, 10, 9, (4, 4, 4)
    fake = _FakeSlidingWindow(K)
    vol = torch.zeros((1, D, H, W, 1))
    sums = torch.zeros((K, D, H, W), dtype=torch.float64)
    wsum = torch.zeros((D, H, W), dtype=torch.float64)
    seg = torch.zeros(D * H * W, dtype=torch.uint8)
    replicas.sliding_window_sharded(fake, None, None, None, vol, patch, 0.25, 2, 1, sums, wsum, seg, None, write_probs=True)
    out[rank] = (sums.numpy().copy(), seg.numpy().copy())
    dist.barrier()
    dist.destroy_process_group()


def test_patch_sharded_sliding_window_over_two_replicas_equals_the_oracle_blend():
    import numpy as np
    from oracle import unet as O
    K, D, H, W, patch = 3, 12, 10, 9, (4, 4, 4)
    fake = _FakeSlidingWindow(K)
    spec = O.UNetSpec(1, [2], 1, 1, K)
    A, seg_ref, n = O.sliding_window(spec, None, None, np.zeros((1, D, H, W, 1)), patch, 0.25, gaussian=True,
                                     patch_probs=lambda i, pa: np.broadcast_to(fake.probs_of(i), pa.shape[:4] + (K,)))
    assert n == fake.lamp_sliding_window_num_patches(D, H, W, patch, 0.25)
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_sw_worker, args=(2, 30417 + os.getpid() % 200, out), nprocs=2, join=True)
    for rank in (0, 1):
        probs, seg = out[rank]
        np.testing.assert_allclose(probs.transpose(1, 2, 3, 0), A, rtol=1e-12)
        assert (seg.reshape(D, H, W) == seg_ref).all()
