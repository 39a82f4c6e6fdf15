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
