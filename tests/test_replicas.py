"""The multi-GPU path is independent replicas; its only cross-rank step is the timing reduction.
Checked with two gloo ranks on CPU."""
import os

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
