"""Host logic of the paper's pipeline (Sec. 2.1 Eq. 1, Sec. 2.2 Eq. 3): the sequentialised U-Net, the balanced
partitioner, the micro-batch schedule and its execution over two gloo ranks on CPU."""
import itertools
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2006_12575_b200 import pipeline as PL


def test_sequential_unet_carries_every_skip_and_can_be_cut_anywhere():
    st = PL.sequential_unet_stages(5, [32, 64, 128, 256, 512], 2, 1, 10)
    names = [s.name for s in st]
    # 5 encoder blocks of 2 convs, 4 down convs, 4 (up, 2 convs), head; one keep / concat per skip (four skips, Eq. 2)
    assert sum(s.kind == "conv" for s in st) == 18 and sum(s.kind == "down" for s in st) == 4
    assert sum(s.kind == "up" for s in st) == 4 and names[-1] == "head"
    assert [s.name for s in st if s.kind == "keep"] == ["keep0", "keep1", "keep2", "keep3"]
    assert [s.name for s in st if s.kind == "concat"] == ["concat3", "concat2", "concat1", "concat0"]
    # run the state machine: the skip stack is never popped empty and ends empty (every e_{i,1} is used exactly once)
    depth = 0
    for s in st:
        if s.kind == "keep":
            depth += 1
        elif s.kind == "concat":
            assert depth > 0
            depth -= 1
    assert depth == 0
    # level-0 convs carry most of the cost (the sweep's reason to exist)
    top = sum(s.cost for s in st if s.level == 0 and s.kind == "conv")
    assert top / sum(s.cost for s in st) > 0.4


def _brute(costs, K):
    n = len(costs)
    best = None
    for cuts in itertools.combinations(range(1, n), K - 1):
        b = [0] + list(cuts) + [n]
        v = max(sum(costs[b[i]:b[i + 1]]) for i in range(K))
        best = v if best is None or v < best else best
    return best


def test_balanced_partition_is_optimal_on_small_cases():
    rs = torch.Generator().manual_seed(0)
    for n, K in ((5, 2), (7, 3), (9, 4), (6, 6), (3, 5)):
        costs = (torch.rand(n, generator=rs) * 10).tolist()
        parts = PL.partition_balanced(costs, K)
        assert parts[0][0] == 0 and parts[-1][1] == n and all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        assert all(e > s for s, e in parts) and len(parts) == min(K, n)
        got = max(sum(costs[s:e]) for s, e in parts)
        assert abs(got - _brute(costs, min(K, n))) < 1e-12
    assert PL.partition_balanced([1, 1, 1, 1], 2) == [(0, 2), (2, 4)]
    # the U-Net over 4 devices: no partition costs more than twice the mean
    st = PL.sequential_unet_stages(5, [32, 64, 128, 256, 512], 2, 1, 10)
    costs = [s.cost for s in st]
    parts = PL.partition_balanced(costs, 4)
    assert max(sum(costs[s:e]) for s, e in parts) <= 2.0 * sum(costs) / 4


def test_schedule_orders_dependencies_and_has_the_published_bubble():
    for K, M in ((1, 1), (3, 4), (4, 2), (2, 8)):
        ticks = PL.gpipe_schedule(K, M)
        assert len(ticks) == 2 * (M + K - 1)
        when = {}
        for t, entries in enumerate(ticks):
            ks = [k for k, m, d in entries]
            assert len(ks) == len(set(ks))                           # a partition does one thing per tick
            for k, m, d in entries:
                when[(k, m, d)] = t
        assert len(when) == 2 * K * M
        for k in range(K):
            for m in range(M):
                if k > 0:
                    assert when[(k, m, "F")] > when[(k - 1, m, "F")]     # F_k needs F_{k-1}'s output
                    assert when[(k - 1, m, "B")] > when[(k, m, "B")]     # B_{k-1} needs B_k's gradient
                assert when[(k, m, "B")] > when[(K - 1, m, "F")]         # backward after the loss of that micro-batch
        busy = sum(len(e) for e in ticks)
        assert abs((1 - busy / (K * len(ticks))) - PL.bubble_fraction(K, M)) < 1e-12
    # the appendix example: 3 devices; t/2 batches per device-time conventionally (1 of 3 devices busy at a time would be
    # t/3; the paper counts forward + backward), pipelined with M = 3 micro-batches the bubble is (K-1)/(M+K-1) = 2/5
    assert PL.bubble_fraction(3, 3) == 0.4
    assert PL.activation_memory_units(16, 40, 4, 8) == 16 + 10 * 2 and PL.activation_memory_units(16, 40, 1, 1, False) == 640


class _ToyStage(PL.PipelineStage):
    """A partition of a toy sequential U-Net in torch (CPU): a few 3-D convs with one skip that crosses the cut, carried
    in the state as Eq. 3 prescribes."""

    def __init__(self, rank, seed=0):
        g = torch.Generator().manual_seed(seed)
        mk = lambda co, ci: (torch.randn(co, ci, 3, 3, 3, generator=g, dtype=torch.float64) * 0.2).requires_grad_(True)
        w = [mk(4, 1), mk(4, 4), mk(4, 4), mk(2, 8)]      # enc conv, (keep), mid conv | mid conv 2, concat, head conv
        self.rank = rank
        self.params = w[:2] if rank == 0 else w[2:]
        self.saved = {}

    def _run(self, state):
        conv = lambda x, w: torch.relu(torch.nn.functional.conv3d(x, w, padding=1))
        if self.rank == 0:
            (x,) = state
            e = conv(x, self.params[0])
            a = conv(e, self.params[1])
            return [a, e]                                   # activation and the kept skip e_{1,1} cross the boundary
        a, e = state
        a = conv(a, self.params[0])
        y = torch.nn.functional.conv3d(torch.cat([e, a], dim=1), self.params[1], padding=1)
        return [(y ** 2).mean()]

    def forward(self, m, state):
        ins = [t.clone().requires_grad_(self.rank > 0) for t in state]
        outs = self._run(ins)
        self.saved[m] = (ins, outs)
        return [o.detach() for o in outs]

    def backward(self, m, grads):
        ins, outs = self.saved.pop(m)
        if grads is None:
            outs[0].backward()
        else:
            torch.autograd.backward(outs, grads)
        return [t.grad for t in ins] if self.rank > 0 else []

    def incoming(self, m):
        return [torch.empty(1, 4, 4, 4, 4, dtype=torch.float64), torch.empty(1, 4, 4, 4, 4, dtype=torch.float64)]

    def outgoing(self, m):
        return self.incoming(m)


def _pipe_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    M = 3
    g = torch.Generator().manual_seed(5)
    batches = [[torch.randn(1, 1, 4, 4, 4, generator=g, dtype=torch.float64)] for _ in range(M)]
    stage = _ToyStage(rank)
    losses = PL.run_pipeline(stage, batches, M)
    out[rank] = ([float(l[0]) for l in losses], [p.grad.clone() for p in stage.params])
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_pipeline_accumulates_the_same_gradients_as_one_device():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_pipe_worker, args=(2, 30717 + os.getpid() % 200, out), nprocs=2, join=True)
    # one device: both partitions back to back on every micro-batch, gradients summed
    M = 3
    g = torch.Generator().manual_seed(5)
    batches = [[torch.randn(1, 1, 4, 4, 4, generator=g, dtype=torch.float64)] for _ in range(M)]
    s0, s1 = _ToyStage(0), _ToyStage(1)
    ref_losses = []
    for b in batches:
        mid = s0._run(b)
        loss = s1._run(mid)[0]
        loss.backward()
        ref_losses.append(float(loss.detach()))
    assert out[0][0] == [] and out[1][0] == pytest.approx(ref_losses, rel=1e-12)
    for got, ref in zip(out[0][1], s0.params):
        assert torch.allclose(got, ref.grad, rtol=1e-10, atol=1e-14)
    for got, ref in zip(out[1][1], s1.params):
        assert torch.allclose(got, ref.grad, rtol=1e-10, atol=1e-14)


def test_forward_only_schedule_is_the_first_half():
    assert PL.forward_schedule(3, 4) == PL.gpipe_schedule(3, 4)[:6]
    assert sum(len(t) for t in PL.forward_schedule(3, 4)) == 12
    assert all(d == "F" for t in PL.forward_schedule(2, 5) for (_, _, d) in t)
