"""Host side of the paper's own method: the sequentialised U-Net cut into K partitions and run as a micro-batch
pipeline (Sec. 2.1, Eq. 1; Sec. 2.2, Eq. 3).

On one B200 every listed network fits unsplit, so the library itself runs no pipeline; what is here is the logic a
multi-GPU pipeline needs on the host, testable with CPU ranks, and (at the end) partitions of whole-volume inference
that run the library's kernels:

* sequential_unet_stages: the U-Net as a plain sequence of steps acting on a state (activation, stack of skips).
  Eq. 3 duplicates every encoder output as e_{i,0} (fed to the next block) and e_{i,1} (kept for the skip); carrying
  e_{i,1} along in the state is what removes the long-range dependency and lets the sequence be cut anywhere.
* partition_balanced: cuts a sequence of per-step costs into K contiguous partitions with the smallest possible
  largest partition (the automated part of the method: Eq. 1's F_k = f_j o ... o f_i with balanced cost).
* gpipe_schedule: which (partition, micro-batch, direction) runs at which clock tick for M micro-batches over K
  partitions, forward then backward, gradients accumulated synchronously; bubble fraction (K - 1) / (M + K - 1).
* activation_memory_units: the memory argument of Sec. 2.1, O(N + L/K * N/M) with re-materialisation against O(N * L).
* run_pipeline: executes the schedule over the ranks of a torch.distributed group (one partition per rank, given as a
  PipelineStage).  A state crossing a partition boundary is sent to the next rank and received into that rank's own
  memory before any of its steps reads it; nothing ever computes on a peer's memory.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


@dataclass
class Stage:
    name: str
    kind: str            # 'conv', 'down', 'up', 'head' (as in the network's layer list), or 'keep' / 'concat'
    level: int
    cost: float          # relative cost (FLOPs of the step at unit volume), 0 for the bookkeeping steps


def sequential_unet_stages(levels: int, channels: Sequence[int], convs_per_level: int, in_channels: int, num_classes: int) -> List[Stage]:
    """The sequential U-Net of Eq. 3 as steps on a state (a, skips): 'keep' pushes a copy of the activation (e_{i,1})
    onto the skip stack, 'concat' pops the matching one in front of the up-sampled activation."""
    out: List[Stage] = []
    c = in_channels
    vox = [8.0 ** -l for l in range(levels)]
    for l in range(levels):
        for j in range(convs_per_level):
            out.append(Stage(f"enc{l}.conv{j}", "conv", l, 2 * 27 * c * channels[l] * vox[l]))
            c = channels[l]
        if l < levels - 1:
            out.append(Stage(f"keep{l}", "keep", l, 0.0))
            out.append(Stage(f"down{l}", "down", l + 1, 2 * 27 * channels[l] * channels[l + 1] * vox[l + 1]))
            c = channels[l + 1]
    for l in range(levels - 2, -1, -1):
        out.append(Stage(f"up{l}", "up", l, 2 * channels[l + 1] * channels[l] * vox[l]))
        out.append(Stage(f"concat{l}", "concat", l, 0.0))
        c = 2 * channels[l]
        for j in range(convs_per_level):
            out.append(Stage(f"dec{l}.conv{j}", "conv", l, 2 * 27 * c * channels[l] * vox[l]))
            c = channels[l]
    out.append(Stage("head", "head", 0, 2 * channels[0] * num_classes * vox[0]))
    return out


def partition_balanced(costs: Sequence[float], K: int) -> List[Tuple[int, int]]:
    """Contiguous partitions [(start, end), ...] of the steps, K of them (fewer if there are fewer steps), such that the
    largest partition cost is minimal (dynamic programme over prefix sums; ties go to the earlier cut)."""
    n = len(costs)
    if n == 0 or K < 1:
        raise ValueError("need at least one step and one partition")
    K = min(K, n)
    pre = [0.0]
    for c in costs:
        pre.append(pre[-1] + float(c))
    INF = float("inf")
    best = [[INF] * (n + 1) for _ in range(K + 1)]
    cut = [[0] * (n + 1) for _ in range(K + 1)]
    best[0][0] = 0.0
    for k in range(1, K + 1):
        for i in range(k, n + 1):
            for j in range(k - 1, i):
                v = max(best[k - 1][j], pre[i] - pre[j])
                if v < best[k][i]:
                    best[k][i], cut[k][i] = v, j
    parts, i = [], n
    for k in range(K, 0, -1):
        j = cut[k][i]
        parts.append((j, i))
        i = j
    return parts[::-1]


def gpipe_schedule(K: int, M: int):
    """Clock ticks of the synchronous micro-batch pipeline: a list of ticks, each a list of (partition, micro_batch,
    'F' | 'B').  Forward of micro-batch m on partition k runs at tick m + k; backward at tick (M + K - 1) + (M - 1 - m)
    + (K - 1 - k); the parameter update follows the last tick."""
    if K < 1 or M < 1:
        raise ValueError("K and M must be positive")
    T = M + K - 1
    ticks = [[] for _ in range(2 * T)]
    for m in range(M):
        for k in range(K):
            ticks[m + k].append((k, m, "F"))
            ticks[T + (M - 1 - m) + (K - 1 - k)].append((k, m, "B"))
    return ticks


def forward_schedule(K: int, M: int):
    """The forward half alone (pipelined inference of M volumes over K partitions): M + K - 1 ticks."""
    return gpipe_schedule(K, M)[:M + K - 1]


def bubble_fraction(K: int, M: int) -> float:
    """Share of partition-ticks in which a partition idles: (K - 1) / (M + K - 1)."""
    return (K - 1) / (M + K - 1)


def activation_memory_units(N: int, L: int, K: int, M: int, rematerialise: bool = True) -> float:
    """Peak activation memory of one device in units of (one sample x one layer), Sec. 2.1: without the pipeline a
    device keeps N * L; with K partitions, M micro-batches and re-materialisation it keeps the N boundary inputs of
    its partition plus the L / K layers of the one micro-batch (N / M samples) whose backward is running."""
    if not rematerialise:
        return float(N) * L / K
    return float(N) + (L / K) * (N / M)


class PipelineStage:
    """What run_pipeline needs from the partition a rank owns.

    forward(m, state) -> state        state: list of tensors (rank 0 gets micro-batch m, the last rank returns its loss)
    backward(m, grads) -> grads       grads: gradients of the state this rank sent forward (None on the last rank);
                                      returns the gradients of the state it received (ignored on rank 0);
                                      parameter gradients accumulate inside the stage over the micro-batches
    incoming(m) -> list of empty tensors with the shapes of the state that enters this rank for micro-batch m
    outgoing(m) -> list of empty tensors with the shapes of the state this rank sent forward for micro-batch m
    """

    def forward(self, m, state):
        raise NotImplementedError

    def backward(self, m, grads):
        raise NotImplementedError

    def incoming(self, m):
        raise NotImplementedError

    def outgoing(self, m):
        raise NotImplementedError


def run_pipeline(stage: PipelineStage, micro_batches: Sequence, M: int, group=None, forward_only: bool = False):
    """Runs gpipe_schedule(world, M) (forward_only: forward_schedule) with one partition per rank of `group`: every rank
    executes its own entries of every tick in order.  Boundary states and their gradients travel by send / recv between neighbouring ranks: the
    receiver owns the memory they land in.  Returns the last partition's forward outputs (other ranks: [])."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    outs = []
    for tick in (forward_schedule(world, M) if forward_only else gpipe_schedule(world, M)):
        for (k, m, direction) in tick:
            if k != rank:
                continue
            if direction == "F":
                if rank == 0:
                    state = micro_batches[m]
                else:
                    state = stage.incoming(m)
                    for t in state:
                        dist.recv(t, src=rank - 1, group=group)
                res = stage.forward(m, state)
                if rank == world - 1:
                    outs.append(res)
                else:
                    for t in res:
                        dist.send(t.contiguous(), dst=rank + 1, group=group)
            else:
                grads = None
                if rank < world - 1:
                    grads = stage.outgoing(m)
                    for t in grads:
                        dist.recv(t, src=rank + 1, group=group)
                gin = stage.backward(m, grads)
                if rank > 0:
                    for t in gin:
                        dist.send(t.contiguous(), dst=rank - 1, group=group)
    return outs


# ------------------------------------------------------------------------------------------------------
# Partitions that run the library's kernels: whole-volume inference cut into F_1 ... F_K (Eq. 1), every partition a
# range of layers executed by lamp_unet_forward_layers in its own workspace.  What crosses a cut is exactly the
# state of the sequential U-Net (Eq. 3): the activation entering the first layer of the partition and every kept
# encoder output e_{i,1} whose skip crosses the cut (plus, in the SEU-Net variant, the first conv's output of a
# level whose stack is cut in the middle).
# ------------------------------------------------------------------------------------------------------
def library_layers(binding, net):
    """Kinds and sizes of the library's layers, derived from lamp_unet_param_layout / lamp_unet_se_layout."""
    out = []
    for i in range(binding.lamp_unet_num_layers(net)):
        _, _, d = binding.lamp_unet_param_layout(net, i)
        kind = "up" if d.transposed else "head" if d.ksize == 1 else "down" if d.stride == 2 else "conv"
        _, cr = binding.lamp_unet_se_layout(net, i)
        out.append(dict(kind=kind, c_in=d.c_in, c_out=d.c_out, se=cr > 0))
    return out


def boundary_tensors(layers, cut, convs_per_level):
    """What the partition that starts at layer `cut` needs from earlier layers: a list of (layer, 'in' | 'out')."""
    need = [(cut, "in")]
    # skips: the last conv of encoder level l (followed by a down conv) is read again by the conv behind up conv l;
    # encoder levels are entered in order, decoder levels left in reverse order
    enc_last = [i for i, ly in enumerate(layers[:-1]) if ly["kind"] == "conv" and layers[i + 1]["kind"] == "down"]
    ups = [i for i, ly in enumerate(layers) if ly["kind"] == "up"]
    for l, i in enumerate(enc_last):
        consumer = ups[len(ups) - 1 - l] + 1
        if i < cut <= consumer and (i, "out") not in need:
            need.append((i, "out"))
    for j, ly in enumerate(layers):
        first = j - (convs_per_level - 1)
        if ly["se"] and j >= cut > first:
            need.append((first, "out"))
    return need


def _tensor_view(binding, net, shape, ws, layer, which):
    import torch as _t
    n, d, h, w = shape
    t, off = binding.lamp_unet_tensor_layout(net, n, d, h, w, binding.MODE_INFER, layer, binding.T_IN if which == "in" else binding.T_OUT)
    V = t.n * t.d * t.h * t.w
    flat = ws[off:off + ((V - 1) * t.c_pitch + t.c) * 2].view(_t.bfloat16)
    return _t.as_strided(flat, (V, t.c), (t.c_pitch, 1))


def copy_boundary(binding, net, shape, need, ws_src, ws_dst):
    """Copies the boundary tensors from one partition's workspace into the next one's (same layout in both)."""
    for layer, which in need:
        _tensor_view(binding, net, shape, ws_dst, layer, which).copy_(_tensor_view(binding, net, shape, ws_src, layer, which))


def partitioned_forward(binding, net, weights, biases, x, cuts, workspaces, probs, argmax, convs_per_level=2):
    """Whole-volume inference as K partitions run one after the other, partition k in workspaces[k] (on one device
    this is the pipeline's arithmetic without its overlap; over several devices every rank runs its own partition and
    the boundary tensors travel by send / recv into the receiver's workspace).  cuts: ascending first layers of
    partitions 1 .. K-1."""
    layers = library_layers(binding, net)
    n, d, h, w = x.shape[0], x.shape[1], x.shape[2], x.shape[3]
    bounds = [0] + list(cuts) + [len(layers)]
    for k in range(len(bounds) - 1):
        if k > 0:
            copy_boundary(binding, net, (n, d, h, w), boundary_tensors(layers, bounds[k], convs_per_level), workspaces[k - 1], workspaces[k])
        last = k == len(bounds) - 2
        binding.lamp_unet_forward_layers(net, weights, biases, x, bounds[k], bounds[k + 1], probs if last else None,
                                         argmax if last else None, workspaces[k])


class LibraryPartition(PipelineStage):
    """One partition of pipelined whole-volume inference on this rank's GPU: layers [first, last) through
    lamp_unet_forward_layers in this rank's own workspace.  forward() takes the boundary state as contiguous tensors
    (as received from the previous rank), copies it to where the layers expect it, runs the layers and returns the
    state for the next rank (the last partition returns clones of probs and argmax)."""

    def __init__(self, binding, net, weights, biases, shape, first, last, workspace, x_like, convs_per_level=2,
                 probs=None, argmax=None):
        self.b, self.net, self.w, self.bias = binding, net, weights, biases
        self.shape, self.first, self.last, self.ws, self.x_like = tuple(shape), first, last, workspace, x_like
        self.probs, self.argmax = probs, argmax
        self.layers = library_layers(binding, net)
        self.need_in = boundary_tensors(self.layers, first, convs_per_level) if first > 0 else []
        self.need_out = boundary_tensors(self.layers, last, convs_per_level) if last < len(self.layers) else []

    def _views(self, need):
        return [_tensor_view(self.b, self.net, self.shape, self.ws, layer, which) for layer, which in need]

    def incoming(self, m):
        return [torch.empty(v.shape, dtype=v.dtype, device=v.device) for v in self._views(self.need_in)]

    def outgoing(self, m):
        return [torch.empty(v.shape, dtype=v.dtype, device=v.device) for v in self._views(self.need_out)]

    def forward(self, m, state):
        x = self.x_like
        if self.first == 0:
            x = state[0]
        else:
            for dst, src in zip(self._views(self.need_in), state):
                dst.copy_(src)
        is_last = self.last == len(self.layers)
        self.b.lamp_unet_forward_layers(self.net, self.w, self.bias, x, self.first, self.last, self.probs if is_last else None,
                                        self.argmax if is_last else None, self.ws)
        if is_last:
            return [t.clone() for t in (self.probs, self.argmax) if t is not None]
        return [v.contiguous() for v in self._views(self.need_out)]
