"""CPU oracle, network level (TEST INFRASTRUCTURE, fp64).

The U-Net of Sec. 2.2 (Eq. 2): an encoder of L blocks e_1..e_L, decoder blocks
d_{L-1}..d_1 with d_i = s_i(e_i, d_{i+1}) where the skip s_i is a channel
concatenation, and a softmax after the decoder.  Widths double per encoder
block and the decoder mirrors the encoder (Sec. 3).  The encoder-block output
is used twice (Eq. 3 duplicates it as e_{i,0}, e_{i,1}): once by the
down-sampling conv and once by the skip, so its gradient is the sum of both.

Operator reading (the paper does not define the blocks):
  encoder level l : convs_per_level x [conv 3x3x3 s1 p1 -> InstanceNorm -> ReLU] = E_l
  down (l < L)    : conv 3x3x3 s2 p1 (C_l -> C_{l+1}) -> InstanceNorm -> ReLU
  decoder level l : U = transposed conv 2x2x2 s2 (C_{l+1} -> C_l) + bias, no norm / activation
                    X = concat(E_l, U) (that channel order)
                    convs_per_level x [conv 3x3x3 s1 p1 -> InstanceNorm -> ReLU]
  head            : conv 1x1x1 (C_1 -> K) + bias -> softmax over K
  loss            : softmax Dice over all K classes (ops.dice_loss)

Layer / parameter order: encoder levels in order (their convs, then the down
conv), decoder levels from deep to shallow (up conv, then the convs), head.

Storage contract mirrored when ``quantise=True`` (the bf16 network path stores
these tensors as bf16, everything else is kept at full precision):
  inputs and weights (given already rounded);
  the raw conv output y of every normalised conv - InstanceNorm statistics are
  taken from the UNROUNDED y, then y is stored rounded, mu and rstd are kept as
  fp32, and z = relu((y_stored - mu) * rstd) is stored rounded;
  the up-conv output; every activation gradient handed between layers.
Logits, probabilities, the loss, weight and bias gradients are never rounded.

SEU-Net variant (spec.se_ratio > 0; Sec. 1 and Sec. 3 name it, the block is this build's reading, ops.se_block_fwd):
the last conv of every level produces z = relu((y_stored - mu) * rstd) WITHOUT storing it, and the level's output is
out = r + e * z with r the stored output of the level's first conv and e the excitation of the channel means of z;
out is stored rounded, and in the backward pass dz = e * dout + ds / V is stored rounded before the InstanceNorm
backward; s, h, e and the squeeze-and-excitation parameters (se[i] = (W1, b1, W2, b2) per such layer) are fp32 values
held in fp64 here.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np

from . import ops


@dataclass
class UNetSpec:
    levels: int
    channels: List[int]
    convs_per_level: int = 2
    in_channels: int = 1
    num_classes: int = 4
    eps: float = 1e-5
    se_ratio: int = 0      # > 0: SEU-Net variant, hidden units = width // se_ratio (at least 1); needs convs_per_level >= 2


@dataclass
class Layer:
    name: str
    kind: str          # 'conv' (3x3x3 s1 p1 + IN + ReLU), 'down' (3x3x3 s2 p1 + IN + ReLU), 'up', 'head'
    level: int         # level of the OUTPUT (0 = full resolution)
    c_in: int
    c_out: int
    taps: int
    fan_in: int
    se_cr: int = 0     # > 0: this conv ends its level's stack with a squeeze-and-excitation residual step (ops.se_block_fwd)


def unet_layers(spec: UNetSpec) -> List[Layer]:
    L, ch = spec.levels, spec.channels
    out = []
    c = spec.in_channels
    for l in range(L):
        for j in range(spec.convs_per_level):
            out.append(Layer(f"enc{l}.conv{j}", "conv", l, c, ch[l], 27, 27 * c))
            c = ch[l]
        if l < L - 1:
            out.append(Layer(f"down{l}", "down", l + 1, ch[l], ch[l + 1], 27, 27 * ch[l]))
            c = ch[l + 1]
    for l in range(L - 2, -1, -1):
        out.append(Layer(f"up{l}", "up", l, ch[l + 1], ch[l], 8, ch[l + 1]))
        c = 2 * ch[l]
        for j in range(spec.convs_per_level):
            out.append(Layer(f"dec{l}.conv{j}", "conv", l, c, ch[l], 27, 27 * c))
            c = ch[l]
    out.append(Layer("head", "head", 0, ch[0], spec.num_classes, 1, ch[0]))
    if spec.se_ratio > 0:
        if spec.convs_per_level < 2:
            raise ValueError("the squeeze-and-excitation residual block needs at least two convs per level")
        for ly in out:
            if ly.kind == "conv" and ly.name.endswith(f".conv{spec.convs_per_level - 1}"):
                ly.se_cr = max(1, ly.c_out // spec.se_ratio)
    return out


def _q(a, quantise):
    return ops.bf16_round(a) if quantise else a


def _norm_conv_fwd(x, w, b, stride, eps, quantise):
    """conv 3x3x3 pad 1 -> InstanceNorm -> ReLU with the storage contract.  Returns (z, cache)."""
    y = ops.conv3d_fwd(x, w, b, 3, stride, 1)
    mu, var, rstd = ops.instnorm_stats(y, eps)
    if quantise:
        mu = mu.astype(np.float32).astype(np.float64)
        rstd = rstd.astype(np.float32).astype(np.float64)
    ys = _q(y, quantise)
    z = _q(ops.instnorm_relu_fwd(ys, mu, rstd), quantise)
    return z, dict(x=x, ys=ys, mu=mu, rstd=rstd, stride=stride)


def forward(spec: UNetSpec, weights, biases, x, quantise=True, want_cache=False, se=None):
    """x [N,D,H,W,Cin] float64 (bf16-valued when quantise).  Returns probs [N,D,H,W,K]
    (and the per-layer cache when want_cache).  se: per layer (W1, b1, W2, b2) or None (SEU-Net variant)."""
    lay = unet_layers(spec)
    cache = [None] * len(lay)
    skips = {}
    a = np.asarray(x, dtype=np.float64)
    for i, ly in enumerate(lay):
        w, b = weights[i], biases[i]
        if ly.kind in ("conv", "down"):
            a, cache[i] = _norm_conv_fwd(a, w, b, 2 if ly.kind == "down" else 1, spec.eps, quantise)
            if ly.kind == "conv" and ly.name.endswith(".conv0"):
                first_out, first_idx = a, i                                     # the residual branch of this level
            if ly.se_cr:
                c = cache[i]
                z = ops.instnorm_relu_fwd(c["ys"], c["mu"], c["rstd"])          # not stored, hence not rounded
                out, c["se"] = ops.se_block_fwd(z, first_out, *se[i])
                c["res_idx"] = first_idx
                a = _q(out, quantise)
            nxt = lay[i + 1]
            if ly.name.startswith("enc") and nxt.kind == "down":
                skips[ly.level] = a                     # E_l, used by the down conv and by the skip
        elif ly.kind == "up":
            u = _q(ops.convT3d_fwd(a, w, b, 2, 2), quantise)
            cache[i] = dict(x=a)
            a = np.concatenate([skips[ly.level], u], axis=-1)
        else:
            logits = ops.conv3d_fwd(a, w, b, 1, 1, 0)
            cache[i] = dict(x=a, logits=logits)
            a = ops.softmax(logits)
    return (a, cache) if want_cache else a


def train_step(spec: UNetSpec, weights, biases, x, labels, quantise=True, se=None):
    """One forward + backward pass.  Returns (loss, dweights, dbiases, probs), and as a fifth item the gradients of the
    squeeze-and-excitation parameters per layer when se is given."""
    lay = unet_layers(spec)
    probs, cache = forward(spec, weights, biases, x, quantise, want_cache=True, se=se)
    dSE = [None] * len(lay)
    res_grad = {}
    loss = ops.dice_loss(probs, labels)
    dW = [None] * len(lay)
    dB = [None] * len(lay)
    skip_grad = {}
    g = ops.dice_loss_grad_logits(probs, labels)        # gradient w.r.t. logits, kept unrounded
    for i in range(len(lay) - 1, -1, -1):
        ly, c = lay[i], cache[i]
        w = weights[i]
        if ly.kind == "head":
            dW[i], dB[i] = ops.conv3d_wgrad(c["x"], g, 1, 1, 0)
            g = _q(ops.conv3d_dgrad(g, w, c["x"].shape[1:4], 1, 1, 0), quantise)
        elif ly.kind in ("conv", "down"):
            if ly.name.startswith("enc") and lay[i + 1].kind == "down":
                g = g + skip_grad.pop(ly.level)         # fan-in at E_l: down-conv path + skip path
                if ly.se_cr:
                    g = _q(g, quantise)                 # the summed gradient is stored: three steps read it
            if ly.se_cr:
                dz, dr, dW1, db1, dW2, db2 = ops.se_block_bwd(g, c["se"])
                dSE[i] = (dW1, db1, dW2, db2)
                res_grad[c["res_idx"]] = dr             # the residual branch: the level's first conv also receives dout
                g = _q(dz, quantise)
            if i in res_grad:
                g = g + res_grad.pop(i)
            dy = _q(ops.instnorm_relu_bwd(g, c["ys"], c["mu"], c["rstd"]), quantise)
            dW[i], dB[i] = ops.conv3d_wgrad(c["x"], dy, 3, c["stride"], 1)
            if i > 0:
                g = _q(ops.conv3d_dgrad(dy, w, c["x"].shape[1:4], 3, c["stride"], 1), quantise)
                if lay[i - 1].kind == "up":             # input was concat(E_l, U): split the gradient
                    C = ly.c_in // 2
                    skip_grad[ly.level] = g[..., :C]
                    g = g[..., C:]
        else:                                           # up conv: no norm, no activation
            dW[i], dB[i] = ops.convT3d_wgrad(c["x"], g, 2, 2)
            g = _q(ops.convT3d_dgrad(g, w, c["x"].shape[1:4], 2, 2), quantise)
    if se is not None:
        return loss, dW, dB, probs, dSE
    return loss, dW, dB, probs


# ----------------------------------------------------------------------------
# sliding-window inference (Sec. 3: small patches versus the whole image)
# ----------------------------------------------------------------------------
def window_starts(length: int, patch: int, overlap: float):
    """Patch origins along one axis: 0, s, 2s, ... while the patch fits, s = round(patch (1 - overlap));
    if the last patch does not end at the border, one more patch is placed flush with it."""
    s = int(round(patch * (1.0 - overlap)))
    st = list(range(0, max(length - patch, 0) + 1, s))
    if st[-1] != max(length - patch, 0):
        st.append(length - patch)
    return st


def gaussian_window(patch, sigma_scale=0.125, floor=1e-3):
    """Separable Gaussian centred on the patch, sigma = sigma_scale * extent per axis,
    normalised to maximum 1 and floored at `floor`."""
    w = np.ones(tuple(patch))
    for ax, P in enumerate(patch):
        t = np.arange(P, dtype=np.float64) - (P - 1) / 2.0
        g = np.exp(-0.5 * (t / (sigma_scale * P)) ** 2)
        sh = [1, 1, 1]
        sh[ax] = P
        w = w * g.reshape(sh)
    return np.maximum(w / w.max(), floor)


def sliding_window(spec, weights, biases, vol, patch, overlap, gaussian=True, quantise=True, patch_probs=None):
    """vol [1,D,H,W,Cin].  Each patch is cut with hard borders and run through the network on
    its own (own InstanceNorm statistics); A[v,k] = sum_p w p_p / sum_p w over the patches that
    cover v, patches visited in ascending (d,h,w) origin order; seg = argmax_k A (lowest index on ties).
    patch_probs, if given, is a function(patch_index, patch_array)->probs replacing the network
    (used by tests that pin the aggregation on its own)."""
    _, D, H, W, _ = vol.shape
    K = spec.num_classes
    sd, sh, sw = (window_starts(n, p, overlap) for n, p in zip((D, H, W), patch))
    win = gaussian_window(patch) if gaussian else np.ones(tuple(patch))
    acc = np.zeros((D, H, W, K))
    wsum = np.zeros((D, H, W))
    idx = 0
    for d0 in sd:
        for h0 in sh:
            for w0 in sw:
                pa = vol[:, d0:d0 + patch[0], h0:h0 + patch[1], w0:w0 + patch[2], :]
                pr = patch_probs(idx, pa) if patch_probs else forward(spec, weights, biases, pa, quantise)
                acc[d0:d0 + patch[0], h0:h0 + patch[1], w0:w0 + patch[2]] += win[..., None] * pr[0]
                wsum[d0:d0 + patch[0], h0:h0 + patch[1], w0:w0 + patch[2]] += win
                idx += 1
    A = acc / wsum[..., None]
    return A, np.argmax(A, axis=-1).astype(np.uint8), idx
