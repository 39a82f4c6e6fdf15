"""CPU oracle, operator level (TEST INFRASTRUCTURE, fp64).

Plain definitions of every operator on the U-Net path: the convolution passes
(direct loops in ``lamp_oracle.c``, called through ctypes), instance
normalisation + ReLU and its derivative, softmax, the softmax-Dice loss and its
derivative, and bf16 storage rounding.  Nothing here is shared with the CUDA
library, and the library never imports this package: only tests, the smoke
check and the benchmark's CPU-baseline leg do.

The paper fixes the topology (Sec. 2.2, Eq. 2: encoder blocks, decoder blocks,
concatenation skips, softmax) and the widths (Sec. 3); it does not define the
operators.  The readings used are stated per function.

Arrays are numpy float64, activations NDHWC, weights w[tap][c_out][c_in].
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lamp_oracle.c")
_SO = os.path.join(_HERE, "_lamp_oracle.so")
_lib_handle = None


def build(force: bool = False) -> str:
    """Compile lamp_oracle.c into a shared object beside it (gcc, OpenMP)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def _lib():
    global _lib_handle
    if _lib_handle is None:
        _lib_handle = ctypes.CDLL(build())
    return _lib_handle


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def n_threads() -> int:
    """Threads the C loops will use (OpenMP default = CPUs this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


# ----------------------------------------------------------------------------
# convolution passes
# ----------------------------------------------------------------------------
def _out(n, k, s, p):
    return (n + 2 * p - k) // s + 1


def conv3d_fwd(x, w, b, k, s, p):
    """Cross-correlation, zero padding p, stride s.  x [N,D,H,W,Ci], w [k^3,Co,Ci], b [Co] or None."""
    x, w = _f64(x), _f64(w)
    N, D, H, W, Ci = x.shape
    T, Co, Ci2 = w.shape
    assert T == k ** 3 and Ci2 == Ci
    b = _f64(b) if b is not None else None
    y = np.empty((N, _out(D, k, s, p), _out(H, k, s, p), _out(W, k, s, p), Co))
    _lib().orc_conv3d_fwd(_p(x), _p(w), _p(b), _p(y), N, D, H, W, Ci, Co, k, s, p)
    return y


def conv3d_dgrad(dy, w, in_dhw, k, s, p):
    """Gradient of conv3d_fwd with respect to x; in_dhw = (D,H,W) of x."""
    dy, w = _f64(dy), _f64(w)
    T, Co, Ci = w.shape
    N = dy.shape[0]
    D, H, W = in_dhw
    assert dy.shape == (N, _out(D, k, s, p), _out(H, k, s, p), _out(W, k, s, p), Co)
    dx = np.empty((N, D, H, W, Ci))
    _lib().orc_conv3d_dgrad(_p(dy), _p(w), _p(dx), N, D, H, W, Ci, Co, k, s, p)
    return dx


def conv3d_wgrad(x, dy, k, s, p):
    """Gradient of conv3d_fwd with respect to w and b.  Returns (dw [k^3,Co,Ci], db [Co])."""
    x, dy = _f64(x), _f64(dy)
    N, D, H, W, Ci = x.shape
    Co = dy.shape[-1]
    assert dy.shape == (N, _out(D, k, s, p), _out(H, k, s, p), _out(W, k, s, p), Co)
    dw = np.empty((k ** 3, Co, Ci))
    db = np.empty((Co,))
    _lib().orc_conv3d_wgrad(_p(x), _p(dy), _p(dw), _p(db), N, D, H, W, Ci, Co, k, s, p)
    return dw, db


def convT3d_fwd(x, w, b, k, s):
    """Transposed convolution, output extent (D-1)*s + k (decoder up-sampling, k = s = 2)."""
    x, w = _f64(x), _f64(w)
    N, D, H, W, Ci = x.shape
    T, Co, Ci2 = w.shape
    assert T == k ** 3 and Ci2 == Ci
    b = _f64(b) if b is not None else None
    y = np.empty((N, (D - 1) * s + k, (H - 1) * s + k, (W - 1) * s + k, Co))
    _lib().orc_convT3d_fwd(_p(x), _p(w), _p(b), _p(y), N, D, H, W, Ci, Co, k, s)
    return y


def convT3d_dgrad(dy, w, in_dhw, k, s):
    dy, w = _f64(dy), _f64(w)
    T, Co, Ci = w.shape
    N = dy.shape[0]
    D, H, W = in_dhw
    assert dy.shape == (N, (D - 1) * s + k, (H - 1) * s + k, (W - 1) * s + k, Co)
    dx = np.empty((N, D, H, W, Ci))
    _lib().orc_convT3d_dgrad(_p(dy), _p(w), _p(dx), N, D, H, W, Ci, Co, k, s)
    return dx


def convT3d_wgrad(x, dy, k, s):
    x, dy = _f64(x), _f64(dy)
    N, D, H, W, Ci = x.shape
    Co = dy.shape[-1]
    dw = np.empty((k ** 3, Co, Ci))
    db = np.empty((Co,))
    _lib().orc_convT3d_wgrad(_p(x), _p(dy), _p(dw), _p(db), N, D, H, W, Ci, Co, k, s)
    return dw, db


def conv3d_fwd_points(x, w, b, pts, k, s, p):
    """conv3d_fwd evaluated at listed output positions pts [P,4] = (n, od, oh, ow).  Returns [P, Co]."""
    x, w = _f64(x), _f64(w)
    N, D, H, W, Ci = x.shape
    Co = w.shape[1]
    b = _f64(b) if b is not None else None
    pts = np.ascontiguousarray(pts, dtype=np.int32)
    out = np.empty((pts.shape[0], Co))
    _lib().orc_conv3d_fwd_points(_p(x), _p(w), _p(b), _p(pts), ctypes.c_int64(pts.shape[0]), _p(out),
                                 N, D, H, W, Ci, Co, k, s, p)
    return out


def conv3d_wgrad_points(x, dy, ent, k, s, p):
    """conv3d_wgrad evaluated at listed entries ent [E,3] = (tap, co, ci).  Returns [E]."""
    x, dy = _f64(x), _f64(dy)
    N, D, H, W, Ci = x.shape
    Co = dy.shape[-1]
    ent = np.ascontiguousarray(ent, dtype=np.int32)
    out = np.empty((ent.shape[0],))
    _lib().orc_conv3d_wgrad_points(_p(x), _p(dy), _p(ent), ctypes.c_int64(ent.shape[0]), _p(out),
                                   N, D, H, W, Ci, Co, k, s, p)
    return out


# ----------------------------------------------------------------------------
# bf16 storage rounding (the oracle's own; used to mirror the documented
# storage points of the bf16 network path)
# ----------------------------------------------------------------------------
def bf16_round(x):
    """Nearest bf16 value (ties to even) of each element, via float32, returned as float64."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = ((u + 0x7FFF + lsb) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


# ----------------------------------------------------------------------------
# instance normalisation + ReLU
# ----------------------------------------------------------------------------
def instnorm_stats(y, eps):
    """Per (n, c) over D*H*W: mean, biased variance (two-pass), rstd = (var + eps)^-1/2."""
    y = _f64(y)
    mu = y.mean(axis=(1, 2, 3), keepdims=True)
    var = ((y - mu) ** 2).mean(axis=(1, 2, 3), keepdims=True)
    return mu, var, 1.0 / np.sqrt(var + eps)


def instnorm_relu_fwd(y, mu, rstd):
    """z = max(0, (y - mu) * rstd); no affine parameters."""
    return np.maximum((_f64(y) - mu) * rstd, 0.0)


def instnorm_relu_bwd(dz, y, mu, rstd):
    """Derivative of z = relu(xhat), xhat = (y - mu) * rstd with mu, rstd functions of y:
    g = dz * [xhat > 0];  dy = rstd * (g - mean(g) - xhat * mean(g * xhat)), means per (n, c)."""
    xhat = (_f64(y) - mu) * rstd
    g = _f64(dz) * (xhat > 0)
    m1 = g.mean(axis=(1, 2, 3), keepdims=True)
    m2 = (g * xhat).mean(axis=(1, 2, 3), keepdims=True)
    return rstd * (g - m1 - xhat * m2)


# ----------------------------------------------------------------------------
# softmax + Dice loss (all classes, background included, unweighted mean)
# ----------------------------------------------------------------------------
def softmax(logits):
    """Softmax over the last axis (max-subtracted), the segmentation output of Sec. 2.2."""
    z = _f64(logits)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def one_hot(labels, K):
    lab = np.asarray(labels).astype(np.int64)
    return (lab[..., None] == np.arange(K)).astype(np.float64)


def dice_loss(p, labels, eps=1e-5):
    """p [N,...,K] probabilities, labels [N,...] ints.  Per sample n:
    I_k = sum p g, P_k = sum p, G_k = sum g, dice_k = (2 I_k + eps)/(P_k + G_k + eps),
    L_n = 1 - mean_k dice_k; the loss is the mean of L_n over n."""
    p = _f64(p)
    N, K = p.shape[0], p.shape[-1]
    g = one_hot(labels, K)
    ax = tuple(range(1, p.ndim - 1))
    I = (p * g).sum(axis=ax)
    P = p.sum(axis=ax)
    G = g.sum(axis=ax)
    dice = (2 * I + eps) / (P + G + eps)
    return float((1.0 - dice.mean(axis=1)).mean())


def dice_loss_grad_logits(p, labels, eps=1e-5):
    """dL/dlogits for L = dice_loss(softmax(logits)).
    dL/dp_vk = -(1/(N K)) [2 g_vk / Den_k - (2 I_k + eps) / Den_k^2], Den_k = P_k + G_k + eps;
    dL/dl_vj = p_vj (dL/dp_vj - sum_k p_vk dL/dp_vk)."""
    p = _f64(p)
    N, K = p.shape[0], p.shape[-1]
    g = one_hot(labels, K)
    ax = tuple(range(1, p.ndim - 1))
    sh = (N,) + (1,) * (p.ndim - 2) + (K,)
    I = (p * g).sum(axis=ax).reshape(sh)
    Den = (p.sum(axis=ax) + g.sum(axis=ax)).reshape(sh) + eps
    dp = -(2 * g / Den - (2 * I + eps) / Den ** 2) / (N * K)
    return p * (dp - (p * dp).sum(axis=-1, keepdims=True))


# ----------------------------------------------------------------------------
# Squeeze-and-excitation residual block (the SEU-Net of Sec. 1 / Sec. 3, Tables 2, 3, 5)
# ----------------------------------------------------------------------------
# The paper names the network ("3D SEU-Net", after AnatomyNet) and never defines the block; the cited paper is not
# at hand.  Reading used here: at the end of a level's conv stack, with
#   r = output of the level's FIRST conv -> InstanceNorm -> ReLU (the residual branch; absent for one conv per level),
#   z = output of the level's LAST  conv -> InstanceNorm -> ReLU,
#   s[n,c] = mean over voxels of z                       (squeeze)
#   h = relu(W1 s + b1),  e = sigmoid(W2 h + b2)         (excitation; W1 [C/ratio, C], W2 [C, C/ratio])
#   out = r + e[n,c] * z                                 (channel rescale + residual; >= 0, so no further ReLU)
def se_excite(s, W1, b1, W2, b2):
    """s [N,C] -> (e [N,C], h [N,Cr])."""
    s = _f64(s)
    h = np.maximum(s @ _f64(W1).T + _f64(b1), 0.0)
    t = h @ _f64(W2).T + _f64(b2)
    return 1.0 / (1.0 + np.exp(-t)), h


def se_block_fwd(z, r, W1, b1, W2, b2):
    """z, r [N,D,H,W,C] (r may be None).  Returns (out, cache)."""
    z = _f64(z)
    s = z.mean(axis=(1, 2, 3))
    e, h = se_excite(s, W1, b1, W2, b2)
    out = e[:, None, None, None, :] * z
    if r is not None:
        out = out + _f64(r)
    return out, dict(z=z, s=s, e=e, h=h, W1=_f64(W1), W2=_f64(W2))


def se_block_bwd(dout, cache):
    """Gradient of se_block_fwd.  Returns (dz, dr, dW1, db1, dW2, db2); dr is dout itself."""
    dout = _f64(dout)
    z, s, e, h, W1, W2 = (cache[k] for k in ("z", "s", "e", "h", "W1", "W2"))
    V = z.shape[1] * z.shape[2] * z.shape[3]
    de = (dout * z).sum(axis=(1, 2, 3))                    # [N,C]
    dt = de * e * (1.0 - e)                                # through the sigmoid
    dW2 = dt.T @ h
    db2 = dt.sum(axis=0)
    dh = (dt @ W2) * (h > 0)
    dW1 = dh.T @ s
    db1 = dh.sum(axis=0)
    ds = dh @ W1                                           # [N,C], gradient w.r.t. the channel means
    dz = e[:, None, None, None, :] * dout + (ds / V)[:, None, None, None, :]
    return dz, dout, dW1, db1, dW2, db2
