"""Seeded synthetic inputs: volumes, label maps, weights, gradients.

This module only *draws* data.  It holds none of the network arithmetic (no
convolution of activations, no normalisation, no loss): the CUDA library and
the CPU oracle each receive the arrays produced here and compute on their own.

All random numbers come from numpy's counter-based Philox generator, so a
(seed, shape) pair always gives the same array.

Stand-ins: the paper evaluates on head-and-neck CT (nine organs + background,
largest image 352x256x288) and on liver CT resampled to 1 mm (largest image
512x512x704), clipped and mapped linearly to a fixed intensity range (Sec. 3).
Neither dataset ships with this repository, so the volumes below take their
shapes, channel count (one), intensity range and small-foreground class
imbalance, and nothing else.
"""
from __future__ import annotations

import math

import numpy as np


# ----------------------------------------------------------------------------
# bf16 helpers (storage format of activations and weights)
# ----------------------------------------------------------------------------
def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32 (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round a float array to the nearest bf16 value, returned as float32."""
    return bf16_to_f32(bf16_bits(np.asarray(x, dtype=np.float32))).reshape(np.shape(x))


def rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed)))


# ----------------------------------------------------------------------------
# smooth random fields
# ----------------------------------------------------------------------------
def _blur_axis(a: np.ndarray, sigma: float, axis: int) -> np.ndarray:
    r = int(math.ceil(4.0 * sigma))
    t = np.arange(-r, r + 1, dtype=np.float64)
    k = np.exp(-0.5 * (t / sigma) ** 2)
    k /= k.sum()
    pad = [(0, 0)] * a.ndim
    pad[axis] = (r, r)
    ap = np.pad(a, pad, mode="edge")
    out = np.zeros_like(a)
    n = a.shape[axis]
    for i, kv in enumerate(k):
        sl = [slice(None)] * a.ndim
        sl[axis] = slice(i, i + n)
        out += kv * ap[tuple(sl)]
    return out


def blurred_noise(shape, sigma: float, seed: int) -> np.ndarray:
    """Gaussian white noise, separable Gaussian blur (radius ceil(4 sigma),
    taps normalised, clamp-to-edge), then an affine map of [min, max] to
    [-1, 1].  Returns float32 of the given D x H x W shape."""
    a = rng(seed).standard_normal(tuple(shape)).astype(np.float32)
    for ax in range(a.ndim):
        a = _blur_axis(a, sigma, ax)
    lo, hi = float(a.min()), float(a.max())
    return ((a - lo) * (2.0 / (hi - lo)) - 1.0).astype(np.float32)


def labels_quartiles(shape, seed: int, classes: int = 4, sigma: float = 2.0) -> np.ndarray:
    """Balanced label map: a blurred field cut at its equally spaced quantiles."""
    f = blurred_noise(shape, sigma, seed)
    qs = np.quantile(f, [i / classes for i in range(1, classes)])
    return np.digitize(f, qs).astype(np.uint8)


def labels_blobs(shape, seed: int, classes: int = 10, sigma: float = 4.0) -> np.ndarray:
    """Imbalanced label map: for k = 1..classes-1 an independent blurred field
    marks as foreground the voxels above its (1 - q_k) quantile, q_k drawn from
    U(0.01, 0.03); a higher class overwrites a lower one; the rest is class 0.
    Mirrors the small-organ imbalance of the paper's datasets (Sec. 1)."""
    g = rng(seed)
    qk = g.uniform(0.01, 0.03, size=classes - 1)
    lab = np.zeros(tuple(shape), dtype=np.uint8)
    for k in range(1, classes):
        f = blurred_noise(shape, sigma, seed * 1000 + k)
        thr = np.quantile(f, 1.0 - qk[k - 1])
        lab[f > thr] = k
    return lab


def ct_volume(shape, seed: int, organs: int = 10) -> np.ndarray:
    """CT-like volume in [-1, 1]: 0.3 x blurred noise plus `organs` random
    ellipsoids of distinct mean intensity (later ones overwrite earlier)."""
    D, H, W = shape
    g = rng(seed)
    vol = 0.3 * blurred_noise(shape, 2.0, seed + 1)
    means = g.permutation(np.linspace(-0.9, 0.9, organs))
    zd = np.arange(D, dtype=np.float32)[:, None, None]
    zh = np.arange(H, dtype=np.float32)[None, :, None]
    zw = np.arange(W, dtype=np.float32)[None, None, :]
    for i in range(organs):
        c = [g.uniform(0.1 * n, 0.9 * n) for n in (D, H, W)]
        # semi-axes scale with the volume so that small test volumes also get organs
        r = [g.uniform(24, 72) * D / 512.0, g.uniform(24, 72) * H / 512.0, g.uniform(8, 24) * W / 128.0]
        r = [max(x, 1.5) for x in r]
        m = ((zd - c[0]) / r[0]) ** 2 + ((zh - c[1]) / r[1]) ** 2 + ((zw - c[2]) / r[2]) ** 2 <= 1.0
        vol = np.where(m, np.float32(means[i]) + 0.05 * vol, vol)
    return np.clip(vol, -1.0, 1.0).astype(np.float32)


# ----------------------------------------------------------------------------
# tensors for single-layer runs
# ----------------------------------------------------------------------------
def normal_bf16(shape, seed: int, scale: float = 1.0) -> np.ndarray:
    """N(0, scale^2) samples already rounded to bf16 values (float32 array)."""
    a = rng(seed).standard_normal(tuple(shape), dtype=np.float32) * np.float32(scale)
    return bf16_round(a)


def kaiming_bf16(taps: int, c_out: int, c_in: int, fan_in: int, seed: int) -> np.ndarray:
    """Kaiming-normal weights w[tap][c_out][c_in], std sqrt(2 / fan_in),
    rounded once to bf16 (float32 array holding bf16 values)."""
    return normal_bf16((taps, c_out, c_in), seed, math.sqrt(2.0 / fan_in))


def kaiming_for_layers(layers, seed: int):
    """`layers`: sequence of (taps, c_out, c_in, fan_in).  Returns one weight
    array per layer, layer i drawn from seed * 1000 + i."""
    return [kaiming_bf16(t, co, ci, fi, seed * 1000 + i) for i, (t, co, ci, fi) in enumerate(layers)]
