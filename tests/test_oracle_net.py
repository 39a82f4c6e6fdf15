"""Pins for the oracle's normalisation, loss, network and sliding-window parts (CPU only)."""
import numpy as np
import pytest

from oracle import ops, unet
from paper_2006_12575_b200 import synth


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ---------------------------------------------------------------- bf16 rounding
def test_bf16_round_trip_exhaustive_and_ties():
    bits = np.arange(1 << 16, dtype=np.uint32)
    vals = (bits << 16).view(np.float32)
    ok = np.isfinite(vals)
    r = ops.bf16_round(vals[ok].astype(np.float64))
    np.testing.assert_array_equal(r.astype(np.float32).view(np.uint32), vals[ok].view(np.uint32))
    # halfway cases go to the even mantissa: 1 + 2^-8 -> 1 ; 1 + 3*2^-8 -> 1 + 2^-6
    assert ops.bf16_round(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert ops.bf16_round(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    assert ops.bf16_round(np.array([1 + 2.0 ** -8 + 2.0 ** -20]))[0] == 1 + 2.0 ** -7
    assert ops.bf16_round(np.array([-(1 + 2.0 ** -8)]))[0] == -1.0
    # the input generator's rounding (separate code) agrees on random data
    x = _rand((10000,), 0).astype(np.float32)
    np.testing.assert_array_equal(ops.bf16_round(x.astype(np.float64)).astype(np.float32), synth.bf16_round(x))


# ---------------------------------------------------------------- InstanceNorm + ReLU
def test_instnorm_moments_and_invariances():
    eps = 1e-5
    y = 3.0 * _rand((2, 4, 5, 6, 3), 1) + 1.5
    mu, var, rstd = ops.instnorm_stats(y, eps)
    xh = (y - mu) * rstd
    np.testing.assert_allclose(xh.mean(axis=(1, 2, 3)), 0, atol=1e-13)
    np.testing.assert_allclose(xh.var(axis=(1, 2, 3)), (var / (var + eps))[:, 0, 0, 0, :], rtol=1e-12)
    # adding a per-channel constant (a bias) changes nothing
    mu2, var2, rstd2 = ops.instnorm_stats(y + np.arange(3.0), eps)
    np.testing.assert_allclose(ops.instnorm_relu_fwd(y + np.arange(3.0), mu2, rstd2),
                               ops.instnorm_relu_fwd(y, mu, rstd), atol=1e-12)


def test_instnorm_relu_bwd_finite_differences_and_null_directions():
    eps = 1e-5
    y = _rand((1, 3, 4, 5, 2), 2)
    dz = _rand(y.shape, 3)

    def f(yy):
        mu, var, rstd = ops.instnorm_stats(yy, eps)
        return float((ops.instnorm_relu_fwd(yy, mu, rstd) * dz).sum())

    mu, var, rstd = ops.instnorm_stats(y, eps)
    dy = ops.instnorm_relu_bwd(dz, y, mu, rstd)
    rs = np.random.default_rng(4)
    for _ in range(25):
        i = tuple(rs.integers(0, n) for n in y.shape)
        yp, ym = y.copy(), y.copy()
        yp[i] += 1e-6
        ym[i] -= 1e-6
        assert abs((f(yp) - f(ym)) / 2e-6 - dy[i]) < 1e-6
    # a constant shift of y does not change z: the gradient sums to zero per (n, c)
    np.testing.assert_allclose(dy.sum(axis=(1, 2, 3)), 0, atol=1e-12)


# ---------------------------------------------------------------- softmax + Dice
def test_softmax_and_dice_closed_forms():
    K, V = 4, 5 * 6 * 7
    lg = _rand((1, 5, 6, 7, K), 5)
    p = ops.softmax(lg)
    np.testing.assert_allclose(p.sum(-1), 1, atol=1e-14)
    np.testing.assert_allclose(ops.softmax(lg + 100.0), p, atol=1e-13)
    lab = np.random.default_rng(6).integers(0, K, size=(1, 5, 6, 7))
    # exactly one-hot prediction: loss 0
    assert abs(ops.dice_loss(ops.one_hot(lab, K), lab)) < 1e-12
    # uniform prediction: dice_k = (2 G_k / K + eps) / (V / K + G_k + eps)
    eps = 1e-5
    G = np.array([(lab == k).sum() for k in range(K)], dtype=np.float64)
    want = 1 - np.mean((2 * G / K + eps) / (V / K + G + eps))
    assert abs(ops.dice_loss(np.full((1, 5, 6, 7, K), 1.0 / K), lab) - want) < 1e-13
    L = ops.dice_loss(p, lab)
    assert 0 <= L < 1


def test_dice_gradient_finite_differences_and_zero_row_sum():
    K = 3
    lg = _rand((2, 3, 4, 2, K), 7)
    lab = np.random.default_rng(8).integers(0, K, size=(2, 3, 4, 2))
    g = ops.dice_loss_grad_logits(ops.softmax(lg), lab)
    np.testing.assert_allclose(g.sum(-1), 0, atol=1e-15)
    rs = np.random.default_rng(9)
    for _ in range(25):
        i = tuple(rs.integers(0, n) for n in lg.shape)
        lp, lm = lg.copy(), lg.copy()
        lp[i] += 1e-5
        lm[i] -= 1e-5
        fd = (ops.dice_loss(ops.softmax(lp), lab) - ops.dice_loss(ops.softmax(lm), lab)) / 2e-5
        assert abs(fd - g[i]) < 1e-9


# ---------------------------------------------------------------- network
def _tiny(seed=1, levels=2, ch=(2, 4), cpl=2, K=3, cin=1):
    spec = unet.UNetSpec(levels, list(ch), cpl, cin, K)
    lay = unet.unet_layers(spec)
    ws = synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in lay], seed)
    ws = [w.astype(np.float64) for w in ws]
    bs = [0.1 * _rand((l.c_out,), 100 + i) for i, l in enumerate(lay)]
    return spec, lay, ws, bs


def test_layer_plan_matches_paper_structure():
    # Sec. 2.2: five encoder blocks, four skips; Sec. 3: widths double, decoder symmetric.
    spec = unet.UNetSpec(5, [32, 64, 128, 256, 512], 2, 1, 10)
    lay = unet.unet_layers(spec)
    assert sum(l.kind == "up" for l in lay) == 4 and sum(l.kind == "down" for l in lay) == 4
    enc = [l for l in lay if l.name.startswith("enc")]
    assert [l.c_out for l in enc[1::2]] == [32, 64, 128, 256, 512]
    dec0 = [l for l in lay if l.name.startswith("dec")]
    assert [l.c_in for l in dec0[0::2]] == [512, 256, 128, 64]        # concat doubles the input width
    assert [l.c_out for l in dec0[0::2]] == [256, 128, 64, 32]
    n_par = sum(l.taps * l.c_in * l.c_out + l.c_out for l in lay)
    ch, want, c = [32, 64, 128, 256, 512], 0, 1
    for l in range(5):                                  # two 3x3x3 convs per level, then the stride-2 conv
        want += 27 * c * ch[l] + ch[l] + 27 * ch[l] * ch[l] + ch[l]
        if l < 4:
            want += 27 * ch[l] * ch[l + 1] + ch[l + 1]
            c = ch[l + 1]
    for l in range(3, -1, -1):                          # 2x2x2 up conv, conv on 2C channels, conv on C channels
        want += 8 * ch[l + 1] * ch[l] + ch[l] + 27 * 2 * ch[l] * ch[l] + ch[l] + 27 * ch[l] * ch[l] + ch[l]
    want += 32 * 10 + 10
    assert n_par == want == 31_976_906
    spec3 = unet.UNetSpec(5, [64, 128, 256, 512, 1024], 3, 1, 10)
    assert abs(sum(l.taps * l.c_in * l.c_out + l.c_out for l in unet.unet_layers(spec3)) / 1e6 - 175.0) < 0.1


def test_network_gradient_finite_differences_and_norm_null_directions():
    spec, lay, ws, bs = _tiny()
    x = synth.blurred_noise((4, 4, 4), 1.0, 3).astype(np.float64)[None, ..., None]
    lab = np.random.default_rng(4).integers(0, 3, size=(1, 4, 4, 4))
    loss, dW, dB, probs = unet.train_step(spec, ws, bs, x, lab, quantise=False)
    np.testing.assert_allclose(probs.sum(-1), 1, atol=1e-13)
    rs = np.random.default_rng(5)
    for li in range(len(lay)):
        for _ in range(3):
            i = tuple(rs.integers(0, n) for n in ws[li].shape)
            wp = [w.copy() for w in ws]
            wm = [w.copy() for w in ws]
            wp[li][i] += 1e-5
            wm[li][i] -= 1e-5
            lp = ops.dice_loss(unet.forward(spec, wp, bs, x, quantise=False), lab)
            lm = ops.dice_loss(unet.forward(spec, wm, bs, x, quantise=False), lab)
            fd = (lp - lm) / 2e-5
            assert abs(fd - dW[li][i]) < 2e-7 + 1e-4 * abs(fd), (lay[li].name, i, fd, dW[li][i])
    for li, l in enumerate(lay):
        if l.kind in ("conv", "down"):
            # InstanceNorm removes the bias of the conv before it exactly, and its scale up to the
            # eps in (var + eps): <dw, w> is smaller than |dw||w| by a factor of order eps / var
            assert np.abs(dB[li]).max() < 1e-12
            assert abs((dW[li] * ws[li]).sum()) < 1e-3 * np.linalg.norm(dW[li]) * np.linalg.norm(ws[li])
        else:
            j = int(np.argmax(np.abs(dB[li])))
            bp = [b.copy() for b in bs]
            bm = [b.copy() for b in bs]
            bp[li][j] += 1e-5
            bm[li][j] -= 1e-5
            fd = (ops.dice_loss(unet.forward(spec, ws, bp, x, quantise=False), lab)
                  - ops.dice_loss(unet.forward(spec, ws, bm, x, quantise=False), lab)) / 2e-5
            assert abs(fd - dB[li][j]) < 2e-7 + 1e-4 * abs(fd)


def test_quantised_path_stays_close_to_full_precision():
    spec, lay, ws, bs = _tiny(ch=(4, 8))
    x = synth.bf16_round(synth.blurred_noise((8, 8, 8), 1.0, 6)).astype(np.float64)[None, ..., None]
    lab = np.random.default_rng(7).integers(0, 3, size=(1, 8, 8, 8))
    l0, dW0, _, p0 = unet.train_step(spec, ws, bs, x, lab, quantise=False)
    l1, dW1, _, p1 = unet.train_step(spec, ws, bs, x, lab, quantise=True)
    assert abs(l0 - l1) < 5e-3
    assert np.linalg.norm(p0 - p1) / np.linalg.norm(p0) < 5e-2
    for a, b in zip(dW0, dW1):
        assert np.linalg.norm(a - b) <= 0.2 * np.linalg.norm(a) + 1e-12


# ---------------------------------------------------------------- sliding window
def test_window_starts_and_patch_count():
    assert unet.window_starts(512, 64, 0.25) == [0, 48, 96, 144, 192, 240, 288, 336, 384, 432, 448]
    assert unet.window_starts(128, 64, 0.25) == [0, 48, 64]
    assert unet.window_starts(64, 64, 0.25) == [0]
    assert len(unet.window_starts(512, 64, 0.25)) ** 2 * len(unet.window_starts(128, 64, 0.25)) == 363


def test_sliding_window_whole_patch_equals_single_forward():
    spec, lay, ws, bs = _tiny()
    x = synth.bf16_round(synth.blurred_noise((4, 4, 4), 1.0, 8)).astype(np.float64)[None, ..., None]
    A, seg, n = unet.sliding_window(spec, ws, bs, x, (4, 4, 4), 0.25)
    p = unet.forward(spec, ws, bs, x)
    assert n == 1
    np.testing.assert_allclose(A, p[0], rtol=1e-14)
    np.testing.assert_array_equal(seg, np.argmax(p[0], -1))


def test_sliding_window_aggregation_properties():
    spec = unet.UNetSpec(1, [2], 1, 1, 3)
    vol = np.zeros((1, 12, 10, 9, 1))
    const = np.array([0.2, 0.5, 0.3])
    A, seg, n = unet.sliding_window(spec, None, None, vol, (4, 4, 4), 0.25,
                                    patch_probs=lambda i, pa: np.broadcast_to(const, pa.shape[:4] + (3,)))
    assert n == len(unet.window_starts(12, 4, .25)) * len(unet.window_starts(10, 4, .25)) * len(unet.window_starts(9, 4, .25))
    np.testing.assert_allclose(A, np.broadcast_to(const, A.shape), rtol=1e-14)
    assert (seg == 1).all()
    # random per-patch fields: rows still sum to one, and a voxel covered by one patch returns that patch
    rs = np.random.default_rng(10)
    fields = {}

    def pp(i, pa):
        fields[i] = ops.softmax(rs.standard_normal(pa.shape[:4] + (3,)))
        return fields[i]

    A, seg, n = unet.sliding_window(spec, None, None, vol, (4, 4, 4), 0.25, patch_probs=pp)
    np.testing.assert_allclose(A.sum(-1), 1, atol=1e-13)
    np.testing.assert_allclose(A[0, 0, 0], fields[0][0, 0, 0, 0], rtol=1e-13)   # corner: one patch only
    w = unet.gaussian_window((4, 4, 4))
    assert w.max() == 1.0 and w.min() >= 1e-3 and np.allclose(w, w[::-1, ::-1, ::-1])
    # voxel (3,0,0) lies in patches with d-origin 0 and 3 (stride 3): weighted mean of the two
    sd = unet.window_starts(12, 4, .25)
    assert sd[:2] == [0, 3]
    nh, nw = len(unet.window_starts(10, 4, .25)), len(unet.window_starts(9, 4, .25))
    p0, p1 = fields[0][0, 3, 0, 0], fields[nh * nw][0, 0, 0, 0]
    want = (w[3, 0, 0] * p0 + w[0, 0, 0] * p1) / (w[3, 0, 0] + w[0, 0, 0])
    np.testing.assert_allclose(A[3, 0, 0], want, rtol=1e-13)


def test_gaussian_window_closed_form_values():
    """The blending window (paper silent: Sec. 3 gives patch sizes only; reading: separable Gaussian centred on the
    patch, sigma = extent / 8 per axis, scaled to maximum 1, floored at 1e-3) against values worked out by hand.
    P = 8: sigma = 1, offsets t = i - 3.5, so relative to the two centre samples (t = +-0.5) the per-axis weight is
    exp(-(t^2 - 0.25) / 2): 1, e^-1, e^-3, e^-6 at |t| = 0.5, 1.5, 2.5, 3.5."""
    w = unet.gaussian_window((8, 8, 8))
    e = np.exp
    np.testing.assert_allclose(w[3, 3, 3], 1.0, rtol=1e-15)
    np.testing.assert_allclose(w[4, 3, 4], 1.0, rtol=1e-15)
    np.testing.assert_allclose(w[2, 3, 4], e(-1.0), rtol=1e-13)            # 0.36788: sigma = P/4 would give e^-0.25
    np.testing.assert_allclose(w[1, 3, 3], e(-3.0), rtol=1e-13)            # 0.049787
    np.testing.assert_allclose(w[3, 6, 4], e(-3.0), rtol=1e-13)            # symmetric in the offset, any axis
    np.testing.assert_allclose(w[0, 3, 3], e(-6.0), rtol=1e-13)            # 2.4788e-3: still above the floor
    np.testing.assert_allclose(w[2, 5, 4], e(-2.0), rtol=1e-13)            # separable: e^-1 * e^-1
    assert w[0, 2, 3] == 1e-3                                              # e^-7 = 9.12e-4 -> floored
    assert w[0, 0, 0] == 1e-3                                              # e^-18 -> floored
    assert w[7, 7, 7] == 1e-3
    assert (w >= 1e-3).all() and w.max() == 1.0
    # the whole window: exponents are sums of one of (0, 1, 3, 6) per axis, each combination occurring 8 times
    total = sum(8 * max(e(-(a + b + c)), 1e-3) for a in (0, 1, 3, 6) for b in (0, 1, 3, 6) for c in (0, 1, 3, 6))
    np.testing.assert_allclose(w.sum(), total, rtol=1e-13)
    assert (w == 1e-3).sum() == 8 * sum(1 for a in (0, 1, 3, 6) for b in (0, 1, 3, 6) for c in (0, 1, 3, 6) if a + b + c >= 7)
    # per-axis sigma follows the axis extent: (64, 32, 16) has sigma (8, 4, 2)
    v = unet.gaussian_window((64, 32, 16))
    np.testing.assert_allclose(v[31, 15, 7], 1.0, rtol=1e-15)
    np.testing.assert_allclose(v[23, 15, 7], e(-0.5 * (8.5 ** 2 - 0.5 ** 2) / 64.0), rtol=1e-13)    # e^-0.5625
    np.testing.assert_allclose(v[31, 11, 7], e(-0.5 * (4.5 ** 2 - 0.5 ** 2) / 16.0), rtol=1e-13)    # e^-0.625
    np.testing.assert_allclose(v[31, 15, 5], e(-0.5 * (2.5 ** 2 - 0.5 ** 2) / 4.0), rtol=1e-13)     # e^-0.75
    # odd extent: a single centre sample
    u = unet.gaussian_window((5, 5, 5))
    np.testing.assert_allclose(u[2, 2, 2], 1.0, rtol=1e-15)
    np.testing.assert_allclose(u[1, 2, 2], e(-0.5 / 0.625 ** 2), rtol=1e-13)


def test_bf16_storage_chain_amplifies_fp32_level_differences_beyond_1e3():
    """Why network-level parity is checked step by step: perturb every conv output of the oracle by a
    relative 1e-7 (the size of an fp32-vs-fp64 accumulation difference) before its bf16 storage rounding.
    Roundings that flip are 2^-8 relative jumps that spread through 27 taps x all channels per layer, so
    the oracle's OWN output moves by more than the 1e-3 bar, though far less than the bf16 storage error."""
    spec = unet.UNetSpec(3, [8, 16, 32], 2, 1, 4)
    lay = unet.unet_layers(spec)
    ws = [w.astype(np.float64) for w in synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in lay], 1)]
    bs = [np.zeros(l.c_out) for l in lay]
    x = synth.bf16_round(synth.blurred_noise((32, 32, 32), 2.0, 0)).astype(np.float64)[None, ..., None]
    ref = unet.forward(spec, ws, bs, x, quantise=True)
    full = unet.forward(spec, ws, bs, x, quantise=False)
    orig = ops.conv3d_fwd
    rs = np.random.default_rng(0)
    try:
        ops.conv3d_fwd = lambda *a, **k: (lambda y: y * (1 + 1e-7 * rs.standard_normal(y.shape)))(orig(*a, **k))
        pert = unet.forward(spec, ws, bs, x, quantise=True)
    finally:
        ops.conv3d_fwd = orig
    moved = np.linalg.norm(pert - ref) / np.linalg.norm(ref)
    budget = np.linalg.norm(ref - full) / np.linalg.norm(full)
    assert 1e-3 < moved < 2 * budget, (moved, budget)
    # without the storage rounding the same perturbation is harmless
    try:
        ops.conv3d_fwd = lambda *a, **k: (lambda y: y * (1 + 1e-7 * rs.standard_normal(y.shape)))(orig(*a, **k))
        pert_f = unet.forward(spec, ws, bs, x, quantise=False)
    finally:
        ops.conv3d_fwd = orig
    assert np.linalg.norm(pert_f - full) / np.linalg.norm(full) < 1e-5
