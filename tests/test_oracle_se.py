"""Pins of the oracle's squeeze-and-excitation residual block (oracle/ops.py): closed forms, the identity that an
excitation of one reproduces the plain residual block, and central finite differences on every input and parameter."""
import numpy as np

from oracle import ops


def _setup(seed, N=2, D=3, H=4, W=5, C=8, Cr=2):
    rs = np.random.default_rng(seed)
    z = np.maximum(rs.standard_normal((N, D, H, W, C)), 0.0)        # post-ReLU activations
    r = np.maximum(rs.standard_normal((N, D, H, W, C)), 0.0)
    W1 = rs.standard_normal((Cr, C)) * 0.7
    b1 = rs.standard_normal(Cr) * 0.3 + 0.5
    W2 = rs.standard_normal((C, Cr)) * 0.7
    b2 = rs.standard_normal(C) * 0.3
    return z, r, W1, b1, W2, b2


def test_excitation_closed_forms():
    # zero weights: h = relu(b1), e = sigmoid(b2) whatever the input
    s = np.array([[1.0, 2.0, 3.0, 4.0]])
    e, h = ops.se_excite(s, np.zeros((2, 4)), np.array([0.5, -1.0]), np.zeros((4, 2)), np.array([0.0, np.log(3.0), -np.log(3.0), 40.0]))
    np.testing.assert_allclose(h, [[0.5, 0.0]], rtol=1e-15)
    np.testing.assert_allclose(e, [[0.5, 0.75, 0.25, 1.0]], rtol=1e-12)
    # one hidden unit that adds up the channel means, one output weight: e = sigmoid(2 * (1 + 2 + 3 + 4) - 19) = sigmoid(1)
    e, h = ops.se_excite(s, np.ones((1, 4)), np.zeros(1), np.full((4, 1), 2.0), np.full(4, -19.0))
    np.testing.assert_allclose(h, [[10.0]], rtol=1e-15)
    np.testing.assert_allclose(e, np.full((1, 4), 1.0 / (1.0 + np.exp(-1.0))), rtol=1e-14)
    # a negative pre-activation is cut by the ReLU: the excitation then depends on b2 only
    e, h = ops.se_excite(s, -np.ones((1, 4)), np.zeros(1), np.full((4, 1), 2.0), np.zeros(4))
    assert h[0, 0] == 0.0 and np.allclose(e, 0.5)


def test_block_with_unit_excitation_is_the_plain_residual_block_and_squeeze_is_the_channel_mean():
    z, r, W1, b1, W2, b2 = _setup(1)
    out, cache = ops.se_block_fwd(z, r, W1, b1, np.zeros_like(W2), np.full_like(b2, 60.0))       # sigmoid(60) = 1 in fp64
    np.testing.assert_allclose(out, z + r, rtol=1e-15)
    np.testing.assert_allclose(cache["s"], z.reshape(2, -1, 8).mean(axis=1), rtol=1e-14)
    # a channel that is constant over the volume squeezes to that constant; e lies in (0, 1), so 0 <= out - r <= z
    z2 = np.broadcast_to(np.arange(1.0, 9.0), z.shape)
    out2, c2 = ops.se_block_fwd(z2, None, W1, b1, W2, b2)
    np.testing.assert_allclose(c2["s"], np.tile(np.arange(1.0, 9.0), (2, 1)), rtol=1e-14)
    assert (c2["e"] > 0).all() and (c2["e"] < 1).all()
    assert (out2 >= 0).all() and (out2 <= z2).all()
    # without a residual branch
    out3, _ = ops.se_block_fwd(z, None, W1, b1, W2, b2)
    out4, _ = ops.se_block_fwd(z, r, W1, b1, W2, b2)
    np.testing.assert_allclose(out4 - out3, r, rtol=1e-12, atol=1e-15)
    # samples are independent: the second sample's output does not depend on the first sample's input
    zb = z.copy()
    zb[0] += 1.0
    outb, _ = ops.se_block_fwd(zb, r, W1, b1, W2, b2)
    np.testing.assert_array_equal(outb[1], out4[1])


def test_block_backward_matches_central_finite_differences():
    z, r, W1, b1, W2, b2 = _setup(2)
    rs = np.random.default_rng(3)
    g = rs.standard_normal(z.shape)
    out, cache = ops.se_block_fwd(z, r, W1, b1, W2, b2)
    dz, dr, dW1, db1, dW2, db2 = ops.se_block_bwd(g, cache)
    loss = lambda *a: float((ops.se_block_fwd(*a)[0] * g).sum())
    args = [z, r, W1, b1, W2, b2]
    grads = [dz, dr, dW1, db1, dW2, db2]
    h = 1e-6
    for ai, (a, ga) in enumerate(zip(args, grads)):
        idxs = [tuple(rs.integers(0, n) for n in a.shape) for _ in range(12)]
        for idx in idxs:
            ap, am = a.copy(), a.copy()
            ap[idx] += h
            am[idx] -= h
            fd = (loss(*(args[:ai] + [ap] + args[ai + 1:])) - loss(*(args[:ai] + [am] + args[ai + 1:]))) / (2 * h)
            assert abs(fd - ga[idx]) <= 1e-6 * max(1.0, abs(fd)), (ai, idx, fd, ga[idx])
    # the gradient w.r.t. z has two parts: the rescaled upstream gradient and, through the squeeze, a constant per (n, c)
    part = dz - cache["e"][:, None, None, None, :] * g
    assert np.allclose(part, part[:, :1, :1, :1, :], rtol=0, atol=1e-14)


def _se_net(seed, cpl=2):
    from oracle import unet
    from paper_2006_12575_b200 import synth
    spec = unet.UNetSpec(2, [4, 8], cpl, 1, 3, se_ratio=2)
    lay = unet.unet_layers(spec)
    ws = [w.astype(np.float64) for w in synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in lay], seed)]
    rs = np.random.default_rng(seed)
    bs = [0.1 * rs.standard_normal(l.c_out) for l in lay]
    se = [None] * len(lay)
    for i, l in enumerate(lay):
        if l.se_cr:
            se[i] = (rs.standard_normal((l.se_cr, l.c_out)) * 0.6, rs.standard_normal(l.se_cr) * 0.2 + 0.4,
                     rs.standard_normal((l.c_out, l.se_cr)) * 0.6, rs.standard_normal(l.c_out) * 0.2)
    x = rs.standard_normal((1, 4, 4, 4, 1))
    lab = rs.integers(0, 3, (1, 4, 4, 4))
    return unet, spec, lay, ws, bs, se, x, lab


def test_seunet_with_three_convs_per_level_takes_the_first_conv_as_residual_branch():
    unet, spec, lay, ws, bs, se, x, lab = _se_net(6, cpl=3)
    assert [l.name for l in lay if l.se_cr] == ["enc0.conv2", "enc1.conv2", "dec0.conv2"]
    loss, dW, dB, probs, dSE = unet.train_step(spec, ws, bs, x, lab, quantise=False, se=se)
    f = lambda: unet.train_step(spec, ws, bs, x, lab, quantise=False, se=se)[0]
    names = [l.name for l in lay]
    rs = np.random.default_rng(2)
    h = 1e-6
    # the first conv of a level feeds the second conv AND the residual branch; the middle conv only the last conv
    for name in ("enc0.conv0", "enc0.conv1", "enc1.conv0", "dec0.conv0", "dec0.conv2"):
        i = names.index(name)
        for _ in range(4):
            idx = tuple(rs.integers(0, n) for n in ws[i].shape)
            old = ws[i][idx]
            ws[i][idx] = old + h
            lp = f()
            ws[i][idx] = old - h
            lm = f()
            ws[i][idx] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - dW[i][idx]) <= 2e-6 * max(1.0, abs(fd) * 1e3), (name, fd, dW[i][idx])


def test_seunet_layers_and_gradients_by_finite_differences():
    """The SEU-Net variant of the oracle's network: which layers end in the block, the excitation-one identity, and the
    whole network's gradient (conv weights in front of, inside and behind the blocks, and the blocks' own parameters)."""
    unet, spec, lay, ws, bs, se, x, lab = _se_net(4)
    assert [l.name for l in lay if l.se_cr] == ["enc0.conv1", "enc1.conv1", "dec0.conv1"]
    assert [l.se_cr for l in lay if l.se_cr] == [2, 4, 2]
    loss, dW, dB, probs, dSE = unet.train_step(spec, ws, bs, x, lab, quantise=False, se=se)
    assert probs.shape == (1, 4, 4, 4, 3) and np.allclose(probs.sum(-1), 1)
    f = lambda: unet.train_step(spec, ws, bs, x, lab, quantise=False, se=se)[0]
    rs = np.random.default_rng(9)
    h = 1e-6
    for i, l in enumerate(lay):
        for _ in range(3):
            idx = tuple(rs.integers(0, n) for n in ws[i].shape)
            old = ws[i][idx]
            ws[i][idx] = old + h
            lp = f()
            ws[i][idx] = old - h
            lm = f()
            ws[i][idx] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - dW[i][idx]) <= 2e-6 * max(1.0, abs(fd) * 1e3), (l.name, fd, dW[i][idx])
        if l.se_cr:
            for k in range(4):
                a = se[i][k]
                idx = tuple(rs.integers(0, n) for n in a.shape)
                old = a[idx]
                a[idx] = old + h
                lp = f()
                a[idx] = old - h
                lm = f()
                a[idx] = old
                fd = (lp - lm) / (2 * h)
                assert abs(fd - dSE[i][k][idx]) <= 2e-6 * max(1.0, abs(fd) * 1e3), (l.name, k, fd, dSE[i][k][idx])
    # the plain network is the variant without the blocks: different function, same layer list and shapes
    plain = unet.UNetSpec(2, [4, 8], 2, 1, 3)
    assert [l.name for l in unet.unet_layers(plain)] == [l.name for l in lay]
    p_plain = unet.forward(plain, ws, bs, x, quantise=False)
    assert np.abs(p_plain - probs).max() > 1e-3
