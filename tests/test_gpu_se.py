"""GPU parity of the squeeze-and-excitation residual block (SEU-Net variant) against the CPU oracle, through the C
ABI: every step on its own from the tensors the GPU stored, then a whole block (two conv -> InstanceNorm -> ReLU
layers, squeeze-and-excitation, residual) forward and backward."""
import numpy as np
import pytest
import torch

from oracle import ops
from paper_2006_12575_b200 import binding as B
from paper_2006_12575_b200 import synth

from _util import assert_close, dev_bf16, host_f64

pytestmark = pytest.mark.gpu

f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def _params(C, Cr, seed):
    rs = synth.rng(seed)
    return (rs.standard_normal((Cr, C)).astype(np.float32) * 0.5, rs.standard_normal(Cr).astype(np.float32) * 0.2 + 0.3,
            rs.standard_normal((C, Cr)).astype(np.float32) * 0.5, rs.standard_normal(C).astype(np.float32) * 0.2)


@pytest.mark.parametrize("shape,Cr,pitch,off,with_res", [((2, 5, 6, 7, 16), 4, 16, 0, True), ((1, 9, 4, 11, 24), 6, 48, 24, False),
                                                         ((2, 16, 16, 16, 64), 16, 128, 64, True), ((1, 3, 5, 7, 256), 64, 256, 0, True)])
def test_se_block_steps_match_oracle(shape, Cr, pitch, off, with_res):
    N, D, H, W, C = shape
    V = D * H * W
    rs = synth.rng(7)
    yfull = rs.standard_normal(shape) * 1.3 + 0.2
    y = synth.bf16_round(yfull).astype(np.float64)
    mu, var, rstd = ops.instnorm_stats(yfull, 1e-5)
    mu32, rstd32 = mu.astype(np.float32).astype(np.float64), rstd.astype(np.float32).astype(np.float64)
    mr = f32(np.stack([mu32[:, 0, 0, 0, :], rstd32[:, 0, 0, 0, :]], axis=-1))
    z = ops.instnorm_relu_fwd(y, mu32, rstd32)                        # never stored on the GPU: recomputed from y
    r = synth.bf16_round(np.maximum(rs.standard_normal(shape), 0)).astype(np.float64) if with_res else None
    W1, b1, W2, b2 = _params(C, Cr, 11)
    yd = dev_bf16(y)
    # squeeze
    sums = torch.full((N, C), float("nan"), dtype=torch.float64, device="cuda")
    B.lamp_se_squeeze(yd, mr, sums)
    assert_close(host_f64(sums), z.sum(axis=(1, 2, 3)), "squeeze sums", rel=1e-6, mx=1e-6)
    # excitation (from the GPU's own sums)
    e = torch.empty((N, C), dtype=torch.float32, device="cuda")
    hid = torch.empty((N, Cr), dtype=torch.float32, device="cuda")
    mean = torch.empty((N, C), dtype=torch.float32, device="cuda")
    B.lamp_se_excite(sums, V, N, C, Cr, f32(W1), f32(b1), f32(W2), f32(b2), e, hid, mean)
    s_gpu = host_f64(sums) / V
    e_ref, h_ref = ops.se_excite(s_gpu, W1, b1, W2, b2)
    assert_close(host_f64(mean), s_gpu, "mean", rel=1e-6, mx=1e-6)
    assert_close(host_f64(hid), h_ref, "hidden", rel=1e-5, mx=1e-5)
    assert_close(host_f64(e), e_ref, "excitation", rel=1e-5, mx=1e-5)
    # apply, into a channel slice
    obuf = torch.full((N, D, H, W, pitch), 5.0, dtype=torch.bfloat16, device="cuda")
    rd = dev_bf16(r) if with_res else None
    B.lamp_se_apply_fwd(yd, mr, e, rd, B.tensor(obuf, C, off))
    e64 = host_f64(e)
    out_ref = e64[:, None, None, None, :] * z + (r if with_res else 0.0)
    assert_close(host_f64(obuf[..., off:off + C]), ops.bf16_round(out_ref), "se apply fwd")
    if off:
        assert (obuf[..., :off] == 5.0).all()
    # backward: reduction, small layers, apply
    g = synth.normal_bf16(shape, 13).astype(np.float64)
    gd = dev_bf16(g)
    de = torch.full((N, C), float("nan"), dtype=torch.float64, device="cuda")
    B.lamp_se_bwd_reduce(gd, yd, mr, de)
    assert_close(host_f64(de), (g * z).sum(axis=(1, 2, 3)), "de sums", rel=1e-5, mx=1e-5)
    dsv = torch.empty((N, C), dtype=torch.float32, device="cuda")
    dw1, db1 = torch.empty((Cr, C), dtype=torch.float32, device="cuda"), torch.empty((Cr,), dtype=torch.float32, device="cuda")
    dw2, db2 = torch.empty((C, Cr), dtype=torch.float32, device="cuda"), torch.empty((C,), dtype=torch.float32, device="cuda")
    B.lamp_se_excite_bwd(de, V, N, C, Cr, e, hid, mean, f32(W1), f32(W2), dsv, dw1, db1, dw2, db2)
    # the oracle's backward from the GPU's stored e, hidden, mean and de sums
    cache = dict(z=z, s=host_f64(mean), e=e64, h=host_f64(hid), W1=W1.astype(np.float64), W2=W2.astype(np.float64))
    de_gpu = host_f64(de)
    dt = de_gpu * e64 * (1 - e64)
    dh = (dt @ cache["W2"]) * (cache["h"] > 0)
    assert_close(host_f64(dw2), dt.T @ cache["h"], "dW2", rel=1e-5, mx=1e-5)
    assert_close(host_f64(db2), dt.sum(0), "db2", rel=1e-5, mx=1e-5)
    assert_close(host_f64(dw1), dh.T @ cache["s"], "dW1", rel=1e-5, mx=1e-5)
    assert_close(host_f64(db1), dh.sum(0), "db1", rel=1e-5, mx=1e-5)
    assert_close(host_f64(dsv), dh @ cache["W1"] / V, "ds / V", rel=1e-5, mx=1e-5)
    dzb = torch.full((N, D, H, W, pitch), 3.0, dtype=torch.bfloat16, device="cuda")
    B.lamp_se_apply_bwd(gd, e, dsv, B.tensor(dzb, C, off))
    dz_ref = e64[:, None, None, None, :] * g + host_f64(dsv)[:, None, None, None, :]
    assert_close(host_f64(dzb[..., off:off + C]), ops.bf16_round(dz_ref), "se apply bwd")
    # the whole backward agrees with the oracle's block derivative (same inputs, unrounded)
    _, ocache = ops.se_block_fwd(z, r, W1, b1, W2, b2)
    dz_o, dr_o, dW1_o, db1_o, dW2_o, db2_o = ops.se_block_bwd(g, ocache)
    assert_close(host_f64(dzb[..., off:off + C]), ops.bf16_round(dz_o), "dz vs oracle block", rel=2e-3, mx=2e-2)
    assert_close(host_f64(dw1), dW1_o, "dW1 vs oracle block", rel=1e-4, mx=1e-4)
    assert_close(host_f64(dw2), dW2_o, "dW2 vs oracle block", rel=1e-4, mx=1e-4)
    assert B.lamp_get_async_status() == 0


def test_se_residual_block_forward_backward_composed_from_the_library_calls():
    """conv -> IN -> ReLU (= r), conv -> IN -> ReLU (= z, not stored), squeeze-and-excitation, out = r + e z; then the
    backward chain down to the block's input gradient and the first conv's weight gradient.  The oracle mirrors the
    bf16 storage points (raw conv outputs, r, out, dz, dy, dx)."""
    N, D, H, W, Ci, C, Cr = 1, 8, 12, 20, 32, 32, 8
    rs = synth.rng(21)
    x = synth.normal_bf16((N, D, H, W, Ci), 22)
    w_a = synth.kaiming_bf16(27, C, Ci, 27 * Ci, 23)
    w_b = synth.kaiming_bf16(27, C, C, 27 * C, 24)
    W1, b1, W2, b2 = _params(C, Cr, 25)
    gout = synth.normal_bf16((N, D, H, W, C), 26).astype(np.float64)
    V = D * H * W
    q = ops.bf16_round
    xd, wad, wbd = dev_bf16(x), dev_bf16(w_a), dev_bf16(w_b)
    desc_a, desc_b = B.conv_desc(Ci, C), B.conv_desc(C, C)
    bf = lambda: torch.empty((N, D, H, W, C), dtype=torch.bfloat16, device="cuda")
    st = lambda: torch.zeros((N, C, 2), dtype=torch.float64, device="cuda")
    mrt = lambda: torch.empty((N, C, 2), dtype=torch.float32, device="cuda")
    # ---- forward on the GPU
    ya, sa, mra, r = bf(), st(), mrt(), bf()
    B.lamp_conv3d_fwd(desc_a, xd, wad, None, ya, sa)
    B.lamp_instnorm_relu_fwd(ya, sa, 1e-5, mra, r)
    yb, sb, mrb = bf(), st(), mrt()
    B.lamp_conv3d_fwd(desc_b, r, wbd, None, yb, sb)
    zb_unused = bf()
    B.lamp_instnorm_relu_fwd(yb, sb, 1e-5, mrb, zb_unused)            # gives mu, rstd of the second conv
    sums = torch.empty((N, C), dtype=torch.float64, device="cuda")
    e, hid, mean = (torch.empty((N, n_), dtype=torch.float32, device="cuda") for n_ in (C, Cr, C))
    out = bf()
    B.lamp_se_squeeze(yb, mrb, sums)
    B.lamp_se_excite(sums, V, N, C, Cr, f32(W1), f32(b1), f32(W2), f32(b2), e, hid, mean)
    B.lamp_se_apply_fwd(yb, mrb, e, r, out)
    # ---- forward in the oracle with the same storage points
    def norm(xin, w):
        y = ops.conv3d_fwd(xin, w, None, 3, 1, 1)
        mu, var, rstd = ops.instnorm_stats(y, 1e-5)
        mu, rstd = mu.astype(np.float32).astype(np.float64), rstd.astype(np.float32).astype(np.float64)
        return q(y), mu, rstd
    ya_o, mua, rsa = norm(x.astype(np.float64), w_a.astype(np.float64))
    r_o = q(ops.instnorm_relu_fwd(ya_o, mua, rsa))
    yb_o, mub, rsb = norm(r_o, w_b.astype(np.float64))
    z_o = ops.instnorm_relu_fwd(yb_o, mub, rsb)
    out_o, cache = ops.se_block_fwd(z_o, r_o, W1, b1, W2, b2)
    assert_close(host_f64(r), r_o, "block r", rel=2e-3, mx=2e-2)
    assert_close(host_f64(e), cache["e"], "block excitation", rel=1e-3, mx=1e-3)
    assert_close(host_f64(out), q(out_o), "block out", rel=3e-3, mx=3e-2)
    # ---- backward on the GPU
    gd = dev_bf16(gout)
    de = torch.empty((N, C), dtype=torch.float64, device="cuda")
    dsv = torch.empty((N, C), dtype=torch.float32, device="cuda")
    dw1, db1_, dw2, db2_ = (torch.empty(s_, dtype=torch.float32, device="cuda") for s_ in ((Cr, C), (Cr,), (C, Cr), (C,)))
    dz, dyb, dr2, dya, dx = bf(), bf(), bf(), bf(), torch.empty((N, D, H, W, Ci), dtype=torch.bfloat16, device="cuda")
    B.lamp_se_bwd_reduce(gd, yb, mrb, de)
    B.lamp_se_excite_bwd(de, V, N, C, Cr, e, hid, mean, f32(W1), f32(W2), dsv, dw1, db1_, dw2, db2_)
    B.lamp_se_apply_bwd(gd, e, dsv, dz)
    scr = torch.empty((N, C, 2), dtype=torch.float64, device="cuda")
    B.lamp_instnorm_relu_bwd(dz, None, yb, mrb, scr, dyb)
    ws = torch.empty(max(B.lamp_conv3d_workspace_bytes(desc_b, r, B.PASS_DGRAD), B.lamp_conv3d_workspace_bytes(desc_a, xd, B.PASS_WGRAD),
                         B.lamp_conv3d_workspace_bytes(desc_a, xd, B.PASS_DGRAD), 256), dtype=torch.uint8, device="cuda")
    B.lamp_conv3d_dgrad(desc_b, dyb, wbd, dr2, ws)
    B.lamp_instnorm_relu_bwd(dr2, gd, ya, mra, scr, dya)               # the residual branch adds dout itself
    dwa = torch.empty((27, C, Ci), dtype=torch.float32, device="cuda")
    B.lamp_conv3d_wgrad(desc_a, xd, dya, dwa, None, ws)
    B.lamp_conv3d_dgrad(desc_a, dya, wad, dx, ws)
    assert B.lamp_get_async_status() == 0
    # ---- backward in the oracle
    dz_o, dr_o, dW1_o, db1_o, dW2_o, db2_o = ops.se_block_bwd(gout, cache)
    dyb_o = q(ops.instnorm_relu_bwd(q(dz_o), yb_o, mub, rsb))
    dr2_o = q(ops.conv3d_dgrad(dyb_o, w_b.astype(np.float64), (D, H, W), 3, 1, 1))
    dya_o = q(ops.instnorm_relu_bwd(dr2_o + dr_o, ya_o, mua, rsa))
    dwa_o, _ = ops.conv3d_wgrad(x.astype(np.float64), dya_o, 3, 1, 1)
    dx_o = q(ops.conv3d_dgrad(dya_o, w_a.astype(np.float64), (D, H, W), 3, 1, 1))
    assert_close(host_f64(dw2), dW2_o, "block dW2", rel=5e-3, mx=5e-2)
    assert_close(host_f64(dw1), dW1_o, "block dW1", rel=5e-3, mx=5e-2)
    assert_close(host_f64(dya), dya_o, "block dy of the first conv", rel=1e-2, mx=1e-1)
    assert_close(host_f64(dwa), dwa_o, "block dW of the first conv", rel=1e-2, mx=1e-1)
    assert_close(host_f64(dx), dx_o, "block dx", rel=1e-2, mx=1e-1)


@pytest.mark.parametrize("cpl", [2, 3])
def test_seunet_train_step_matches_the_mirrored_oracle_within_the_storage_budget(cpl):
    """The SEU-Net variant through lamp_unet_create(se_ratio) / lamp_unet_train_step / lamp_unet_forward: probabilities,
    loss and every gradient (conv weights, biases, squeeze-and-excitation parameters) against the oracle that mirrors
    the bf16 storage points, held to the arithmetic's own budget (mirrored oracle against unrounded oracle) as the
    plain network is; the steps of the block themselves are checked one by one above."""
    from oracle import unet as O
    levels, ch, K, ratio = 2, [32, 64], 5, 4
    D, H, W = 8, 12, 20
    net = B.lamp_unet_create(B.unet_spec(levels, ch, cpl, 1, K, se_ratio=ratio))
    spec = O.UNetSpec(levels, list(ch), cpl, 1, K, se_ratio=ratio)
    lay = O.unet_layers(spec)
    ws = synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in lay], 61)
    rs = synth.rng(62)
    bs = [0.1 * rs.standard_normal(l.c_out).astype(np.float32) for l in lay]
    se = [None] * len(lay)
    wflat = np.zeros(B.lamp_unet_weight_count(net), dtype=np.float32)
    bflat = np.zeros(B.lamp_unet_bias_count(net), dtype=np.float32)
    offs = []
    for i, l in enumerate(lay):
        wo, bo, _ = B.lamp_unet_param_layout(net, i)
        so, cr = B.lamp_unet_se_layout(net, i)
        assert cr == l.se_cr
        wflat[wo:wo + ws[i].size] = ws[i].ravel()
        bflat[bo:bo + l.c_out] = bs[i]
        if cr:
            c = l.c_out
            W1, b1, W2, b2 = _params(c, cr, 70 + i)
            se[i] = (W1, b1, W2, b2)
            bflat[so:so + 2 * c * cr + c + cr] = np.concatenate([W1.ravel(), b1, W2.ravel(), b2])
        offs.append((wo, bo, so, cr))
    assert sum(1 for l in lay if l.se_cr) == 3
    x = synth.bf16_round(np.stack([synth.blurred_noise((D, H, W), 1.5, s) for s in (63, 64)]))[..., None]
    lab = np.stack([synth.labels_blobs((D, H, W), 65 + s, K, 1.5) for s in (0, 1)])
    V = 2 * D * H * W
    wd, bd = dev_bf16(wflat), f32(bflat)
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    gw = torch.full((wflat.size,), float("nan"), dtype=torch.float32, device="cuda")
    gb = torch.full((bflat.size,), float("nan"), dtype=torch.float32, device="cuda")
    probs = torch.empty((V, K), dtype=torch.float32, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 2, D, H, W, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    B.lamp_unet_train_step(net, wd, bd, dev_bf16(x), torch.from_numpy(lab).cuda().reshape(-1), loss, gw, gb, probs, wsb)
    assert B.lamp_get_async_status() == 0
    ws64 = [a.astype(np.float64) for a in ws]
    bs64 = [a.astype(np.float64) for a in bs]
    se64 = [None if t is None else tuple(a.astype(np.float64) for a in t) for t in se]
    l_q, dWq, dBq, p_q, dSq = O.train_step(spec, ws64, bs64, x.astype(np.float64), lab, quantise=True, se=se64)
    l_f, dWf, dBf, p_f, dSf = O.train_step(spec, ws64, bs64, x.astype(np.float64), lab, quantise=False, se=se64)
    relerr = lambda a, b: np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)
    p_gpu = host_f64(probs).reshape(p_q.shape)
    budget = relerr(p_q, p_f)
    assert relerr(p_gpu, p_q) <= max(1e-3, 2 * budget), (relerr(p_gpu, p_q), budget)
    assert np.abs(p_gpu - p_q).max() <= max(1e-2 * np.abs(p_q).max(), 2 * np.abs(p_q - p_f).max())
    assert abs(float(loss.item()) - l_q) <= max(1e-3, 2 * abs(l_q - l_f) / abs(l_f)) * abs(l_q)
    gw_h, gb_h = host_f64(gw), host_f64(gb)
    assert np.isfinite(gw_h).all() and np.isfinite(gb_h).all()
    for i, l in enumerate(lay):
        wo, bo, so, cr = offs[i]
        got = gw_h[wo:wo + ws[i].size].reshape(ws[i].shape)
        assert relerr(got, dWq[i]) <= max(1e-3, 2 * relerr(dWq[i], dWf[i])), (l.name, relerr(got, dWq[i]), relerr(dWq[i], dWf[i]))
        if cr:
            c = l.c_out
            blk = gb_h[so:so + 2 * c * cr + c + cr]
            got_se = (blk[:cr * c].reshape(cr, c), blk[cr * c:cr * c + cr], blk[cr * c + cr:cr * c + cr + c * cr].reshape(c, cr),
                      blk[cr * c + cr + c * cr:])
            for k in range(4):
                bud = relerr(dSq[i][k], dSf[i][k])
                assert relerr(got_se[k], dSq[i][k]) <= max(2e-3, 2 * bud), (l.name, k, relerr(got_se[k], dSq[i][k]), bud)
    # the forward pass alone gives the same probabilities as the training step
    p2 = torch.empty_like(probs)
    wsf = torch.empty(B.lamp_unet_workspace_bytes(net, 2, D, H, W, B.MODE_INFER), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(x), p2, None, wsf)
    assert torch.equal(p2, probs)
    B.lamp_unet_destroy(net)
    # one conv per level has no residual branch: refused
    with pytest.raises(B.LampError) as e:
        B.lamp_unet_create(B.unet_spec(2, [32, 64], 1, 1, K, se_ratio=4))
    assert e.value.status == 2
