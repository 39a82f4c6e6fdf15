"""GPU parity of the normalisation steps, the U-Net passes and sliding-window inference
against the CPU oracle (bf16 storage points mirrored by the oracle), through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ops, unet as O
from paper_2006_12575_b200 import binding as B
from paper_2006_12575_b200 import synth

from _util import assert_close, dev_bf16, host_f64

pytestmark = pytest.mark.gpu


def make_net(levels, ch, cpl, K, seed, cin=1, bias_scale=0.1):
    """Builds the library plan, the oracle's layer list, and one set of seeded parameters for both."""
    net = B.lamp_unet_create(B.unet_spec(levels, ch, cpl, cin, K))
    spec = O.UNetSpec(levels, list(ch), cpl, cin, K)
    lay = O.unet_layers(spec)
    ws = synth.kaiming_for_layers([(l.taps, l.c_out, l.c_in, l.fan_in) for l in lay], seed)
    bs = [bias_scale * synth.rng(seed * 77 + i).standard_normal(l.c_out).astype(np.float32) for i, l in enumerate(lay)]
    wflat = np.zeros(B.lamp_unet_weight_count(net), dtype=np.float32)
    bflat = np.zeros(B.lamp_unet_bias_count(net), dtype=np.float32)
    offs = []
    for i, l in enumerate(lay):
        wo, bo, _ = B.lamp_unet_param_layout(net, i)
        wflat[wo:wo + ws[i].size] = ws[i].ravel()
        bflat[bo:bo + l.c_out] = bs[i]
        offs.append((wo, bo))
    return net, spec, lay, ws, bs, dev_bf16(wflat), torch.from_numpy(bflat).cuda(), offs


def tie_aware_agreement(seg, ref_scores, tau=None):
    """Fraction of voxels whose class equals the oracle's, counting either of the oracle's two best
    classes as correct where their margin is below tau (default: 1e-3 of the largest score)."""
    order = np.argsort(-ref_scores, axis=-1, kind="stable")
    best, second = order[..., 0], order[..., 1]
    top = np.take_along_axis(ref_scores, order[..., :2], axis=-1)
    if tau is None:
        tau = 1e-3 * np.abs(ref_scores).max()
    near = (top[..., 0] - top[..., 1]) < tau
    ok = (seg == best) | (near & (seg == second))
    return float(ok.mean()), float((seg == best).mean()), int(near.sum())


def end_to_end_figures(got, ref_q, ref_f, what):
    """End-to-end comparison of class scores [..., K] with the storage-mirrored oracle (ref_q), held to the
    arithmetic's own budget: the distance between the mirrored and the unrounded oracle (ref_f) is the bf16
    storage error of the chain, and two correct bf16 evaluations can differ by about that much (their roundings
    flip on fp32-level differences).  Asserted: rel-L2 <= max(1e-3, 2 budget); max-abs <= max(1e-2 max|ref|,
    2 max-abs budget); arg max agreement >= 99.99 % where either of the oracle's two best classes counts once
    their margin is inside twice the max-abs budget.  The strict figure and the one at the 1e-3 margin are
    returned (and printed by the callers) beside the budgets."""
    got, ref_q, ref_f = (np.asarray(a, dtype=np.float64) for a in (got, ref_q, ref_f))
    budget = np.linalg.norm(ref_q - ref_f) / np.linalg.norm(ref_f)
    budget_abs = np.abs(ref_q - ref_f).max()
    rel = np.linalg.norm(got - ref_q) / np.linalg.norm(ref_q)
    mabs = np.abs(got - ref_q).max()
    mref = np.abs(ref_q).max()
    assert rel <= max(1e-3, 2.0 * budget), f"{what}: end-to-end rel L2 {rel:.3e}, budget {budget:.3e}"
    assert mabs <= max(1e-2 * mref, 2.0 * budget_abs), f"{what}: end-to-end max abs {mabs:.3e}, budget {budget_abs:.3e}"
    seg = np.argmax(got, axis=-1)
    a_budget, strict, near_b = tie_aware_agreement(seg, ref_q, tau=max(1e-3 * mref, 2.0 * budget_abs))
    a_1e3, _, near = tie_aware_agreement(seg, ref_q)
    assert a_budget >= 0.9999, f"{what}: end-to-end arg max agreement {a_budget:.6f} (strict {strict:.6f})"
    r = dict(rel_l2=rel, budget_rel_l2=budget, max_abs=mabs, budget_max_abs=budget_abs, argmax_strict=strict,
             argmax_tie_1e3=a_1e3, argmax_tie_budget=a_budget, near_ties_1e3=near, near_ties_budget=near_b)
    print(f"end to end, {what}: " + ", ".join(f"{k}={v:.4g}" for k, v in r.items()))
    return r


@pytest.mark.parametrize("shape,pitch,off", [((2, 5, 6, 7, 16), 16, 0), ((1, 9, 4, 11, 24), 48, 24),
                                             ((1, 16, 16, 16, 64), 128, 64)])
def test_instnorm_relu_fwd_bwd_match_oracle(shape, pitch, off):
    N, D, H, W, Cc = shape
    yfull = synth.rng(1).standard_normal(shape) * 1.7 + 0.3
    y = synth.bf16_round(yfull).astype(np.float64)
    stats = np.stack([yfull.sum(axis=(1, 2, 3)), (yfull ** 2).sum(axis=(1, 2, 3))], axis=-1)
    eps = 1e-5
    mu, var, rstd = ops.instnorm_stats(yfull, eps)
    mu = mu.astype(np.float32).astype(np.float64)
    rstd = rstd.astype(np.float32).astype(np.float64)
    z_ref = ops.bf16_round(ops.instnorm_relu_fwd(y, mu, rstd))
    yd = dev_bf16(y)
    zbuf = torch.full((N, D, H, W, pitch), 5.0, dtype=torch.bfloat16, device="cuda")
    mr = torch.empty((N, Cc, 2), dtype=torch.float32, device="cuda")
    B.lamp_instnorm_relu_fwd(yd, torch.from_numpy(stats).cuda(), eps, mr, B.tensor(zbuf, Cc, off))
    assert_close(host_f64(zbuf[..., off:off + Cc]), z_ref, "instnorm fwd")
    if off:
        assert (zbuf[..., :off] == 5.0).all()
    assert_close(host_f64(mr[..., 0]), mu[:, 0, 0, 0, :], "mu", rel=1e-6, mx=1e-6)
    assert_close(host_f64(mr[..., 1]), rstd[:, 0, 0, 0, :], "rstd", rel=1e-6, mx=1e-6)
    # backward with two gradient sources
    ga = synth.normal_bf16(shape, 2).astype(np.float64)
    gb = synth.normal_bf16(shape, 3).astype(np.float64)
    sums = torch.empty((N, Cc, 2), dtype=torch.float64, device="cuda")
    dy = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    for second in (None, gb):
        g = ga if second is None else ga + gb
        ref = ops.bf16_round(ops.instnorm_relu_bwd(g, y, mu, rstd))
        B.lamp_instnorm_relu_bwd(dev_bf16(ga), None if second is None else dev_bf16(gb), yd, mr, sums, dy)
        assert_close(host_f64(dy), ref, "instnorm bwd")


def ws_read(wsb, layout):
    """Copies a tensor kept in the workspace to the host as float64 [n,d,h,w,c]."""
    t, off = layout
    es = {B.LAMP_BF16: 2, B.LAMP_F32: 4}[t.dtype]
    dt = {B.LAMP_BF16: torch.bfloat16, B.LAMP_F32: torch.float32}[t.dtype]
    V = t.n * t.d * t.h * t.w
    count = (V - 1) * t.c_pitch + t.c
    flat = wsb[off:off + count * es].view(dt)
    return host_f64(torch.as_strided(flat, (V, t.c), (t.c_pitch, 1))).reshape(t.n, t.d, t.h, t.w, t.c)


def ws_read_f64(wsb, layout):
    t, off = layout
    return wsb[off:off + t.n * t.c * 8].view(torch.float64).cpu().numpy().reshape(t.n, t.c // 2, 2)


def check_network_layer_by_layer(levels, ch, cpl, K, dhw, seed, x, lab, tight=2e-5):
    """Runs lamp_unet_train_step once, then checks EVERY step of the forward and backward pass on
    its own: the oracle recomputes each step in fp64 from the tensors the GPU actually stored as
    that step's inputs, and the GPU's stored output must match (bf16-rounded where the path stores
    bf16).  This isolates each kernel's arithmetic from the chaotic growth of rounding differences
    along a deep bf16 chain, which the end-to-end comparison below then bounds separately."""
    net, spec, lay, ws, bs, wd, bd, offs = make_net(levels, ch, cpl, K, seed=seed)
    D, H, W = dhw
    N = x.shape[0]
    V = N * D * H * W
    loss = torch.zeros((1,), dtype=torch.float32, device="cuda")
    gw = torch.full((B.lamp_unet_weight_count(net),), float("nan"), dtype=torch.float32, device="cuda")
    gb = torch.full((B.lamp_unet_bias_count(net),), float("nan"), dtype=torch.float32, device="cuda")
    probs = torch.empty((V, K), dtype=torch.float32, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, N, D, H, W, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    B.lamp_unet_train_step(net, wd, bd, dev_bf16(x), torch.from_numpy(lab).cuda(), loss, gw, gb, probs, wsb)
    assert B.lamp_get_async_status() == 0
    gw_h, gb_h = host_f64(gw), host_f64(gb)
    p_gpu = host_f64(probs).reshape(N, D, H, W, K)
    lay_of = lambda i, which: B.lamp_unet_tensor_layout(net, N, D, H, W, B.MODE_TRAIN, i, which)
    eps = spec.eps
    for i, l in enumerate(lay):
        w64, b64 = ws[i].astype(np.float64), bs[i].astype(np.float64)
        x_in = x.astype(np.float64) if i == 0 else ws_read(wsb, lay_of(i, B.T_IN))
        wo, bo = offs[i]
        dW = gw_h[wo:wo + ws[i].size].reshape(ws[i].shape)
        dB = gb_h[bo:bo + l.c_out]
        what = f"{l.name}"
        if l.kind in ("conv", "down"):
            s = 2 if l.kind == "down" else 1
            y_ref = ops.conv3d_fwd(x_in, w64, b64, 3, s, 1)
            y_gpu = ws_read(wsb, lay_of(i, B.T_Y))
            assert_close(y_gpu, ops.bf16_round(y_ref), what + " y")
            st = ws_read_f64(wsb, lay_of(i, B.T_STATS))
            st_ref = np.stack([y_ref.sum(axis=(1, 2, 3)), (y_ref ** 2).sum(axis=(1, 2, 3))], -1)
            assert_close(st, st_ref, what + " stats", rel=1e-5, mx=1e-4)
            mu, var, rstd = ops.instnorm_stats(y_ref, eps)
            t, off = lay_of(i, B.T_MU_RSTD)
            mr = wsb[off:off + N * l.c_out * 8].view(torch.float32).cpu().numpy().reshape(N, l.c_out, 2).astype(np.float64)
            assert_close(mr[..., 0], mu[:, 0, 0, 0, :], what + " mu", rel=1e-4, mx=1e-4)
            assert_close(mr[..., 1], rstd[:, 0, 0, 0, :], what + " rstd", rel=1e-4, mx=1e-4)
            mu_g, rs_g = mr[..., 0][:, None, None, None, :], mr[..., 1][:, None, None, None, :]
            z_gpu = ws_read(wsb, lay_of(i, B.T_OUT))
            assert_close(z_gpu, ops.bf16_round(ops.instnorm_relu_fwd(y_gpu, mu_g, rs_g)), what + " z", rel=2e-4, mx=4e-3)
            # backward
            g = ws_read(wsb, lay_of(i, B.T_DOUT))
            l2 = lay_of(i, B.T_DOUT2)
            assert (l2 is not None) == (l.name.startswith("enc") and lay[i + 1].kind == "down")
            if l2 is not None:
                g = g + ws_read(wsb, l2)
            dy_gpu = ws_read(wsb, lay_of(i, B.T_DY))
            assert_close(dy_gpu, ops.bf16_round(ops.instnorm_relu_bwd(g, y_gpu, mu_g, rs_g)), what + " dy")
            dw_ref, db_ref = ops.conv3d_wgrad(x_in, dy_gpu, 3, s, 1)
            assert_close(dW, dw_ref, what + " dw", rel=tight, mx=tight)
            # dy sums to (nearly) zero per channel after InstanceNorm: the bias gradient is a
            # cancellation, so its error is measured against sum |dy|
            assert np.abs(dB - db_ref).max() <= 1e-5 * np.abs(dy_gpu).sum(axis=(0, 1, 2, 3)).max(), what + " db"
            if i > 0:
                din = ws_read(wsb, lay_of(i, B.T_DIN))
                assert_close(din, ops.bf16_round(ops.conv3d_dgrad(dy_gpu, w64, x_in.shape[1:4], 3, s, 1)), what + " din")
            else:
                assert lay_of(i, B.T_DIN) is None
        elif l.kind == "up":
            u_gpu = ws_read(wsb, lay_of(i, B.T_OUT))
            assert_close(u_gpu, ops.bf16_round(ops.convT3d_fwd(x_in, w64, b64, 2, 2)), what + " out")
            dy_gpu = ws_read(wsb, lay_of(i, B.T_DY))
            dw_ref, db_ref = ops.convT3d_wgrad(x_in, dy_gpu, 2, 2)
            assert_close(dW, dw_ref, what + " dw", rel=tight, mx=tight)
            assert_close(dB, db_ref, what + " db", rel=1e-4, mx=1e-4)
            din = ws_read(wsb, lay_of(i, B.T_DIN))
            assert_close(din, ops.bf16_round(ops.convT3d_dgrad(dy_gpu, w64, x_in.shape[1:4], 2, 2)), what + " din")
        else:
            p_ref = ops.softmax(ops.conv3d_fwd(x_in, w64, b64, 1, 1, 0))
            assert_close(p_gpu, p_ref, what + " probs", rel=1e-5, mx=1e-5)
            assert abs(float(loss.item()) - ops.dice_loss(p_gpu, lab)) < 1e-5
            dl = ops.dice_loss_grad_logits(p_gpu, lab)
            dw_ref, db_ref = ops.conv3d_wgrad(x_in, dl, 1, 1, 0)
            assert_close(dW, dw_ref, what + " dw", rel=1e-4, mx=1e-4)
            assert_close(dB, db_ref, what + " db", rel=1e-4, mx=1e-4)
            din = ws_read(wsb, lay_of(i, B.T_DIN))
            assert_close(din, ops.bf16_round(ops.conv3d_dgrad(dl, w64, x_in.shape[1:4], 1, 1, 0)), what + " din")
    # End to end against the storage-mirrored oracle.  Two correct bf16 evaluations differ by rounding
    # decisions that flip on fp32-level differences and then spread; their distance is bounded by the
    # bf16 storage error itself, measured here as |mirrored oracle - unrounded oracle|.
    ws64 = [a.astype(np.float64) for a in ws]
    bs64 = [a.astype(np.float64) for a in bs]
    loss_q, dWq, dBq, p_q = O.train_step(spec, ws64, bs64, x.astype(np.float64), lab, quantise=True)
    loss_f, dWf, dBf, p_f = O.train_step(spec, ws64, bs64, x.astype(np.float64), lab, quantise=False)
    fig = end_to_end_figures(p_gpu, p_q, p_f, "train step probabilities")
    assert abs(float(loss.item()) - loss_q) <= max(1e-3, 2.0 * abs(loss_q - loss_f) / abs(loss_f)) * abs(loss_q)
    for i, l in enumerate(lay):
        wo, _ = offs[i]
        got = gw_h[wo:wo + ws[i].size].reshape(ws[i].shape)
        bud = np.linalg.norm(dWq[i] - dWf[i]) / np.linalg.norm(dWf[i])
        err = np.linalg.norm(got - dWq[i]) / np.linalg.norm(dWq[i])
        assert err <= max(1e-3, 2.0 * bud), (l.name, err, bud)
    B.lamp_unet_destroy(net)
    return fig


CFG0 = dict(levels=3, ch=[8, 16, 32], cpl=2, K=4)


def _cfg0_inputs():
    x = synth.bf16_round(synth.blurred_noise((32, 32, 32), 2.0, 0))[None, ..., None]
    lab = synth.labels_quartiles((32, 32, 32), 1000, 4)[None]
    return x, lab


def test_train_step_tiny_unet_every_step_matches_oracle():
    x, lab = _cfg0_inputs()
    r = check_network_layer_by_layer(CFG0["levels"], CFG0["ch"], CFG0["cpl"], CFG0["K"], (32, 32, 32), 1, x, lab)
    print("tiny U-Net:", r)


def test_train_step_wide_unet_every_step_matches_oracle():
    # widths that take the tensor-core path, a ragged non-cubic volume, batch of 2
    D, H, W = 8, 12, 20
    x = synth.bf16_round(np.stack([synth.blurred_noise((D, H, W), 1.5, s) for s in (3, 4)]))[..., None]
    lab = np.stack([synth.labels_blobs((D, H, W), 5 + s, 5, 1.5) for s in (0, 1)])
    r = check_network_layer_by_layer(2, [32, 64], 2, 5, (D, H, W), 2, x, lab)
    print("wide U-Net:", r)


def test_train_step_unet_128_first_level_every_step_matches_oracle():
    # the paper's widest first level (Sec. 3: 128 filters): head forward and backward on 128 channels
    D, H, W = 8, 8, 16
    x = synth.bf16_round(synth.blurred_noise((D, H, W), 1.5, 31))[None, ..., None]
    lab = synth.labels_blobs((D, H, W), 32, 10, 1.5)[None]
    r = check_network_layer_by_layer(2, [128, 256], 1, 10, (D, H, W), 3, x, lab)
    print("U-Net-128:", r)


def test_unet_forward_head_argmax_matches_oracle_on_stored_input():
    net, spec, lay, ws, bs, wd, bd, _ = make_net(CFG0["levels"], CFG0["ch"], CFG0["cpl"], CFG0["K"], seed=1)
    x, _ = _cfg0_inputs()
    V = 32 ** 3
    probs = torch.empty((V, 4), dtype=torch.float32, device="cuda")
    seg = torch.empty((V,), dtype=torch.uint8, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 1, 32, 32, 32, B.MODE_INFER), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(x), probs, seg, wsb)
    assert B.lamp_get_async_status() == 0
    # the head on its own: oracle applied to the input the GPU stored for it
    hi = len(lay) - 1
    z = ws_read(wsb, B.lamp_unet_tensor_layout(net, 1, 32, 32, 32, B.MODE_INFER, hi, B.T_IN))
    p_ref = ops.softmax(ops.conv3d_fwd(z, ws[hi].astype(np.float64), bs[hi].astype(np.float64), 1, 1, 0)).reshape(V, 4)
    assert_close(host_f64(probs), p_ref, "head probs", rel=1e-5, mx=1e-5)
    agree, strict, near = tie_aware_agreement(seg.cpu().numpy(), p_ref)
    assert agree >= 0.9999, (agree, strict, near)
    assert (seg.cpu().numpy() == np.argmax(host_f64(probs), -1)).all()
    # the arg-max map alone (no probabilities written) is the same map
    seg_only = torch.full((V,), 255, dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(x), None, seg_only, wsb)
    assert torch.equal(seg_only, seg)
    # inference and training forward passes give the same probabilities
    loss = torch.zeros((1,), dtype=torch.float32, device="cuda")
    gw = torch.empty((B.lamp_unet_weight_count(net),), dtype=torch.float32, device="cuda")
    gb = torch.empty((B.lamp_unet_bias_count(net),), dtype=torch.float32, device="cuda")
    p2 = torch.empty_like(probs)
    wst = torch.empty(B.lamp_unet_workspace_bytes(net, 1, 32, 32, 32, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    lab = torch.zeros((V,), dtype=torch.uint8, device="cuda")
    B.lamp_unet_train_step(net, wd, bd, dev_bf16(x), lab, loss, gw, gb, p2, wst)
    assert torch.equal(p2, probs)
    # end to end against the mirrored oracle, within the bf16 storage budget
    ws64 = [a.astype(np.float64) for a in ws]
    bs64 = [a.astype(np.float64) for a in bs]
    p_q = O.forward(spec, ws64, bs64, x.astype(np.float64), quantise=True).reshape(V, 4)
    p_f = O.forward(spec, ws64, bs64, x.astype(np.float64), quantise=False).reshape(V, 4)
    end_to_end_figures(host_f64(probs), p_q, p_f, "forward pass, tiny U-Net")
    B.lamp_unet_destroy(net)


def test_unet_forward_batch_and_noncubic():
    net, spec, lay, ws, bs, wd, bd, _ = make_net(2, [8, 16], 1, 3, seed=5)
    x = synth.bf16_round(np.stack([synth.blurred_noise((6, 8, 12), 1.5, s) for s in (7, 8)])[..., None])
    ref = O.forward(spec, ws, bs, x.astype(np.float64), quantise=True)
    V = 2 * 6 * 8 * 12
    probs = torch.empty((V, 3), dtype=torch.float32, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 2, 6, 8, 12, B.MODE_INFER), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(x), probs, None, wsb)
    full = O.forward(spec, ws, bs, x.astype(np.float64), quantise=False)
    end_to_end_figures(host_f64(probs), ref.reshape(V, 3), full.reshape(V, 3), "batched forward")
    B.lamp_unet_destroy(net)


def test_overlap_add_matches_oracle():
    D, H, W, K, P = 20, 12, 16, 5, (8, 8, 8)
    spec = O.UNetSpec(1, [8], 1, 1, K)
    sd, sh, sw = (O.window_starts(n, p, 0.25) for n, p in zip((D, H, W), P))
    n_p = len(sd) * len(sh) * len(sw)
    fields = ops.softmax(synth.rng(11).standard_normal((n_p, 8, 8, 8, K))).astype(np.float32)
    for window in (1, 0):
        A, seg, cnt = O.sliding_window(spec, None, None, np.zeros((1, D, H, W, 1)), P, 0.25, gaussian=bool(window),
                                       patch_probs=lambda i, pa: fields[i][None].astype(np.float64))
        assert cnt == n_p
        planar = torch.empty((K, D, H, W), dtype=torch.float32, device="cuda")
        am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
        B.lamp_overlap_add(torch.from_numpy(fields).cuda(), K, D, H, W, P, 0.25, window, planar, am)
        assert_close(host_f64(planar), A.transpose(3, 0, 1, 2), "overlap-add", rel=1e-5, mx=1e-5)
        agree, strict, near = tie_aware_agreement(am.cpu().numpy().reshape(D, H, W), A)
        assert agree == 1.0
    # W not a multiple of 4 takes the scalar path
    D, H, W = 9, 10, 11
    sd, sh, sw = (O.window_starts(n, p, 0.25) for n, p in zip((D, H, W), P))
    n_p = len(sd) * len(sh) * len(sw)
    fields = ops.softmax(synth.rng(12).standard_normal((n_p, 8, 8, 8, K))).astype(np.float32)
    A, seg, cnt = O.sliding_window(spec, None, None, np.zeros((1, D, H, W, 1)), P, 0.25,
                                   patch_probs=lambda i, pa: fields[i][None].astype(np.float64))
    planar = torch.empty((K, D, H, W), dtype=torch.float32, device="cuda")
    am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
    B.lamp_overlap_add(torch.from_numpy(fields).cuda(), K, D, H, W, P, 0.25, 1, planar, am)
    assert_close(host_f64(planar), A.transpose(3, 0, 1, 2), "overlap-add scalar", rel=1e-5, mx=1e-5)


def test_sliding_window_matches_oracle_and_whole_patch_equals_forward():
    net, spec, lay, ws, bs, wd, bd, _ = make_net(2, [8, 16], 1, 3, seed=9)
    D, H, W, P = 12, 8, 10, (8, 8, 8)
    vol = synth.bf16_round(synth.ct_volume((D, H, W), 21))[None, ..., None]
    A, seg_ref, n_p = O.sliding_window(spec, ws, bs, vol.astype(np.float64), P, 0.25, gaussian=True, quantise=True)
    A_full, _, _ = O.sliding_window(spec, ws, bs, vol.astype(np.float64), P, 0.25, gaussian=True, quantise=False)
    assert n_p == 2 * 1 * 2
    sd, sh, sw = (O.window_starts(n, p, 0.25) for n, p in zip((D, H, W), P))
    origins = [(a, b, c) for a in sd for b in sh for c in sw]
    for sw_batch in (1, 3):
        planar = torch.empty((3, D, H, W), dtype=torch.float32, device="cuda")
        am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
        nbytes = B.lamp_sliding_window_workspace_bytes(net, D, H, W, P, 0.25, sw_batch)
        wsb = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        B.lamp_sliding_window_infer(net, wd, bd, dev_bf16(vol), P, 0.25, sw_batch, 1, planar, am, wsb)
        assert B.lamp_get_async_status() == 0
        # step by step: (1) each patch's probabilities (kept at the start of the workspace) equal a
        # plain forward pass on that patch cut out on the host, bit for bit
        pp = wsb[:n_p * 512 * 3 * 4].view(torch.float32).reshape(n_p, 8, 8, 8, 3)
        for i, (a, b, c) in enumerate(origins):
            cut = np.ascontiguousarray(vol[:, a:a + 8, b:b + 8, c:c + 8, :])
            pr = torch.empty((512, 3), dtype=torch.float32, device="cuda")
            wsf = torch.empty(B.lamp_unet_workspace_bytes(net, 1, 8, 8, 8, B.MODE_INFER), dtype=torch.uint8, device="cuda")
            B.lamp_unet_forward(net, wd, bd, dev_bf16(cut), pr, None, wsf)
            assert torch.equal(pr.reshape(8, 8, 8, 3), pp[i])
        # (2) the blend of exactly those probabilities equals the oracle's blend of them
        pp_h = host_f64(pp)
        A_loc, seg_loc, _ = O.sliding_window(spec, None, None, vol.astype(np.float64), P, 0.25, gaussian=True,
                                             patch_probs=lambda i, pa: pp_h[i][None])
        assert_close(host_f64(planar), A_loc.transpose(3, 0, 1, 2), "sliding window blend", rel=1e-5, mx=1e-5)
        agree, strict, near = tie_aware_agreement(am.cpu().numpy().reshape(D, H, W), A_loc)
        assert agree >= 0.9999
        # (3) end to end against the mirrored oracle, within the bf16 storage budget
        end_to_end_figures(host_f64(planar).transpose(1, 2, 3, 0), A, A_full, "sliding window")
    # patch = whole volume: identical to one forward pass
    probs = torch.empty((D * H * W, 3), dtype=torch.float32, device="cuda")
    wsf = torch.empty(B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_INFER), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(vol), probs, None, wsf)
    planar = torch.empty((3, D, H, W), dtype=torch.float32, device="cuda")
    am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
    wsb = torch.empty(B.lamp_sliding_window_workspace_bytes(net, D, H, W, (D, H, W), 0.25, 1), dtype=torch.uint8, device="cuda")
    B.lamp_sliding_window_infer(net, wd, bd, dev_bf16(vol), (D, H, W), 0.25, 1, 1, planar, am, wsb)
    assert torch.allclose(planar.permute(1, 2, 3, 0).reshape(-1, 3), probs, rtol=1e-6, atol=1e-7)
    B.lamp_unet_destroy(net)


@pytest.mark.parametrize("K", [4, 10, 7])
def test_overlap_add_vector_path_matches_oracle(K):
    # every patch origin and extent along W is a multiple of 4: the 16-byte vector path (K = 7: generic path)
    D, H, W, P, ov = 10, 12, 24, (8, 8, 8), 0.5
    spec = O.UNetSpec(1, [8], 1, 1, K)
    sd, sh, sw = (O.window_starts(n, p, ov) for n, p in zip((D, H, W), P))
    assert all(s % 4 == 0 for s in sw)
    n_p = len(sd) * len(sh) * len(sw)
    fields = ops.softmax(synth.rng(13 + K).standard_normal((n_p, 8, 8, 8, K))).astype(np.float32)
    for window in (1, 0):
        A, seg, cnt = O.sliding_window(spec, None, None, np.zeros((1, D, H, W, 1)), P, ov, gaussian=bool(window),
                                       patch_probs=lambda i, pa: fields[i][None].astype(np.float64))
        planar = torch.empty((K, D, H, W), dtype=torch.float32, device="cuda")
        am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
        B.lamp_overlap_add(torch.from_numpy(fields).cuda(), K, D, H, W, P, ov, window, planar, am)
        assert_close(host_f64(planar), A.transpose(3, 0, 1, 2), "overlap-add vector path", rel=1e-5, mx=1e-5)
        agree, strict, near = tie_aware_agreement(am.cpu().numpy().reshape(D, H, W), A)
        assert agree == 1.0


def test_train_step_replayed_from_a_cuda_graph_matches_the_eager_call():
    """The training step forks onto the handle's side stream and joins again before it returns, so a stream
    capture of the call must close and its replay must give what the eager call gives (loss, weight and bias
    gradients; the InstanceNorm sums are fp64 atomics, so the comparison is to rounding, not bitwise)."""
    net, spec, lay, ws, bs, wd, bd, offs = make_net(3, [32, 64, 128], 2, 4, 21)
    D = H = W = 16
    V = D * H * W
    x = dev_bf16(synth.bf16_round(synth.blurred_noise((D, H, W), 1.5, 22))[None, ..., None])
    lab = torch.from_numpy(synth.labels_quartiles((D, H, W), 23, 4)[None]).cuda().reshape(-1)
    nw, nb = B.lamp_unet_weight_count(net), B.lamp_unet_bias_count(net)
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    res = []
    for mode in ("eager", "graph"):
        loss = torch.zeros(1, dtype=torch.float32, device="cuda")
        gw = torch.full((nw,), 7.0, dtype=torch.float32, device="cuda")
        gb = torch.full((nb,), 7.0, dtype=torch.float32, device="cuda")
        call = lambda: B.lamp_unet_train_step(net, wd, bd, x, lab, loss, gw, gb, None, wsb)
        if mode == "eager":
            call()                      # also the first step of the handle: creates the side stream before any capture
        else:
            s = torch.cuda.Stream()
            s.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=s):
                    call()
                gw.fill_(7.0)
                gb.fill_(7.0)
                g.replay()
                g.replay()
            s.synchronize()
        torch.cuda.synchronize()
        assert B.lamp_get_async_status() == 0
        res.append((float(loss.item()), host_f64(gw), host_f64(gb)))
    (l0, w0, b0), (l1, w1, b1) = res
    assert abs(l0 - l1) <= 1e-6 * abs(l0)
    for i, l in enumerate(lay):
        wo, bo = offs[i]
        n = ws[i].size
        assert_close(w1[wo:wo + n], w0[wo:wo + n], f"layer {i} dW, graph vs eager", rel=1e-5, mx=1e-4)
    assert np.abs(b1 - b0).max() <= 1e-4 * max(np.abs(b0).max(), 1e-6) + 1e-7
    B.lamp_unet_destroy(net)


def test_train_step_with_bucket_events_equals_the_plain_step_and_events_mark_final_ranges():
    """lamp_unet_train_step_buckets (the data-parallel form): same gradients as lamp_unet_train_step; a stream that
    waits for bucket b's event and copies that range of grad_w gets its final values although the copy is enqueued
    before the step has finished; the buckets end on layer boundaries."""
    from paper_2006_12575_b200 import replicas
    net, spec, lay, ws, bs, wd, bd, offs = make_net(3, [32, 64, 128], 2, 4, 41)
    D = H = W = 16
    x = dev_bf16(synth.bf16_round(synth.blurred_noise((D, H, W), 1.5, 42))[None, ..., None])
    lab = torch.from_numpy(synth.labels_quartiles((D, H, W), 43, 4)[None]).cuda().reshape(-1)
    nw, nb = B.lamp_unet_weight_count(net), B.lamp_unet_bias_count(net)
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    loss0 = torch.zeros(1, dtype=torch.float32, device="cuda")
    gw0 = torch.full((nw,), 7.0, dtype=torch.float32, device="cuda")
    gb0 = torch.full((nb,), 7.0, dtype=torch.float32, device="cuda")
    B.lamp_unet_train_step(net, wd, bd, x, lab, loss0, gw0, gb0, None, wsb)
    torch.cuda.synchronize()
    starts = replicas.plan_buckets([o[0] for o in offs], nw, 200000)
    assert len(starts) >= 3 and set(starts) <= {o[0] for o in offs}
    ends = starts[1:] + [nw]
    events = [torch.cuda.Event() for _ in starts]
    loss1 = torch.zeros(1, dtype=torch.float32, device="cuda")
    gw1 = torch.full((nw,), float("nan"), dtype=torch.float32, device="cuda")
    gb1 = torch.full((nb,), 7.0, dtype=torch.float32, device="cuda")
    copies = [torch.full((e - s,), float("nan"), dtype=torch.float32, device="cuda") for s, e in zip(starts, ends)]
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    B.lamp_unet_train_step_buckets(net, wd, bd, x, lab, loss1, gw1, gb1, None, wsb, starts, events)
    for b in range(len(starts) - 1, -1, -1):
        side.wait_event(events[b])
        with torch.cuda.stream(side):
            copies[b].copy_(gw1[starts[b]:ends[b]])
    torch.cuda.synchronize()
    assert B.lamp_get_async_status() == 0
    assert abs(float(loss1.item()) - float(loss0.item())) <= 1e-6 * abs(float(loss0.item()))
    for b, (s, e) in enumerate(zip(starts, ends)):
        assert torch.equal(copies[b], gw1[s:e]), f"bucket {b} was not final when its event fired"
    for i, l in enumerate(lay):
        wo, bo = offs[i]
        n = ws[i].size
        assert_close(host_f64(gw1[wo:wo + n]), host_f64(gw0[wo:wo + n]), f"layer {i} dW, bucket form vs plain", rel=1e-5, mx=1e-4)
    assert np.abs(host_f64(gb1) - host_f64(gb0)).max() <= 1e-4 * max(np.abs(host_f64(gb0)).max(), 1e-6) + 1e-7
    # the single-replica glue: nothing to exchange, the buffers hold the step's own gradients
    gw2 = torch.empty_like(gw1)
    gb2 = torch.empty_like(gb1)
    replicas.train_step_overlapped(B, net, wd, bd, x, lab, loss1, gw2, gb2, None, wsb, starts, events, torch.cuda.Stream())
    torch.cuda.synchronize()
    assert_close(host_f64(gw2), host_f64(gw0), "overlapped step, one replica", rel=1e-5, mx=1e-4)
    # invalid bucket lists are refused on the host
    for bad in ([1, 5], [0, 5, 5], [0, nw]):
        with pytest.raises(B.LampError) as e:
            B.lamp_unet_train_step_buckets(net, wd, bd, x, lab, loss1, gw1, gb1, None, wsb, bad, events[:len(bad)])
        assert e.value.status == 1
    B.lamp_unet_destroy(net)


def test_patch_sharded_sliding_window_one_replica_is_bit_identical_and_two_shares_add_up():
    from paper_2006_12575_b200 import replicas
    net, spec, lay, ws, bs, wd, bd, _ = make_net(2, [8, 16], 1, 3, seed=9)
    D, H, W, P, K = 12, 8, 12, (8, 8, 8), 3
    vol = dev_bf16(synth.bf16_round(synth.ct_volume((D, H, W), 21))[None, ..., None])
    n_p = B.lamp_sliding_window_num_patches(D, H, W, P, 0.25)
    assert n_p == len(O.window_starts(D, 8, 0.25)) * len(O.window_starts(H, 8, 0.25)) * len(O.window_starts(W, 8, 0.25)) == 4
    wsb = torch.empty(B.lamp_sliding_window_workspace_bytes(net, D, H, W, P, 0.25, 3), dtype=torch.uint8, device="cuda")
    planar = torch.empty((K, D, H, W), dtype=torch.float32, device="cuda")
    am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
    B.lamp_sliding_window_infer(net, wd, bd, vol, P, 0.25, 3, 1, planar, am, wsb)
    # one replica: the sharded path is the same arithmetic
    sums = torch.empty_like(planar)
    wsum = torch.empty((D, H, W), dtype=torch.float32, device="cuda")
    am1 = torch.empty_like(am)
    replicas.sliding_window_sharded(B, net, wd, bd, vol, P, 0.25, 3, 1, sums, wsum, am1, wsb, write_probs=True)
    assert torch.equal(sums, planar) and torch.equal(am1, am)
    # two shares computed one after the other and added, as two replicas' all-reduce would
    parts = []
    for r in range(2):
        mine = replicas.shard_patches(n_p, r, 2)
        s_r = torch.full_like(planar, float("nan"))
        w_r = torch.full_like(wsum, float("nan"))
        B.lamp_sliding_window_partial(net, wd, bd, vol, P, 0.25, 3, 1, mine.start, len(mine), s_r, w_r, wsb)
        parts.append((s_r, w_r))
    s2, w2 = parts[0][0] + parts[1][0], parts[0][1] + parts[1][1]
    assert torch.isfinite(s2).all() and (w2 > 0).all()
    am2 = torch.empty_like(am)
    B.lamp_sliding_window_finish(s2, w2, K, D * H * W, True, am2)
    assert_close(host_f64(s2), host_f64(planar), "two shares vs one pass", rel=1e-6, mx=1e-6)
    agree, strict, near = tie_aware_agreement(am2.cpu().numpy(), host_f64(planar).reshape(K, -1).T)
    assert agree == 1.0
    assert B.lamp_get_async_status() == 0
    with pytest.raises(B.LampError):
        B.lamp_sliding_window_partial(net, wd, bd, vol, P, 0.25, 3, 1, 3, 2, s2, w2, wsb)      # range beyond the grid
    B.lamp_unet_destroy(net)


@pytest.mark.parametrize("se_ratio", [0, 4])
def test_forward_pass_cut_into_partitions_equals_the_unsplit_pass(se_ratio):
    """lamp_unet_forward_layers (Sec. 2.1 Eq. 1, Sec. 2.2 Eq. 3): the network cut at ANY layer into two partitions, and by
    the balanced partitioner into three, each partition in its own workspace that starts out as garbage and receives
    only the boundary state of the sequential U-Net (entering activation + the kept encoder outputs whose skip crosses
    the cut): probabilities and arg max are bit-identical to the unsplit forward pass."""
    from paper_2006_12575_b200 import pipeline as PL
    levels, ch, cpl, K = 3, [32, 64, 128], 2, 4
    net = B.lamp_unet_create(B.unet_spec(levels, ch, cpl, 1, K, se_ratio=se_ratio))
    nl = B.lamp_unet_num_layers(net)
    g = torch.Generator().manual_seed(77)
    wflat = torch.zeros(B.lamp_unet_weight_count(net), dtype=torch.float32)
    for i in range(nl):
        wo, bo, d = B.lamp_unet_param_layout(net, i)
        n = d.ksize ** 3 * d.c_in * d.c_out
        wflat[wo:wo + n] = torch.randn(n, generator=g) * (2.0 / ((1 if d.transposed else d.ksize ** 3) * d.c_in)) ** 0.5
    wd = wflat.cuda().to(torch.bfloat16)
    bd = (torch.randn(B.lamp_unet_bias_count(net), generator=g) * 0.2).cuda()
    D, H, W = 16, 16, 32
    V = D * H * W
    x = dev_bf16(synth.bf16_round(synth.blurred_noise((D, H, W), 1.5, 78))[None, ..., None])
    nbytes = B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_INFER)
    ws0 = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    p_ref = torch.empty((V, K), dtype=torch.float32, device="cuda")
    a_ref = torch.empty((V,), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, x, p_ref, a_ref, ws0)
    layers = PL.library_layers(B, net)
    assert [l["kind"] for l in layers] == ["conv", "conv", "down", "conv", "conv", "down", "conv", "conv", "up", "conv", "conv",
                                          "up", "conv", "conv", "head"]
    # the skip of level 0 crosses every cut between its producer (layer 1) and its consumer (layer 12)
    assert (1, "out") in PL.boundary_tensors(layers, 7, cpl) and (4, "out") in PL.boundary_tensors(layers, 7, cpl)
    assert PL.boundary_tensors(layers, 13, cpl) == [(13, "in")] + ([(12, "out")] if se_ratio else [])
    fresh = lambda: torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda")
    costs = [2.0 * (27 if l["kind"] in ("conv", "down") else 1) * l["c_in"] * l["c_out"] for l in layers]
    three = [s for s, e in PL.partition_balanced(costs, 3)][1:]
    for cuts in [[c] for c in range(1, nl)] + [three]:
        probs = torch.full((V, K), float("nan"), dtype=torch.float32, device="cuda")
        am = torch.full((V,), 255, dtype=torch.uint8, device="cuda")
        PL.partitioned_forward(B, net, wd, bd, x, cuts, [fresh() for _ in range(len(cuts) + 1)], probs, am, cpl)
        assert B.lamp_get_async_status() == 0
        assert torch.equal(probs, p_ref), f"cuts {cuts}"
        assert torch.equal(am, a_ref), f"cuts {cuts}"
    with pytest.raises(B.LampError):
        B.lamp_unet_forward_layers(net, wd, bd, x, 3, 3, None, None, ws0)
    B.lamp_unet_destroy(net)


def test_pipelined_inference_of_two_volumes_over_three_library_partitions():
    """pipeline.LibraryPartition: three partitions, each with its own workspace, run two volumes in the order of the
    forward schedule; the state handed from partition to partition is what a rank would send to the next (here passed
    on directly: one GPU, so the partitions' kernels simply follow one another).  Every volume's result equals the
    unsplit forward pass."""
    from paper_2006_12575_b200 import pipeline as PL
    net, spec, lay, ws, bs, wd, bd, _ = make_net(3, [32, 64, 128], 2, 4, seed=81)
    D, H, W, K = 16, 16, 16, 4
    V = D * H * W
    vols = [dev_bf16(synth.bf16_round(synth.blurred_noise((D, H, W), 1.5, 82 + i))[None, ..., None]) for i in range(2)]
    nbytes = B.lamp_unet_workspace_bytes(net, 1, D, H, W, B.MODE_INFER)
    refs = []
    for v in vols:
        p = torch.empty((V, K), dtype=torch.float32, device="cuda")
        a = torch.empty((V,), dtype=torch.uint8, device="cuda")
        B.lamp_unet_forward(net, wd, bd, v, p, a, torch.empty(nbytes, dtype=torch.uint8, device="cuda"))
        refs.append((p, a))
    layers = PL.library_layers(B, net)
    costs = [2.0 * (27 if l["kind"] in ("conv", "down") else 1) * l["c_in"] * l["c_out"] for l in layers]
    parts = PL.partition_balanced(costs, 3)
    probs = torch.empty((V, K), dtype=torch.float32, device="cuda")
    am = torch.empty((V,), dtype=torch.uint8, device="cuda")
    stages = [PL.LibraryPartition(B, net, wd, bd, (1, D, H, W), s, e, torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda"),
                                  vols[0], 2, probs, am) for s, e in parts]
    in_flight, outs = {}, {}
    for tick in PL.forward_schedule(3, 2):
        for (k, m, _) in tick:
            state = [vols[m]] if k == 0 else in_flight.pop((k, m))
            if k > 0:
                assert [tuple(t.shape) for t in state] == [tuple(t.shape) for t in stages[k].incoming(m)]
            res = stages[k].forward(m, state)
            if k == 2:
                outs[m] = res
            else:
                in_flight[(k + 1, m)] = res
    assert B.lamp_get_async_status() == 0
    for m in range(2):
        assert torch.equal(outs[m][0], refs[m][0]) and torch.equal(outs[m][1], refs[m][1])
    B.lamp_unet_destroy(net)
