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


def tie_aware_agreement(seg, ref_scores):
    """Fraction of voxels whose class equals the oracle's, counting either of the oracle's two best
    classes as correct where their margin is below 1e-3 of the largest score."""
    order = np.argsort(-ref_scores, axis=-1, kind="stable")
    best, second = order[..., 0], order[..., 1]
    top = np.take_along_axis(ref_scores, order[..., :2], axis=-1)
    near = (top[..., 0] - top[..., 1]) < 1e-3 * np.abs(ref_scores).max()
    ok = (seg == best) | (near & (seg == second))
    return float(ok.mean()), float((seg == best).mean()), int(near.sum())


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


CFG0 = dict(levels=3, ch=[8, 16, 32], cpl=2, K=4)


def _cfg0_inputs():
    x = synth.bf16_round(synth.blurred_noise((32, 32, 32), 2.0, 0))[None, ..., None]
    lab = synth.labels_quartiles((32, 32, 32), 1000, 4)[None]
    return x, lab


def test_unet_forward_tiny_matches_oracle():
    net, spec, lay, ws, bs, wd, bd, _ = make_net(CFG0["levels"], CFG0["ch"], CFG0["cpl"], CFG0["K"], seed=1)
    x, _ = _cfg0_inputs()
    ref = O.forward(spec, ws, bs, x.astype(np.float64), quantise=True)
    V = 32 ** 3
    probs = torch.empty((V, 4), dtype=torch.float32, device="cuda")
    seg = torch.empty((V,), dtype=torch.uint8, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 1, 32, 32, 32, B.MODE_INFER), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(x), probs, seg, wsb)
    assert B.lamp_get_async_status() == 0
    assert_close(host_f64(probs), ref.reshape(V, 4), "unet forward probs")
    agree, strict, near = tie_aware_agreement(seg.cpu().numpy(), ref.reshape(V, 4))
    assert agree >= 0.9999, (agree, strict, near)
    B.lamp_unet_destroy(net)


def test_unet_train_step_tiny_matches_oracle():
    net, spec, lay, ws, bs, wd, bd, offs = make_net(CFG0["levels"], CFG0["ch"], CFG0["cpl"], CFG0["K"], seed=1,
                                                    bias_scale=0.0)
    x, lab = _cfg0_inputs()
    loss_ref, dW, dB, p_ref = O.train_step(spec, ws, bs, x.astype(np.float64), lab, quantise=True)
    V = 32 ** 3
    loss = torch.zeros((1,), dtype=torch.float32, device="cuda")
    gw = torch.full((B.lamp_unet_weight_count(net),), float("nan"), dtype=torch.float32, device="cuda")
    gb = torch.full((B.lamp_unet_bias_count(net),), float("nan"), dtype=torch.float32, device="cuda")
    probs = torch.empty((V, 4), dtype=torch.float32, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 1, 32, 32, 32, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    B.lamp_unet_train_step(net, wd, bd, dev_bf16(x), torch.from_numpy(lab).cuda(), loss, gw, gb, probs, wsb)
    assert B.lamp_get_async_status() == 0
    assert abs(float(loss.item()) - loss_ref) <= 1e-3 * abs(loss_ref)
    assert_close(host_f64(probs), p_ref.reshape(V, 4), "train probs")
    gw_h, gb_h = host_f64(gw), host_f64(gb)
    gnorm = np.sqrt(sum((d ** 2).sum() for d in dW))
    for i, l in enumerate(lay):
        wo, bo = offs[i]
        got = gw_h[wo:wo + dW[i].size].reshape(dW[i].shape)
        assert_close(got, dW[i], f"grad_w {l.name}", rel=3e-3, mx=2e-2)
        gotb = gb_h[bo:bo + l.c_out]
        if l.kind in ("conv", "down"):
            # InstanceNorm makes the preceding bias inert: both sides must give (numerically) zero
            assert np.abs(gotb).max() <= 2e-2 * np.abs(dW[i]).max() * 27
        else:
            assert_close(gotb, dB[i], f"grad_b {l.name}", rel=3e-3, mx=2e-2)
    assert gnorm > 0
    B.lamp_unet_destroy(net)


def test_unet_forward_batch_and_noncubic():
    net, spec, lay, ws, bs, wd, bd, _ = make_net(2, [8, 16], 1, 3, seed=5)
    x = synth.bf16_round(np.stack([synth.blurred_noise((6, 8, 12), 1.5, s) for s in (7, 8)])[..., None])
    ref = O.forward(spec, ws, bs, x.astype(np.float64), quantise=True)
    V = 2 * 6 * 8 * 12
    probs = torch.empty((V, 3), dtype=torch.float32, device="cuda")
    wsb = torch.empty(B.lamp_unet_workspace_bytes(net, 2, 6, 8, 12, B.MODE_INFER), dtype=torch.uint8, device="cuda")
    B.lamp_unet_forward(net, wd, bd, dev_bf16(x), probs, None, wsb)
    assert_close(host_f64(probs), ref.reshape(V, 3), "batched forward")
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
    assert n_p == 2 * 1 * 2
    for sw_batch in (1, 3):
        planar = torch.empty((3, D, H, W), dtype=torch.float32, device="cuda")
        am = torch.empty((D * H * W,), dtype=torch.uint8, device="cuda")
        nbytes = B.lamp_sliding_window_workspace_bytes(net, D, H, W, P, 0.25, sw_batch)
        wsb = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        B.lamp_sliding_window_infer(net, wd, bd, dev_bf16(vol), P, 0.25, sw_batch, 1, planar, am, wsb)
        assert B.lamp_get_async_status() == 0
        assert_close(host_f64(planar), A.transpose(3, 0, 1, 2), "sliding window probs")
        agree, strict, near = tie_aware_agreement(am.cpu().numpy().reshape(D, H, W), A)
        assert agree >= 0.9999
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
