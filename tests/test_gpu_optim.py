"""Parameter update on the GPU (lamp_rmsprop_step) against the fp64 oracle, element by element, and a short
training loop on a small network: with fixed data the Dice loss must go down."""
import numpy as np
import pytest
import torch

from oracle import optim as O
from oracle import ops
from paper_2006_12575_b200 import binding as B
from paper_2006_12575_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 3, 4, 1023, 4096, 1 << 20, (1 << 20) + 6])
def test_rmsprop_matches_oracle(n):
    r = synth.rng(50 + n % 97)
    w0 = r.standard_normal(n).astype(np.float32)
    v0 = (r.standard_normal(n) ** 2).astype(np.float32) * 1e-2
    g = (r.standard_normal(n) * 10.0 ** r.integers(-4, 2, n)).astype(np.float32)
    g[::7] = 0.0                                                # zero gradients leave the parameter alone
    w, v, gd = (torch.from_numpy(a.copy()).cuda() for a in (w0, v0, g))
    wb = torch.full((n,), float("nan"), dtype=torch.bfloat16, device="cuda")
    for step in range(2):
        B.lamp_rmsprop_step(gd, w, v, wb, 1e-3, 0.99, 1e-8)
        w_ref, v_ref, wb_ref = O.rmsprop_step(w0 if step == 0 else w_ref, g, v0 if step == 0 else v_ref, 1e-3, 0.99, 1e-8)
    assert B.lamp_get_async_status() == 0
    got_w, got_v = w.cpu().numpy().astype(np.float64), v.cpu().numpy().astype(np.float64)
    # fp32 arithmetic against fp64.  v: a few ulp.  w: its own rounding (rtol) plus, per step, the rounding of the
    # step lr * g / (sqrt(v) + eps) <= lr / sqrt(1 - alpha) = 0.01, i.e. a few ulp of 0.01 ~ 5e-9 each
    np.testing.assert_allclose(got_v, v_ref, rtol=2e-6, atol=1e-30)
    np.testing.assert_allclose(got_w, w_ref, rtol=2e-6, atol=2e-8)
    np.testing.assert_array_equal(got_w[::7], w0[::7].astype(np.float64))
    # the bf16 copy is the nearest bf16 of the fp32 master copy the kernel holds
    np.testing.assert_array_equal(wb.float().cpu().numpy().astype(np.float64), ops.bf16_round(got_w))


def test_rmsprop_without_bf16_copy_and_unaligned_views():
    n = 1000
    r = synth.rng(7)
    buf = torch.from_numpy(r.standard_normal(3 * n + 3).astype(np.float32)).cuda()
    g, w, v = buf[1:n + 1], buf[n + 2:2 * n + 2].clone(), buf[2 * n + 3:3 * n + 3].abs().clone()
    w0, v0 = w.cpu().numpy().astype(np.float64), v.cpu().numpy().astype(np.float64)
    B.lamp_rmsprop_step(g, w, v, None, 1e-2, 0.9, 1e-6)        # g starts 4 bytes off a 16-byte boundary: scalar path
    w_ref, v_ref, _ = O.rmsprop_step(w0, g.cpu().numpy(), v0, 1e-2, 0.9, 1e-6)
    np.testing.assert_allclose(w.cpu().numpy(), w_ref, rtol=2e-6, atol=1e-7)      # steps up to lr / sqrt(1 - alpha) = 0.03
    np.testing.assert_allclose(v.cpu().numpy(), v_ref, rtol=2e-6)
    # an empty update is a no-op, bad hyper-parameters are refused
    B.lamp_rmsprop_step(g[:0], w[:0], v[:0], None)
    with pytest.raises(B.LampError):
        B.lamp_rmsprop_step(g, w, v, None, 1e-3, 1.5, 1e-8)


def test_training_loop_reduces_the_loss():
    # forward + backward + update, repeated on one fixed volume: the softmax-Dice loss falls
    spec = dict(levels=2, channels=(16, 32), convs_per_level=2, num_classes=3, in_channels=1)
    net = B.lamp_unet_create(B.unet_spec(**spec))
    nw, nb = B.lamp_unet_weight_count(net), B.lamp_unet_bias_count(net)
    N, D, H, W = 1, 16, 16, 16
    x = torch.from_numpy(synth.normal_bf16((N, D, H, W, 1), 3).astype(np.float32)).cuda().to(torch.bfloat16)
    lab_np = (synth.rng(4).integers(0, 3, (N, D, H, W))).astype(np.uint8)
    lab_np[:, :, :, : W // 2] = 0                               # some structure to learn
    lab = torch.from_numpy(lab_np).cuda()
    wm = torch.from_numpy((synth.rng(5).standard_normal(nw) * 0.1).astype(np.float32)).cuda()
    bm = torch.zeros(nb, dtype=torch.float32, device="cuda")
    wb = wm.to(torch.bfloat16)
    vw, vb = torch.zeros_like(wm), torch.zeros_like(bm)
    gw, gb = torch.empty_like(wm), torch.empty_like(bm)
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    ws = torch.empty(B.lamp_unet_workspace_bytes(net, N, D, H, W, B.MODE_TRAIN), dtype=torch.uint8, device="cuda")
    losses = []
    for step in range(30):
        B.lamp_unet_train_step(net, wb, bm, x, lab, loss, gw, gb, None, ws)
        losses.append(float(loss.item()))
        B.lamp_rmsprop_step(gw, wm, vw, wb, 1e-3, 0.99, 1e-8)
        B.lamp_rmsprop_step(gb, bm, vb, None, 1e-3, 0.99, 1e-8)
    assert B.lamp_get_async_status() == 0
    B.lamp_unet_destroy(net)
    assert all(np.isfinite(losses))
    assert losses[-1] < losses[0] - 0.02, losses
    assert min(losses[-5:]) < min(losses[:5]), losses
