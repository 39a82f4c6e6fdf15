"""GPU parity of the single-layer convolution passes against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ops
from paper_2006_12575_b200 import binding as B
from paper_2006_12575_b200 import synth

from _util import assert_close, dev_bf16, host_f64

pytestmark = pytest.mark.gpu

# (name, N, D, H, W, Ci, Co, k, s, p, transposed)
CASES = [
    ("first_layer_c1", 1, 9, 7, 10, 1, 8, 3, 1, 1, 0),
    ("first_layer_c1_32", 2, 9, 17, 12, 1, 32, 3, 1, 1, 0),
    ("first_layer_c1_64", 1, 6, 5, 21, 1, 64, 3, 1, 1, 0),
    ("first_layer_c1_32_wide", 2, 4, 32, 16, 1, 32, 3, 1, 1, 0),
    ("first_layer_c1_64_wide", 1, 3, 16, 24, 1, 64, 3, 1, 1, 0),
    ("first_layer_c1_32_ragged_lines", 1, 20, 36, 40, 1, 32, 3, 1, 1, 0),
    ("first_layer_c1_96_batch", 3, 5, 9, 16, 1, 96, 3, 1, 1, 0),
    ("first_layer_c1_64_cube", 1, 32, 32, 32, 1, 64, 3, 1, 1, 0),
    ("narrow_16_24", 2, 6, 5, 9, 16, 24, 3, 1, 1, 0),
    ("down_8_16", 1, 8, 6, 10, 8, 16, 3, 2, 1, 0),
    ("down_32_64", 1, 16, 8, 12, 32, 64, 3, 2, 1, 0),
    ("down_64_128_odd", 1, 9, 10, 14, 64, 128, 3, 2, 1, 0),
    ("down_256_512", 2, 4, 4, 8, 256, 512, 3, 2, 1, 0),
    ("down_32_32_big", 1, 20, 34, 18, 32, 32, 3, 2, 1, 0),
    ("up_128_64", 1, 4, 5, 6, 128, 64, 2, 2, 0, 1),
    ("up_512_256", 1, 2, 2, 4, 512, 256, 2, 2, 0, 1),
    ("up_32_32_big", 2, 9, 10, 7, 32, 32, 2, 2, 0, 1),
    ("up_16_8", 2, 3, 4, 5, 16, 8, 2, 2, 0, 1),
    ("up_64_32", 1, 6, 4, 8, 64, 32, 2, 2, 0, 1),
    ("head_8_4", 1, 5, 4, 6, 8, 4, 1, 1, 0, 0),
    ("c32_ragged", 1, 9, 17, 33, 32, 32, 3, 1, 1, 0),
    ("c64_ragged", 1, 33, 17, 9, 64, 64, 3, 1, 1, 0),
    ("c64_cube16", 2, 16, 16, 16, 64, 64, 3, 1, 1, 0),
    ("c64_to_32", 1, 8, 12, 20, 64, 32, 3, 1, 1, 0),
    ("c128_64", 1, 8, 8, 24, 128, 64, 3, 1, 1, 0),
    ("c32_to_128", 1, 4, 8, 16, 32, 128, 3, 1, 1, 0),
    ("c256", 1, 4, 6, 8, 256, 256, 3, 1, 1, 0),
    ("t_c64_h40", 1, 5, 40, 24, 64, 64, 3, 1, 1, 0),
    ("t_c32_h33", 2, 6, 33, 15, 32, 32, 3, 1, 1, 0),
    ("t_c128_h64", 1, 3, 64, 16, 128, 128, 3, 1, 1, 0),
    ("t_c64_to_32", 1, 7, 32, 8, 64, 32, 3, 1, 1, 0),
    ("t_c128_to_64", 1, 3, 36, 10, 128, 64, 3, 1, 1, 0),
    ("t_c32_to_128", 1, 4, 34, 9, 32, 128, 3, 1, 1, 0),
    ("t_single_plane", 1, 1, 32, 8, 64, 64, 3, 1, 1, 0),
    ("t_c256_h32", 1, 3, 32, 8, 256, 256, 3, 1, 1, 0),
    ("t_c512_to_256", 1, 2, 32, 8, 512, 256, 3, 1, 1, 0),
    ("t_c128_to_384", 1, 2, 30, 16, 128, 384, 3, 1, 1, 0),
    ("t_down_32_64", 1, 12, 64, 16, 32, 64, 3, 2, 1, 0),
    ("t_down_64_128_ragged_odd", 1, 7, 60, 31, 64, 128, 3, 2, 1, 0),
    ("t_down_32_32_batch", 2, 8, 64, 16, 32, 32, 3, 2, 1, 0),
    ("t_down_128_256", 1, 4, 64, 16, 128, 256, 3, 2, 1, 0),
    # narrow layers on volumes large enough for the rotating-slot kernel (runs of >= 10 planes per CTA, cut inside
    # window columns; ragged windows; two samples; two channel chunks; columns shorter than a run)
    ("r_c64_runs", 1, 38, 64, 160, 64, 64, 3, 1, 1, 0),
    ("r_c64_ragged_batch", 2, 33, 70, 60, 64, 64, 3, 1, 1, 0),
    ("r_c128_to_64", 1, 25, 96, 160, 128, 64, 3, 1, 1, 0),
    ("r_c64_thin_columns", 1, 3, 352, 288, 64, 64, 3, 1, 1, 0),
    ("r_c32_runs", 1, 60, 128, 104, 32, 32, 3, 1, 1, 0),
    ("r_c64_to_32_ragged", 1, 44, 90, 140, 64, 32, 3, 1, 1, 0),
    ("r_c32_batch_odd_rows", 2, 29, 75, 100, 32, 32, 3, 1, 1, 0),
    ("r_c32_to_64", 1, 30, 128, 104, 32, 64, 3, 1, 1, 0),
    ("r_c64_single_plane", 1, 1, 352, 288, 64, 64, 3, 1, 1, 0),
    ("r_c32_two_planes", 1, 2, 384, 288, 32, 32, 3, 1, 1, 0),
    ("deep_512_cube8", 1, 8, 8, 8, 512, 512, 3, 1, 1, 0),
    ("deep_512_to_256_ragged", 2, 3, 5, 7, 512, 256, 3, 1, 1, 0),
    ("deep_down_256_512", 1, 8, 8, 8, 256, 512, 3, 2, 1, 0),
    ("deep_up_512_256", 1, 4, 4, 4, 512, 256, 2, 2, 0, 1),
    ("tiny_volume", 1, 2, 2, 2, 64, 64, 3, 1, 1, 0),
    ("single_voxel", 1, 1, 1, 1, 32, 32, 3, 1, 1, 0),
]


def _oracle_shapes(N, D, H, W, k, s, p, tr):
    if tr:
        return (N, D * 2, H * 2, W * 2)
    o = lambda n: (n + 2 * p - k) // s + 1
    return (N, o(D), o(H), o(W))


def _inputs(case, seed):
    name, N, D, H, W, Ci, Co, k, s, p, tr = case
    x = synth.normal_bf16((N, D, H, W, Ci), seed)
    w = synth.kaiming_bf16(k ** 3, Co, Ci, (1 if tr else k ** 3) * Ci, seed + 1)
    b = synth.rng(seed + 2).standard_normal(Co).astype(np.float32)
    oshape = _oracle_shapes(N, D, H, W, k, s, p, tr) + (Co,)
    dy = synth.normal_bf16(oshape, seed + 3)
    return x, w, b, dy, oshape


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_conv_fwd_matches_oracle(case):
    name, N, D, H, W, Ci, Co, k, s, p, tr = case
    x, w, b, dy, oshape = _inputs(case, 100)
    ref = ops.convT3d_fwd(x, w, b, k, s) if tr else ops.conv3d_fwd(x, w, b, k, s, p)
    desc = B.conv_desc(Ci, Co, k, s, p, tr)
    xd, wd, bd = dev_bf16(x), dev_bf16(w), torch.from_numpy(b).cuda()
    # fp32 output + statistics
    y32 = torch.full(oshape, float("nan"), dtype=torch.float32, device="cuda")
    stats = torch.zeros((N, Co, 2), dtype=torch.float64, device="cuda")
    B.lamp_conv3d_fwd(desc, xd, wd, bd, y32, stats)
    assert B.lamp_get_async_status() == 0
    assert_close(host_f64(y32), ref, f"{name} fwd f32", rel=2e-5, mx=2e-5)
    s_ref = np.stack([ref.sum(axis=(1, 2, 3)), (ref ** 2).sum(axis=(1, 2, 3))], axis=-1)
    # the sum of zero-mean values cancels, so its error relative to its own size exceeds that of a single y (fp32
    # accumulation over up to 27 * 512 products)
    assert_close(host_f64(stats), s_ref, f"{name} stats", rel=5e-5, mx=1e-4)
    # bf16 output into a channel slice of a wider buffer, no bias
    pitch, off = Co + 16, 8
    ybuf = torch.full(oshape[:4] + (pitch,), 7.0, dtype=torch.bfloat16, device="cuda")
    B.lamp_conv3d_fwd(desc, xd, wd, None, B.tensor(ybuf, Co, off))
    refnb = ref - b
    assert_close(host_f64(ybuf[..., off:off + Co]), ops.bf16_round(refnb), f"{name} fwd bf16 slice")
    assert (ybuf[..., :off] == 7.0).all() and (ybuf[..., off + Co:] == 7.0).all()
    # twice the same call -> bit-identical output
    y2 = torch.empty_like(y32)
    B.lamp_conv3d_fwd(desc, xd, wd, bd, y2)
    assert torch.equal(y2, y32)
    # with the full workspace a small volume splits its reduction over several CTAs: same checks again
    nbytes = B.lamp_conv3d_workspace_bytes(desc, xd, B.PASS_FWD)
    assert B.lamp_conv3d_workspace_min_bytes(desc, xd, B.PASS_FWD) == 0
    if nbytes:
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        y3 = torch.full(oshape, float("nan"), dtype=torch.float32, device="cuda")
        stats.zero_()
        B.lamp_conv3d_fwd(desc, xd, wd, bd, y3, stats, ws)
        assert B.lamp_get_async_status() == 0
        assert_close(host_f64(y3), ref, f"{name} fwd f32 split", rel=2e-5, mx=2e-5)
        assert_close(host_f64(stats), s_ref, f"{name} stats split", rel=5e-5, mx=1e-4)
        ybuf.fill_(7.0)
        B.lamp_conv3d_fwd(desc, xd, wd, None, B.tensor(ybuf, Co, off), None, ws)
        assert_close(host_f64(ybuf[..., off:off + Co]), ops.bf16_round(refnb), f"{name} fwd bf16 slice split")
        assert (ybuf[..., :off] == 7.0).all() and (ybuf[..., off + Co:] == 7.0).all()
        y4 = torch.empty_like(y32)
        B.lamp_conv3d_fwd(desc, xd, wd, bd, y4, None, ws)
        assert torch.equal(y4, y3)


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_conv_dgrad_matches_oracle(case):
    name, N, D, H, W, Ci, Co, k, s, p, tr = case
    x, w, b, dy, oshape = _inputs(case, 200)
    ref = ops.convT3d_dgrad(dy, w, (D, H, W), k, s) if tr else ops.conv3d_dgrad(dy, w, (D, H, W), k, s, p)
    desc = B.conv_desc(Ci, Co, k, s, p, tr)
    dyd, wd = dev_bf16(dy), dev_bf16(w)
    dx = torch.full((N, D, H, W, Ci), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = B.lamp_conv3d_workspace_bytes(desc, dx, B.PASS_DGRAD)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device="cuda")
    B.lamp_conv3d_dgrad(desc, dyd, wd, dx, ws)
    assert B.lamp_get_async_status() == 0
    assert_close(host_f64(dx), ref, f"{name} dgrad f32", rel=2e-5, mx=2e-5)
    if Ci % 8 == 0:
        pitch, off = Ci + 8, 8
        dxb = torch.full((N, D, H, W, pitch), 3.0, dtype=torch.bfloat16, device="cuda")
        # dy read from a channel slice as well
        dyp = torch.zeros(oshape[:4] + (Co + 8,), dtype=torch.bfloat16, device="cuda")
        dyp[..., 8:] = dyd
        B.lamp_conv3d_dgrad(desc, B.tensor(dyp, Co, 8), wd, B.tensor(dxb, Ci, off), ws)
        assert_close(host_f64(dxb[..., off:]), ops.bf16_round(ref), f"{name} dgrad bf16 slice")
        assert (dxb[..., :off] == 3.0).all()
    # the smallest accepted workspace (reduction not split) gives the same result within rounding
    nmin = B.lamp_conv3d_workspace_min_bytes(desc, dx, B.PASS_DGRAD)
    assert nmin <= nbytes
    if nmin < nbytes:
        dx2 = torch.full((N, D, H, W, Ci), float("nan"), dtype=torch.float32, device="cuda")
        B.lamp_conv3d_dgrad(desc, dyd, wd, dx2, ws[:max(nmin, 16)])
        assert B.lamp_get_async_status() == 0
        assert_close(host_f64(dx2), ref, f"{name} dgrad f32 unsplit", rel=2e-5, mx=2e-5)
    if nmin > 256:
        with pytest.raises(B.LampError) as e:
            B.lamp_conv3d_dgrad(desc, dyd, wd, dx, ws[:256])
        assert e.value.status == 3


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_conv_wgrad_matches_oracle(case):
    name, N, D, H, W, Ci, Co, k, s, p, tr = case
    x, w, b, dy, oshape = _inputs(case, 300)
    dw_ref, db_ref = ops.convT3d_wgrad(x, dy, k, s) if tr else ops.conv3d_wgrad(x, dy, k, s, p)
    desc = B.conv_desc(Ci, Co, k, s, p, tr)
    xd, dyd = dev_bf16(x), dev_bf16(dy)
    dw = torch.full((k ** 3, Co, Ci), float("nan"), dtype=torch.float32, device="cuda")
    db = torch.full((Co,), float("nan"), dtype=torch.float32, device="cuda")
    nbytes = B.lamp_conv3d_workspace_bytes(desc, xd, B.PASS_WGRAD)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device="cuda")
    B.lamp_conv3d_wgrad(desc, xd, dyd, dw, db, ws)
    assert B.lamp_get_async_status() == 0
    assert_close(host_f64(dw), dw_ref, f"{name} wgrad", rel=2e-5, mx=2e-5)
    assert_close(host_f64(db), db_ref, f"{name} dbias", rel=2e-5, mx=2e-5)
    # too small a workspace is refused
    if nbytes > 256:
        with pytest.raises(B.LampError) as e:
            B.lamp_conv3d_wgrad(desc, xd, dyd, dw, db, ws[:256])
        assert e.value.status == 3


def test_empty_volume_is_a_no_op():
    desc = B.conv_desc(8, 8)
    x = torch.empty((1, 0, 4, 4, 8), dtype=torch.bfloat16, device="cuda")
    y = torch.empty((1, 0, 4, 4, 8), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((27, 8, 8), dtype=torch.bfloat16, device="cuda")
    B.lamp_conv3d_fwd(desc, B.Tensor(w.data_ptr(), 0, 1, 0, 4, 4, 8, 8, 0), w, None,
                      B.Tensor(w.data_ptr(), 0, 1, 0, 4, 4, 8, 8, 0))
    assert B.lamp_get_async_status() == 0


def test_bounded_wait_reports_timeout_and_context_stays_usable():
    # a wait that nothing satisfies runs out, the status word says so once, and later calls work
    assert B.lamp_get_async_status() == 0
    B.lamp_selftest_wait_timeout()
    assert B.lamp_get_async_status() == 5
    assert B.lamp_get_async_status() == 0
    desc = B.conv_desc(64, 64)
    x = dev_bf16(synth.normal_bf16((1, 4, 32, 8, 64), 1))
    w = dev_bf16(synth.kaiming_bf16(27, 64, 64, 27 * 64, 2))
    y = torch.empty((1, 4, 32, 8, 64), dtype=torch.float32, device="cuda")
    B.lamp_conv3d_fwd(desc, x, w, None, y)
    assert B.lamp_get_async_status() == 0
    assert torch.isfinite(y).all()
