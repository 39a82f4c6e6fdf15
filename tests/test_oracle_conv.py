"""Pins for the oracle's convolution passes (CPU only).

Each test ties the oracle to something other than itself: a closed form, an
impulse response, an adjoint identity, a sub-sampling identity, or a library
routine (torch fp64 CPU convolutions / autograd) used purely as a cross-check.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ops


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _torch_w(w, k):
    # w[tap][co][ci] -> torch [co][ci][kd][kh][kw]
    T, Co, Ci = w.shape
    return torch.from_numpy(w.reshape(k, k, k, Co, Ci)).permute(3, 4, 0, 1, 2).contiguous()


def _torch_wT(w, k):
    # transposed conv in torch: weight [ci][co][kd][kh][kw]
    T, Co, Ci = w.shape
    return torch.from_numpy(w.reshape(k, k, k, Co, Ci)).permute(4, 3, 0, 1, 2).contiguous()


def _ncdhw(x):
    return torch.from_numpy(x).permute(0, 4, 1, 2, 3).contiguous()


def _ndhwc(t):
    return t.permute(0, 2, 3, 4, 1).contiguous().numpy()


CASES = [  # (N, D, H, W, Ci, Co, k, s, p)
    (1, 5, 6, 7, 3, 4, 3, 1, 1),
    (2, 6, 4, 8, 2, 5, 3, 2, 1),
    (1, 4, 4, 4, 5, 3, 1, 1, 0),
    (1, 7, 5, 6, 1, 2, 3, 1, 1),
    (1, 6, 6, 6, 4, 4, 2, 2, 0),
]


@pytest.mark.parametrize("case", CASES)
def test_conv_passes_match_library_special_case(case):
    N, D, H, W, Ci, Co, k, s, p = case
    x = _rand((N, D, H, W, Ci), 1)
    w = _rand((k ** 3, Co, Ci), 2)
    b = _rand((Co,), 3)
    y = ops.conv3d_fwd(x, w, b, k, s, p)
    xt = _ncdhw(x).requires_grad_(True)
    wt = _torch_w(w, k).requires_grad_(True)
    bt = torch.from_numpy(b).requires_grad_(True)
    yt = F.conv3d(xt, wt, bt, stride=s, padding=p)
    np.testing.assert_allclose(y, _ndhwc(yt.detach()), rtol=1e-12, atol=1e-12)
    dy = _rand(y.shape, 4)
    gx, gw, gb = torch.autograd.grad(yt, (xt, wt, bt), _ncdhw(dy))
    dx = ops.conv3d_dgrad(dy, w, (D, H, W), k, s, p)
    dw, db = ops.conv3d_wgrad(x, dy, k, s, p)
    np.testing.assert_allclose(dx, _ndhwc(gx), rtol=1e-12, atol=1e-12)
    gw_np = gw.permute(2, 3, 4, 0, 1).reshape(k ** 3, Co, Ci).numpy()
    np.testing.assert_allclose(dw, gw_np, rtol=1e-12, atol=1e-11)
    np.testing.assert_allclose(db, gb.numpy(), rtol=1e-12, atol=1e-11)


@pytest.mark.parametrize("shape", [(1, 3, 4, 5, 3, 2), (2, 2, 3, 2, 4, 5)])
def test_transposed_conv_matches_library_special_case(shape):
    N, D, H, W, Ci, Co = shape
    x = _rand((N, D, H, W, Ci), 5)
    w = _rand((8, Co, Ci), 6)
    b = _rand((Co,), 7)
    y = ops.convT3d_fwd(x, w, b, 2, 2)
    xt = _ncdhw(x).requires_grad_(True)
    wt = _torch_wT(w, 2).requires_grad_(True)
    bt = torch.from_numpy(b).requires_grad_(True)
    yt = F.conv_transpose3d(xt, wt, bt, stride=2)
    np.testing.assert_allclose(y, _ndhwc(yt.detach()), rtol=1e-12, atol=1e-12)
    dy = _rand(y.shape, 8)
    gx, gw, gb = torch.autograd.grad(yt, (xt, wt, bt), _ncdhw(dy))
    np.testing.assert_allclose(ops.convT3d_dgrad(dy, w, (D, H, W), 2, 2), _ndhwc(gx), rtol=1e-12, atol=1e-12)
    dw, db = ops.convT3d_wgrad(x, dy, 2, 2)
    np.testing.assert_allclose(dw, gw.permute(2, 3, 4, 1, 0).reshape(8, Co, Ci).numpy(), rtol=1e-12, atol=1e-11)
    np.testing.assert_allclose(db, gb.numpy(), rtol=1e-12, atol=1e-11)


def test_all_ones_counts_in_bounds_taps():
    # x = 1, w = 1, b = 0: y = C_in * (# taps inside the volume): 27 interior, 18 face, 12 edge, 8 corner
    Ci = 3
    y = ops.conv3d_fwd(np.ones((1, 5, 5, 5, Ci)), np.ones((27, 2, Ci)), None, 3, 1, 1)
    assert y[0, 2, 2, 2, 0] == 27 * Ci
    assert y[0, 0, 2, 2, 1] == 18 * Ci
    assert y[0, 0, 0, 2, 0] == 12 * Ci
    assert y[0, 0, 0, 0, 1] == 8 * Ci
    assert y[0, 4, 4, 4, 0] == 8 * Ci


def test_delta_impulse_reproduces_mirrored_kernel():
    # cross-correlation: an impulse at v0 in channel ci puts w[(kd,kh,kw)][co][ci] at v0 - (k - 1)
    D = 7
    w = _rand((27, 2, 3), 9)
    x = np.zeros((1, D, D, D, 3))
    x[0, 3, 3, 3, 1] = 1.0
    y = ops.conv3d_fwd(x, w, None, 3, 1, 1)
    for kd in range(3):
        for kh in range(3):
            for kw in range(3):
                t = (kd * 3 + kh) * 3 + kw
                np.testing.assert_array_equal(y[0, 3 - (kd - 1), 3 - (kh - 1), 3 - (kw - 1), :], w[t, :, 1])
    assert np.count_nonzero(y) == 27 * 2


def test_transposed_conv_one_input_per_output():
    w = _rand((8, 2, 3), 10)
    x = np.zeros((1, 3, 3, 3, 3))
    x[0, 1, 2, 0, 2] = 1.0
    y = ops.convT3d_fwd(x, w, None, 2, 2)
    for a in range(2):
        for b in range(2):
            for c in range(2):
                np.testing.assert_array_equal(y[0, 2 + a, 4 + b, 0 + c, :], w[(a * 2 + b) * 2 + c, :, 2])
    assert np.count_nonzero(y) == 8 * 2


@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (3, 2, 1), (1, 1, 0)])
def test_adjoint_identities(k, s, p):
    N, D, H, W, Ci, Co = 1, 6, 4, 8, 3, 4
    x = _rand((N, D, H, W, Ci), 11)
    w = _rand((k ** 3, Co, Ci), 12)
    y = ops.conv3d_fwd(x, w, None, k, s, p)
    g = _rand(y.shape, 13)
    # <conv(x), g> = <x, dgrad(g)>
    lhs = float((y * g).sum())
    assert abs(lhs - float((x * ops.conv3d_dgrad(g, w, (D, H, W), k, s, p)).sum())) <= 1e-12 * abs(lhs) + 1e-12
    # <dw, w'> = <g, conv(x; w')>
    w2 = _rand(w.shape, 14)
    dw, db = ops.conv3d_wgrad(x, g, k, s, p)
    rhs = float((g * ops.conv3d_fwd(x, w2, None, k, s, p)).sum())
    assert abs(float((dw * w2).sum()) - rhs) <= 1e-11 * abs(rhs) + 1e-11
    np.testing.assert_allclose(db, g.sum(axis=(0, 1, 2, 3)), rtol=1e-12)


def test_transposed_adjoint_is_stride2_k2_conv():
    # <up(x), y> = <x, conv_{k2,s2,p0}(y)> with the same w read as [tap][ci-as-out][co-as-in]
    x = _rand((1, 3, 4, 2, 3), 15)
    w = _rand((8, 5, 3), 16)            # [tap][co][ci]
    u = ops.convT3d_fwd(x, w, None, 2, 2)
    g = _rand(u.shape, 17)
    wt = np.ascontiguousarray(w.transpose(0, 2, 1))     # conv weights [tap][out=ci][in=co]
    rhs = float((x * ops.conv3d_fwd(g, wt, None, 2, 2, 0)).sum())
    assert abs(float((u * g).sum()) - rhs) <= 1e-12 * abs(rhs)


def test_stride2_is_subsampled_stride1():
    x = _rand((1, 8, 6, 10, 2), 18)
    w = _rand((27, 3, 2), 19)
    b = _rand((3,), 20)
    y1 = ops.conv3d_fwd(x, w, b, 3, 1, 1)
    y2 = ops.conv3d_fwd(x, w, b, 3, 2, 1)
    np.testing.assert_array_equal(y2, y1[:, ::2, ::2, ::2, :])


def test_dgrad_s1p1_is_fwd_with_mirrored_taps_and_swapped_channels():
    x = _rand((1, 5, 4, 6, 4), 21)
    w = _rand((27, 4, 3), 22)          # [t][co=4][ci=3]
    dx = ops.conv3d_dgrad(x, w, (5, 4, 6), 3, 1, 1)
    wm = np.ascontiguousarray(w[::-1].transpose(0, 2, 1))
    np.testing.assert_allclose(dx, ops.conv3d_fwd(x, wm, None, 3, 1, 1), rtol=1e-13, atol=1e-13)


def test_wgrad_finite_differences():
    x = _rand((1, 4, 5, 4, 2), 23)
    w = _rand((27, 3, 2), 24)
    g = _rand((1, 4, 5, 4, 3), 25)
    dw, _ = ops.conv3d_wgrad(x, g, 3, 1, 1)
    rs = np.random.default_rng(26)
    for _ in range(20):
        i = tuple(rs.integers(0, n) for n in w.shape)
        wp, wm = w.copy(), w.copy()
        wp[i] += 1e-5
        wm[i] -= 1e-5
        fd = ((ops.conv3d_fwd(x, wp, None, 3, 1, 1) - ops.conv3d_fwd(x, wm, None, 3, 1, 1)) * g).sum() / 2e-5
        assert abs(fd - dw[i]) <= 1e-6 * max(1.0, abs(dw[i]))


def test_point_evaluated_variants_equal_full():
    x = _rand((2, 5, 6, 4, 3), 27)
    w = _rand((27, 4, 3), 28)
    b = _rand((4,), 29)
    for s in (1, 2):
        y = ops.conv3d_fwd(x, w, b, 3, s, 1)
        pts = np.array([[n, d, h, ww] for n in range(2) for d in range(y.shape[1])
                        for h in range(y.shape[2]) for ww in range(y.shape[3])], dtype=np.int32)
        np.testing.assert_array_equal(ops.conv3d_fwd_points(x, w, b, pts, 3, s, 1).reshape(y.shape), y)
        g = _rand(y.shape, 30)
        dw, _ = ops.conv3d_wgrad(x, g, 3, s, 1)
        ent = np.array([[t, co, ci] for t in range(27) for co in range(4) for ci in range(3)], dtype=np.int32)
        np.testing.assert_array_equal(ops.conv3d_wgrad_points(x, g, ent, 3, s, 1).reshape(dw.shape), dw)
