"""Pins of the parameter-update oracle (Sec. 3, training setup: RMSProp, learning rate 1e-3) against what the
method and the mathematics fix: a library implementation of the same published update, closed forms of the first and
of the stationary step, invariances, and the zero-gradient case."""
import numpy as np
import torch

from oracle import optim as O
from oracle import ops
from paper_2006_12575_b200 import synth


def _rand(n, seed, scale=1.0):
    return synth.rng(seed).standard_normal(n) * scale


def test_matches_library_rmsprop_over_several_steps():
    w0 = _rand(257, 1)
    p = torch.tensor(w0.copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.RMSprop([p], lr=1e-3, alpha=0.99, eps=1e-8, momentum=0.0, centered=False, weight_decay=0.0)
    w, v = w0.copy(), np.zeros_like(w0)
    for step in range(4):
        g = _rand(257, 10 + step, scale=10.0 ** (step - 2))
        p.grad = torch.tensor(g.copy(), dtype=torch.float64)
        opt.step()
        w, v, _ = O.rmsprop_step(w, g, v, 1e-3, 0.99, 1e-8)
        np.testing.assert_allclose(w, p.detach().numpy(), rtol=1e-13, atol=1e-15)


def test_first_step_closed_form():
    # from v = 0: dw = -lr * g / (sqrt(1 - alpha) * |g| + eps)
    g = _rand(100, 2)
    w = _rand(100, 3)
    lr, alpha, eps = 1e-3, 0.9, 1e-8
    w1, v1, _ = O.rmsprop_step(w, g, np.zeros(100), lr, alpha, eps)
    np.testing.assert_allclose(v1, (1 - alpha) * g * g, rtol=1e-14)
    np.testing.assert_allclose(w1 - w, -lr * g / (np.sqrt(1 - alpha) * np.abs(g) + eps), rtol=1e-12)
    # with eps = 0 the step has the same size for every element: lr / sqrt(1 - alpha), against the gradient's sign
    w2, _, _ = O.rmsprop_step(w, g, np.zeros(100), lr, alpha, 0.0)
    np.testing.assert_allclose(w2 - w, -np.sign(g) * lr / np.sqrt(1 - alpha), rtol=1e-12)


def test_constant_gradient_reaches_unit_steps():
    # v converges to g^2 (v_t = (1 - alpha^t) g^2), so the step tends to lr * sign(g)
    g = np.array([3.0, -0.25, 1e-3])
    w, v = np.zeros(3), np.zeros(3)
    for t in range(1, 400):
        w_prev = w
        w, v, _ = O.rmsprop_step(w, g, v, 1e-3, 0.9, 0.0)
        np.testing.assert_allclose(v, (1 - 0.9 ** t) * g * g, rtol=1e-10)
    np.testing.assert_allclose(w - w_prev, -1e-3 * np.sign(g), rtol=1e-9)


def test_scale_invariance_and_sign():
    # without eps, scaling all gradients of the history by c > 0 leaves the parameters unchanged
    w0 = _rand(64, 4)
    for c in (1e-3, 7.0):
        wa, va = w0.copy(), np.zeros(64)
        wb, vb = w0.copy(), np.zeros(64)
        for step in range(3):
            g = _rand(64, 20 + step)
            wa, va, _ = O.rmsprop_step(wa, g, va, 1e-3, 0.99, 0.0)
            wb, vb, _ = O.rmsprop_step(wb, c * g, vb, 1e-3, 0.99, 0.0)
        np.testing.assert_allclose(wa, wb, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(vb, c * c * va, rtol=1e-12)
    # every element moves against its gradient
    g = _rand(64, 5)
    w1, _, _ = O.rmsprop_step(w0, g, np.ones(64), 1e-3, 0.99, 1e-8)
    assert (np.sign(w1 - w0) == -np.sign(g)).all()


def test_zero_gradient_and_bf16_copy():
    w = _rand(50, 6)
    v = np.abs(_rand(50, 7))
    w1, v1, wb = O.rmsprop_step(w, np.zeros(50), v, 1e-3, 0.99, 1e-8)
    np.testing.assert_array_equal(w1, w)
    np.testing.assert_allclose(v1, 0.99 * v, rtol=1e-15)
    np.testing.assert_array_equal(wb, ops.bf16_round(w))          # the bf16 copy is the rounded master copy
    assert np.abs(wb - w).max() <= np.abs(w).max() * 2.0 ** -8
