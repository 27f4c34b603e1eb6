"""Pins of the oracle's Adam step (one learning rate per column, App. C.1): closed forms of the
textbook algorithm, the library implementation in torch.optim on CPU, and the remark of Sec. 3.1 that
folding Y0 into the base colour's learning rate leaves the step in colour space unchanged."""
import math

import numpy as np
import pytest


def test_first_step_is_lr_times_normalised_gradient(oracle):
    rng = np.random.default_rng(1)
    p0, g = rng.normal(size=(7, 3)), rng.normal(size=(7, 3))
    lr = np.array([1e-2, 2e-3, 5e-1])
    eps = 1e-8
    p1, m1, v1 = oracle.adam_step(p0, g, np.zeros_like(p0), np.zeros_like(p0), lr, 0.9, 0.999, eps, step=1)
    # bias correction makes m_hat = g and v_hat = g^2 at step 1, whatever the betas
    assert np.allclose(p1, p0 - lr * g / (np.abs(g) + eps), rtol=1e-12, atol=0)
    assert np.allclose(m1, 0.1 * g) and np.allclose(v1, 0.001 * g * g)


def test_constant_gradient_moves_linearly(oracle):
    """With the same gradient every step, m_hat = g and v_hat = g^2 at every step: t steps move t times
    the first one.  A wrong power in either bias correction breaks this at t = 2 already."""
    p = np.array([[0.3, -1.2]]); g = np.array([[0.02, -5.0]]); lr = np.array([1e-3, 4e-2])
    m, v = np.zeros_like(p), np.zeros_like(p)
    for t in range(1, 21):
        p, m, v = oracle.adam_step(p, g, m, v, lr, 0.9, 0.99, 1e-15, step=t)
        assert np.allclose(p, np.array([[0.3, -1.2]]) - t * lr * np.sign(g), rtol=1e-10, atol=0)


def test_zero_gradient_leaves_fresh_parameters_alone(oracle):
    p0 = np.arange(12.0).reshape(4, 3)
    z = np.zeros_like(p0)
    p1, m1, v1 = oracle.adam_step(p0, z, z, z, np.ones(3), step=1)
    assert np.array_equal(p1, p0) and not m1.any() and not v1.any()
    # ... but warmed-up moments keep moving them (the update must touch Gaussians without a gradient too)
    p2, _, _ = oracle.adam_step(p0, z, np.full_like(p0, 0.5), np.full_like(p0, 0.25), np.ones(3), step=3)
    assert np.all(p2 < p0)


def test_learning_rate_is_per_column(oracle):
    g = np.tile(np.array([[0.7]]), (5, 4)); p0 = np.zeros((5, 4))
    lr = np.array([1.0, 3.0, 0.0, 0.5]) * 1e-3
    p1, _, _ = oracle.adam_step(p0, g, p0, p0, lr, step=1)
    assert np.allclose(p1 / p1[:, :1], lr / lr[0])        # same state, same gradient: steps in the ratio of the rates
    assert not p1[:, 2].any()


def test_against_torch_adam_on_cpu(oracle):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    rows, cols, steps = 9, 4, 6
    lr = np.array([1e-2, 3e-3, 8e-3, 2.5e-4]); b1, b2, eps = 0.9, 0.99, 1e-8
    p0 = rng.normal(size=(rows, cols))
    grads = rng.normal(size=(steps, rows, cols)) * np.array([1.0, 10.0, 0.1, 1.0])
    p, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
    for t in range(steps):
        p, m, v = oracle.adam_step(p, grads[t], m, v, lr, b1, b2, eps, step=t + 1)
    # the library routine: one parameter group per column
    cols_t = [torch.tensor(p0[:, c].copy(), dtype=torch.float64, requires_grad=True) for c in range(cols)]
    opt = torch.optim.Adam([{"params": [cols_t[c]], "lr": float(lr[c])} for c in range(cols)], betas=(b1, b2), eps=eps)
    for t in range(steps):
        for c in range(cols):
            cols_t[c].grad = torch.tensor(grads[t][:, c].copy(), dtype=torch.float64)
        opt.step()
    want = np.stack([c.detach().numpy() for c in cols_t], 1)
    assert np.allclose(p, want, rtol=1e-11, atol=1e-14)


def test_folding_y0_into_the_learning_rate_keeps_the_colour_step(oracle):
    """Sec. 3.1: the colour is Y0 * theta in Eq. 1 and c0 in Eq. 2; optimising c0 with the rate scaled by
    Y0 moves the colour as optimising theta does, because Adam normalises the gradient's magnitude."""
    y0 = 0.5 / math.sqrt(math.pi)
    rng = np.random.default_rng(9)
    theta = rng.normal(size=(6, 3)); c0 = y0 * theta
    m_t = v_t = m_c = v_c = np.zeros_like(theta)
    lr = np.full(3, 0.0025)
    for t in range(1, 6):
        g_colour = rng.normal(size=theta.shape)            # dL/d colour
        theta, m_t, v_t = oracle.adam_step(theta, y0 * g_colour, m_t, v_t, lr, step=t)
        c0, m_c, v_c = oracle.adam_step(c0, g_colour, m_c, v_c, lr * y0, step=t)
        assert np.allclose(y0 * theta, c0, rtol=1e-9, atol=1e-12)
