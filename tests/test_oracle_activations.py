"""Pins of the colour activations of Sec. 3.1: the printed formulas evaluated by hand, the facts the paper
states about them (all map zero to 0.5 and match the baseline's slope there; the bounded ones stay in
[0, 1]), and the derivative against finite differences through the oracle's appearance backward."""
import math

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes

ACTS = [0, 1, 2, 3]


def _by_hand(act, x):
    z = x + 0.5
    if act == 0:
        return max(z, 0.0)
    if act == 1:
        return math.log(1.0 + math.exp(10.0 * z)) / 10.0
    if act == 2:
        return 1.0 / (1.0 + math.exp(-4.0 * x))
    return min(max(z, 0.0), 1.0)


@pytest.mark.parametrize("act", ACTS)
def test_formula_and_operating_point(oracle, act):
    for x in (-1.3, -0.5, -0.2, 0.0, 0.1, 0.49, 0.7, 2.0):
        assert abs(oracle.color_act(act, x) - _by_hand(act, x)) < 1e-14
    # "all four map zero to 0.5 ... and closely match the baseline ReLU near this operating point"
    assert abs(oracle.color_act(act, 0.0) - 0.5) < 1e-3
    assert abs(oracle.color_act_grad(act, 0.0) - 1.0) < 1e-2
    assert abs(oracle.color_act(act, 0.05) - oracle.color_act(0, 0.05)) < 2e-3
    xs = np.linspace(-3, 3, 601)
    ys = np.array([oracle.color_act(act, float(x)) for x in xs])
    assert np.all(np.diff(ys) >= 0) and ys.min() >= 0
    if act in (2, 3):
        assert ys.max() <= 1.0
    if act == 3:
        assert oracle.color_act(act, -0.6) == 0.0 and oracle.color_act(act, 0.6) == 1.0
    if act == 1:                                          # the smooth rectifier approaches the baseline away from the kink
        assert abs(oracle.color_act(1, 1.0) - 1.5) < 1e-6 and oracle.color_act(1, -1.5) < 1e-4


@pytest.mark.parametrize("act", ACTS)
def test_derivative_by_finite_differences(oracle, act):
    for x in (-0.8, -0.3, 0.0, 0.2, 0.45, 0.9):
        if act in (0, 3) and min(abs(x + 0.5), abs(x - 0.5)) < 1e-3:
            continue
        h = 1e-6
        fd = (oracle.color_act(act, x + h) - oracle.color_act(act, x - h)) / (2 * h)
        assert abs(fd - oracle.color_act_grad(act, x)) < 1e-7


@pytest.mark.parametrize("act", [1, 2, 3])
@pytest.mark.parametrize("app", [scenes.APP_SH, scenes.APP_NEURAL])
def test_appearance_backward_uses_the_activation(oracle, act, app):
    """dL/d(base colour) of the separate-pass decode against central differences of its forward."""
    w = scenes.config2(n=40, app=app)
    sc = w.scene
    sc.color_activation = act
    rng = np.random.default_rng(act)
    sc.base_color = rng.uniform(-0.6, 0.6, sc.base_color.shape).astype(np.float32)
    if app == scenes.APP_NEURAL:
        sc.features = rng.normal(0, 0.5, sc.features.shape).astype(np.float16)
    d = scenes.unit_directions(sc.n, 5)
    g = rng.normal(size=(sc.n, 3))
    out = oracle.appearance_backward(sc, d, g)
    g_base = out.base_color if hasattr(out, "base_color") else out[0]
    col0 = oracle.appearance_forward(sc, d)
    col0 = col0[0] if isinstance(col0, tuple) else col0
    assert np.abs(col0 - (np.maximum(sc.base_color + 0.5, 0))).max() > 1e-3       # not the baseline's colours
    h = 1e-4
    base0 = sc.base_color.copy()
    fd = np.zeros_like(g_base)
    for c in range(3):
        for sgn in (+1, -1):
            sc.base_color = base0.astype(np.float64).copy()
            sc.base_color[:, c] += sgn * h
            col = oracle.appearance_forward(sc, d)
            col = col[0] if isinstance(col, tuple) else col
            fd[:, c] += sgn * (col[:, c] * g[:, c]) / (2 * h)
    sc.base_color = base0
    ok = np.ones_like(fd, bool)
    if act == 3:                                             # skip elements within h of a kink of the clamp
        A = col0 * 0
        ok = (np.abs(col0) > 1e-3) & (np.abs(col0 - 1) > 1e-3)
    assert np.abs(fd - g_base)[ok].max() < 1e-6
