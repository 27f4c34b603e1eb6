"""The oracle's analytic backward against central finite differences of its own forward
(double precision, tiny scenes), plus closed forms and invariants of the gradients."""
import copy
import math
from types import SimpleNamespace

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes


def tiny_scene(app, seed, n=12, deg=3):
    rng = np.random.default_rng(seed)
    means = np.stack([rng.uniform(-0.9, 0.9, n), rng.uniform(-0.9, 0.9, n), rng.uniform(2, 4, n)], 1)
    sc = SimpleNamespace(
        means=means, log_scales=rng.normal(-1.8, 0.4, (n, 3)), quats=rng.standard_normal((n, 4)),
        opacity_logits=rng.normal(0.5, 1.0, n), base_color=rng.normal(0.0, 0.3, (n, 3)), app=app,
        active_degree=deg, sh_rest=None, features=None, mlp_weights=None)
    sc.opacity_logits[0] = 6.0            # alpha clamped at 0.99 near its centre
    sc.log_scales[0] = -2.5
    sc.means[1] = [2.6, 0.3, 3.0]         # outside 1.3 x the frustum: the clamped Jacobian branch
    sc.log_scales[1] = [-0.3, -0.8, -0.5]  # ... but large enough to reach into the image
    sc.base_color[2] = [-0.7, 0.1, -0.6]  # two channels cut by the ReLU
    if app == 0:
        sc.sh_rest = rng.normal(0, 0.2, (n, 15, 3))
    else:
        sc.features = rng.normal(0, 0.7, (n, 8))
        sc.mlp_weights = rng.uniform(-0.6, 0.6, 816)
    return sc


def tiny_cam(theta=None):
    if theta is None:
        cam = scenes.identity_camera(24, 24, 32.0, background=(0.2, 0.5, 0.1))
    else:
        cam = scenes.orbit_camera(24, 24, theta, radius=3.0, background=(0.2, 0.5, 0.1))
        cam.w2c = np.asarray(cam.w2c, np.float64)
    return cam


PARAMS = {0: ["means", "log_scales", "quats", "opacity_logits", "base_color", "sh_rest"],
          1: ["means", "log_scales", "quats", "opacity_logits", "base_color", "features", "mlp_weights"]}


def loss(oracle, sc, cam, G):
    fwd, _ = oracle.render(sc, cam)
    return float((G * fwd.image).sum())


def fd_check(oracle, sc, cam, G, names, h=1e-6, stride=1):
    _, grads = oracle.render(sc, cam, G)
    report = {}
    for name in names:
        an = getattr(grads, name).reshape(-1)
        arr = getattr(sc, name)
        flat = arr.reshape(-1)
        bad, skipped, checked, worst = 0, 0, 0, 0.0
        for k in range(0, flat.size, stride):
            keep = flat[k]
            vals = []
            for step in (h, 2 * h):
                flat[k] = keep + step; lp = loss(oracle, sc, cam, G)
                flat[k] = keep - step; lm = loss(oracle, sc, cam, G)
                vals.append((lp - lm) / (2 * step))
            flat[k] = keep
            scale = max(abs(vals[0]), abs(an[k]))
            if abs(vals[0] - vals[1]) > 1e-6 * scale + 5e-7:
                skipped += 1          # an integer decision flipped inside the stencil
                continue
            checked += 1
            err = abs(vals[0] - an[k])
            worst = max(worst, err / (scale + 1e-30) if scale > 1e-3 else 0.0)
            if err > 1e-6 * scale + 5e-7:
                bad += 1
        report[name] = (checked, skipped, bad, worst, float(np.abs(an).max()))
    return report


@pytest.mark.parametrize("app", [0, 1])
@pytest.mark.parametrize("theta", [None, 1.1])
def test_full_backward_against_finite_differences(oracle, app, theta):
    sc = tiny_scene(app, seed=20 + app)
    cam = tiny_cam(theta)
    if theta is not None:   # put the scene in front of the orbit camera
        sc.means = sc.means - np.array([0.0, 0.0, 3.0])
    G = np.random.default_rng(99).standard_normal((3, cam.height, cam.width))
    fwd, _ = oracle.render(sc, cam)
    assert fwd.pre.visible.sum() >= 10
    stride = {"sh_rest": 3, "mlp_weights": 5}
    for name in PARAMS[app]:
        rep = fd_check(oracle, sc, cam, G, [name], stride=stride.get(name, 1))[name]
        checked, skipped, bad, worst, gmax = rep
        assert gmax > 1e-3, (name, rep)                   # the gradient is actually exercised
        assert bad == 0, (name, rep)
        assert skipped <= 0.1 * (checked + skipped), (name, rep)


def test_clamped_branches_are_exercised(oracle):
    """The tiny scene really hits the alpha clamp, the Jacobian clamp and the ReLU cut."""
    sc = tiny_scene(0, seed=20)
    cam = tiny_cam()
    fwd, _ = oracle.render(sc, cam)
    pre = fwd.pre
    assert pre.visible[0] and pre.opacity[0] > 0.99
    assert pre.visible[1] and abs(sc.means[1, 0] / sc.means[1, 2]) > 1.3 * 12 / 32
    assert (fwd.color[2] == 0).sum() == 2


@pytest.mark.parametrize("app", [0, 1])
def test_gradient_invariants(oracle, app):
    sc = tiny_scene(app, seed=31)
    cam = tiny_cam(0.4)
    sc.means = sc.means - np.array([0.0, 0.0, 3.0])
    G = np.random.default_rng(5).standard_normal((3, 24, 24))
    fwd, g = oracle.render(sc, cam, G)
    vis = fwd.pre.visible.astype(bool)
    # a quaternion's scale does not matter: its gradient is orthogonal to it
    assert np.abs((g.quats * sc.quats).sum(1)).max() < 1e-12 * max(1, np.abs(g.quats).max())
    # culled Gaussians get exact zeros everywhere
    for name in PARAMS[app]:
        if name == "mlp_weights":
            continue
        a = getattr(g, name).reshape(sc.means.shape[0], -1)
        assert np.all(a[~vis] == 0)
    # appearance-only part of dL/dmean is tangent to the view direction
    zero = np.zeros_like
    gp = oracle.preprocess_backward(sc.means, sc.log_scales, sc.quats, sc.opacity_logits, cam,
                                    fwd.pre.visible, zero(g.blend.mean2d), zero(g.blend.conic),
                                    zero(g.blend.opacity), g.dirs)
    assert np.abs(gp.means).max() > 1e-4           # colour gradients do reach the positions
    assert np.abs((gp.means * fwd.pre.dir).sum(1)).max() < 1e-12
    assert np.all(gp.log_scales == 0) and np.all(gp.quats == 0)


def test_single_gaussian_gradient_closed_forms(oracle):
    cam = scenes.identity_camera(32, 32, 32.0)      # black background
    o = 0.6
    sc = SimpleNamespace(means=np.array([[0.1, -0.05, 3.0]]), log_scales=np.full((1, 3), math.log(0.25)),
                         quats=np.array([[1.0, 0, 0, 0]]), opacity_logits=np.array([math.log(o / (1 - o))]),
                         base_color=np.array([[0.2, -0.1, 0.3]]), app=0, active_degree=0,
                         sh_rest=np.zeros((1, 15, 3)), features=None, mlp_weights=None)
    G = np.random.default_rng(6).standard_normal((3, 32, 32))
    fwd, g = oracle.render(sc, cam, G)
    alpha = 1 - fwd.final_T                       # single Gaussian: alpha(p) = 1 - T(p)
    c = fwd.color[0]
    assert np.allclose(g.blend.color[0], (alpha[None] * G).sum((1, 2)), rtol=1e-13)
    assert np.allclose(g.base_color[0], (alpha[None] * G).sum((1, 2)), rtol=1e-13)
    # d alpha / d o = alpha / o where the Gaussian is composited (no clamp at o = 0.6)
    dldo = ((alpha / o)[None] * G * c[:, None, None]).sum()
    assert abs(g.blend.opacity[0] - dldo) < 1e-12 * abs(dldo)
    assert abs(g.opacity_logits[0] - dldo * o * (1 - o)) < 1e-12 * abs(dldo)


def test_appearance_backward_finite_differences_on_free_directions(oracle):
    """Standalone decode: gradients w.r.t. directions taken as free R^3 vectors."""
    rng = np.random.default_rng(7)
    n = 6
    for app in (0, 1):
        sc = tiny_scene(app, seed=40, n=n, deg=3)
        d = rng.standard_normal((n, 3)) * 0.8
        gc = rng.standard_normal((n, 3))
        g = oracle.appearance_backward(sc, d, gc)
        h = 1e-6
        for i in range(n):
            for a in range(3):
                dp = d.copy(); dp[i, a] += h
                dm = d.copy(); dm[i, a] -= h
                fd = ((oracle.appearance_forward(sc, dp)[0] - oracle.appearance_forward(sc, dm)[0]) * gc).sum() / (2 * h)
                assert abs(fd - g.dirs[i, a]) < 1e-7 * max(1, abs(fd))
