"""Pins for the CPU oracle: closed forms, invariants, brute force and the values the paper
prints.  None of these re-types an oracle formula; each checks a consequence that a dropped
term, a wrong sign or a transposed operand would break.  (Finite differences are in
test_oracle_gradients.py.)"""
import math
import os
from types import SimpleNamespace

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def one_gaussian_scene(mean, log_scale, logit, base, quat=(1, 0, 0, 0), sh_rest=None):
    return SimpleNamespace(
        means=np.array([mean], np.float64), log_scales=np.array([[log_scale] * 3], np.float64)
        if np.isscalar(log_scale) else np.array([log_scale], np.float64),
        quats=np.array([quat], np.float64), opacity_logits=np.array([logit], np.float64),
        base_color=np.array([base], np.float64), app=0, active_degree=3,
        sh_rest=np.zeros((1, 15, 3)) if sh_rest is None else sh_rest, features=None, mlp_weights=None)


# ------------------------------------------------------------------------------ paper values

def test_paper_printed_values(oracle):
    g = golden()
    assert oracle.num_mlp_weights() == g["mlp_parameters"]
    assert g["mlp_input_dim"] * g["mlp_hidden"] + g["mlp_hidden"] ** 2 + g["mlp_hidden"] * g["mlp_outputs"] \
        == g["mlp_parameters"]
    assert oracle.mlp_macs(False) == g["mac_full"]
    assert oracle.mlp_macs(True) == g["mac_folded"]
    assert 3 * 4 + g["num_features"] * 2 == g["bytes_neural"]
    assert g["sh3_coefficients"] * 4 == g["bytes_sh3"]
    assert scenes.MLP_NUM_WEIGHTS == g["mlp_parameters"]
    Y = oracle.sh_basis([0.0, 0.0, 1.0])
    assert round(Y[0], 3) == g["y0"]
    assert abs(Y[0] - 1.0 / math.sqrt(4 * math.pi)) < 1e-15
    assert oracle.TILE == g["tile_size"]


# ------------------------------------------------------------------------------ rotations

def test_quaternion_rotation(oracle):
    rng = np.random.default_rng(1)
    for _ in range(20):
        q = rng.standard_normal(4) * rng.uniform(0.1, 5)
        R = oracle.quat_to_rot(q)
        assert np.abs(R.T @ R - np.eye(3)).max() < 1e-14
        assert abs(np.linalg.det(R) - 1) < 1e-14
        # rotating by q: v' = q v q^-1; check against the axis-angle (Rodrigues) form
        qn = q / np.linalg.norm(q)
        ang = 2 * math.atan2(np.linalg.norm(qn[1:]), qn[0])
        ax = qn[1:] / np.linalg.norm(qn[1:])
        K = np.array([[0, -ax[2], ax[1]], [ax[2], 0, -ax[0]], [-ax[1], ax[0], 0]])
        Rod = np.eye(3) + math.sin(ang) * K + (1 - math.cos(ang)) * K @ K
        assert np.abs(R - Rod).max() < 1e-13
    assert np.abs(oracle.quat_to_rot([1, 0, 0, 0]) - np.eye(3)).max() == 0
    Rz = oracle.quat_to_rot([math.cos(math.pi / 4), 0, 0, math.sin(math.pi / 4)])
    assert np.abs(Rz - np.array([[0, -1, 0], [1, 0, 0], [0, 0, 1.0]])).max() < 1e-15


# ------------------------------------------------------------------------------ projection

def test_on_axis_isotropic_projection(oracle):
    cam = scenes.identity_camera(64, 64, 64.0)
    s, z = 0.1, 3.0
    rng = np.random.default_rng(2)
    for _ in range(5):
        q = rng.standard_normal(4)  # isotropic: any rotation gives Sigma = s^2 I
        sc = one_gaussian_scene([0, 0, z], math.log(s), 0.3, [0, 0, 0], quat=q)
        pre = oracle.preprocess(sc.means, sc.log_scales, sc.quats, sc.opacity_logits, cam)
        var = (s * 64.0 / z) ** 2 + 0.3
        assert pre.visible[0] == 1
        assert np.allclose(pre.mean2d[0], [32, 32], atol=1e-13)
        assert np.allclose(pre.cov2d[0], [var, 0, var], atol=1e-13)
        assert np.allclose(pre.conic[0], [1 / var, 0, 1 / var], atol=1e-13)
        assert abs(pre.opacity[0] - 1 / (1 + math.exp(-0.3))) < 1e-15
        assert pre.depth32[0] == np.float32(z)
        assert np.allclose(pre.dir[0], [0, 0, 1])
        # extent: alpha = 1/255 exactly at the edge of the box along the axes
        ex = pre.extent[0, 0]
        assert abs(pre.opacity[0] * math.exp(-0.5 * ex * ex / var) - 1 / 255) < 1e-15


def test_off_axis_isotropic_projection(oracle):
    cam = scenes.identity_camera(128, 96, 100.0)
    cam.fy = 90.0
    s = 0.05
    x, y, z = 0.4, -0.3, 2.5  # inside the 1.3 x frustum limit
    sc = one_gaussian_scene([x, y, z], math.log(s), 1.0, [0, 0, 0], quat=[0.3, -0.5, 0.1, 0.8])
    pre = oracle.preprocess(sc.means, sc.log_scales, sc.quats, sc.opacity_logits, cam)
    fx, fy = cam.fx, cam.fy
    jj = np.array([[fx * fx / z ** 2 * (1 + x * x / z ** 2), fx * fy * x * y / z ** 4],
                   [fx * fy * x * y / z ** 4, fy * fy / z ** 2 * (1 + y * y / z ** 2)]])
    cov = s * s * jj + 0.3 * np.eye(2)
    assert np.allclose(pre.cov2d[0], [cov[0, 0], cov[0, 1], cov[1, 1]], rtol=1e-13)
    Q = np.linalg.inv(cov)
    assert np.allclose(pre.conic[0], [Q[0, 0], Q[0, 1], Q[1, 1]], rtol=1e-12)
    assert np.allclose(pre.mean2d[0], [fx * x / z + 64, fy * y / z + 48], rtol=1e-14)
    d = np.array([x, y, z]) / np.linalg.norm([x, y, z])
    assert np.allclose(pre.dir[0], d, atol=1e-15)


def test_anisotropic_projection_against_numpy(oracle):
    """Sigma' = J W Sigma W^T J^T with a rotated camera, written with numpy matrices."""
    rng = np.random.default_rng(3)
    cam = scenes.orbit_camera(200, 120, 0.7)
    mu = np.array([0.3, -0.2, 0.4]); ls = np.array([-2.0, -3.0, -1.5]); q = rng.standard_normal(4)
    sc = one_gaussian_scene(mu, ls, 0.0, [0, 0, 0], quat=q)
    pre = oracle.preprocess(sc.means, sc.log_scales, sc.quats, sc.opacity_logits, cam)
    Rw = np.asarray(cam.w2c, np.float64)[:, :3]; tw = np.asarray(cam.w2c, np.float64)[:, 3]
    t = Rw @ mu + tw
    R = oracle.quat_to_rot(q)
    Sigma = R @ np.diag(np.exp(2 * ls)) @ R.T
    J = np.array([[cam.fx / t[2], 0, -cam.fx * t[0] / t[2] ** 2], [0, cam.fy / t[2], -cam.fy * t[1] / t[2] ** 2]])
    cov = J @ Rw @ Sigma @ Rw.T @ J.T + 0.3 * np.eye(2)
    assert np.allclose(pre.cov2d[0], [cov[0, 0], cov[0, 1], cov[1, 1]], rtol=1e-12)
    eye = -Rw.T @ tw
    assert np.allclose(pre.dir[0], (mu - eye) / np.linalg.norm(mu - eye), atol=1e-14)
    assert abs(pre.depth32[0] - t[2]) < 1e-6


def test_culling_rules(oracle):
    cam = scenes.identity_camera(64, 64, 64.0)
    def vis(mean, logit, ls=-3.0, quat=(1, 0, 0, 0)):
        sc = one_gaussian_scene(mean, ls, logit, [0, 0, 0], quat=quat)
        return int(oracle.preprocess(sc.means, sc.log_scales, sc.quats, sc.opacity_logits, cam).visible[0])
    assert vis([0, 0, 3], 0.0) == 1
    assert vis([0, 0, 0.1], 0.0) == 0            # in front of the near plane (0.2)
    assert vis([0, 0, -3], 0.0) == 0             # behind the camera
    on_centre = [0.5 * 3 / 64, 0.5 * 3 / 64, 3]  # projects onto the centre of pixel (32, 32)
    assert vis(on_centre, math.log(1 / 254.0 / (1 - 1 / 254.0))) == 1   # opacity 1/254
    assert vis(on_centre, math.log(1 / 256.0 / (1 - 1 / 256.0))) == 0   # opacity 1/256 < 1/255
    # opacity 1/254 reaches 1/255 only within ~0.1 px: no pixel centre inside => empty rect
    assert vis([0, 0, 3], math.log(1 / 254.0 / (1 - 1 / 254.0))) == 0
    assert vis([50, 0, 3], 0.0) == 0             # far outside the image
    assert vis([float("nan"), 0, 3], 0.0) == 0
    assert vis([0, 0, 3], float("inf")) == 0
    assert vis([0, 0, 3], 0.0, quat=(0, 0, 0, 0)) == 0


# ------------------------------------------------------------------------------ SH basis

def _sphere_quadrature(n_theta=64, n_phi=128):
    # Gauss-Legendre in cos(theta) x uniform in phi: exact for polynomials of the degrees used
    ct, w = np.polynomial.legendre.leggauss(n_theta)
    phi = (np.arange(n_phi) + 0.5) * 2 * math.pi / n_phi
    st = np.sqrt(1 - ct * ct)
    d = np.stack([np.outer(st, np.cos(phi)), np.outer(st, np.sin(phi)), np.outer(ct, np.ones_like(phi))], -1)
    wt = np.outer(w, np.full(n_phi, 2 * math.pi / n_phi))
    return d.reshape(-1, 3), wt.reshape(-1)


def test_sh_basis_is_orthonormal(oracle):
    d, w = _sphere_quadrature()
    Y = np.stack([oracle.sh_basis(v) for v in d])
    gram = (Y * w[:, None]).T @ Y
    assert np.abs(gram - np.eye(16)).max() < 1e-12


def test_sh_addition_theorem_and_parity(oracle):
    rng = np.random.default_rng(4)
    for _ in range(50):
        v = rng.standard_normal(3); v /= np.linalg.norm(v)
        Y = oracle.sh_basis(v)
        for l in range(4):
            assert abs((Y[l * l:(l + 1) ** 2] ** 2).sum() - (2 * l + 1) / (4 * math.pi)) < 1e-14
        Ym = oracle.sh_basis(-v)  # parity (-1)^l
        for l in range(4):
            assert np.allclose(Ym[l * l:(l + 1) ** 2], (-1) ** l * Y[l * l:(l + 1) ** 2], atol=1e-15)
    # sign convention of the degree-1 band: (-y, z, -x) * sqrt(3/4pi)
    c1 = math.sqrt(3 / (4 * math.pi))
    assert np.allclose(oracle.sh_basis([0, 0, 1.0])[1:4], [0, c1, 0])
    assert np.allclose(oracle.sh_basis([1.0, 0, 0])[1:4], [0, 0, -c1])
    assert np.allclose(oracle.sh_basis([0, 1.0, 0])[1:4], [-c1, 0, 0])


def test_sh_basis_gradient_finite_differences(oracle):
    rng = np.random.default_rng(5)
    for _ in range(10):
        v = rng.standard_normal(3)
        G = oracle.sh_basis_grad(v)
        h = 1e-6
        for a in range(3):
            e = np.zeros(3); e[a] = h
            fd = (oracle.sh_basis(v + e) - oracle.sh_basis(v - e)) / (2 * h)
            assert np.abs(fd - G[:, a]).max() < 1e-8


def test_sh_degree0_is_constant_colour(oracle):
    g = golden()
    rng = np.random.default_rng(6)
    n = 64
    sc = SimpleNamespace(app=0, active_degree=0, base_color=rng.normal(0, 0.4, (n, 3)),
                         sh_rest=rng.normal(0, 1, (n, 15, 3)), features=None, mlp_weights=None)
    d = rng.standard_normal((n, 3)); d /= np.linalg.norm(d, axis=1, keepdims=True)
    col, res = oracle.appearance_forward(sc, d)
    assert np.array_equal(col, np.maximum(sc.base_color + g["activation_at_zero"], 0))
    assert np.all(res == 0)
    # c0 = phi^-1(c_sfm) reproduces the SfM colour (Sec. 3.1 initialisation)
    c_sfm = rng.uniform(0, 1, (n, 3))
    sc.base_color = c_sfm - 0.5
    sc.sh_rest = np.zeros((n, 15, 3)); sc.active_degree = 3
    col, _ = oracle.appearance_forward(sc, d)
    assert np.allclose(col, c_sfm, atol=1e-15)


def test_sh_colour_matches_eq1_with_explicit_y0(oracle):
    """Eq. 1 with a separate DC coefficient equals the folded interface of Eq. 2."""
    rng = np.random.default_rng(7)
    n = 32
    dc = rng.normal(0.5, 0.3, (n, 3)); rest = rng.normal(0, 0.3, (n, 15, 3))
    d = rng.standard_normal((n, 3)); d /= np.linalg.norm(d, axis=1, keepdims=True)
    Y0 = 1 / math.sqrt(4 * math.pi)
    sc = SimpleNamespace(app=0, active_degree=2, base_color=Y0 * dc, sh_rest=rest, features=None, mlp_weights=None)
    col, _ = oracle.appearance_forward(sc, d)
    for i in range(n):
        Y = oracle.sh_basis(d[i])
        ref = 0.5 + Y0 * dc[i] + sum(Y[k] * rest[i, k - 1] for k in range(1, 9))  # bands 1..2 only
        assert np.allclose(col[i], np.maximum(ref, 0), atol=1e-14)


# ------------------------------------------------------------------------------ neural decoder

def _neural_scene(rng, n, weights=None, feats=None, base=None, deg=3):
    w = rng.uniform(-0.5, 0.5, 816) if weights is None else weights
    return SimpleNamespace(app=1, active_degree=deg,
                           base_color=rng.normal(0, 0.2, (n, 3)) if base is None else base,
                           features=rng.normal(0, 0.5, (n, 8)) if feats is None else feats,
                           mlp_weights=w, sh_rest=None)


def _dirs(rng, n):
    d = rng.standard_normal((n, 3))
    return d / np.linalg.norm(d, axis=1, keepdims=True)


def test_mlp_zero_output_layer_gives_zero_residual(oracle):
    rng = np.random.default_rng(8)
    w = rng.uniform(-1, 1, 816); w[512 + 256:] = 0
    sc = _neural_scene(rng, 40, weights=w)
    col, res = oracle.appearance_forward(sc, _dirs(rng, 40))
    assert np.all(res == 0)
    assert np.array_equal(col, np.maximum(sc.base_color + 0.5, 0))


def test_mlp_residual_is_bounded_and_disabled_at_degree0(oracle):
    rng = np.random.default_rng(9)
    sc = _neural_scene(rng, 200, weights=rng.uniform(-1, 1, 816))
    d = _dirs(rng, 200)
    _, res = oracle.appearance_forward(sc, d)
    assert np.all(np.abs(res) < 1) and np.abs(res).max() > 0.5
    sc_big = _neural_scene(rng, 200, weights=rng.uniform(-30, 30, 816))
    assert np.all(np.abs(oracle.appearance_forward(sc_big, d)[1]) <= 1)
    _, res0 = oracle.appearance_forward(sc, d, deg=0)
    assert np.all(res0 == 0)


def test_mlp_one_hot_routes(oracle):
    """Hand-set weights that route one input to one output give tanh(w * input)."""
    rng = np.random.default_rng(10)
    n = 16
    d = _dirs(rng, n); f = rng.normal(0, 1, (n, 8))
    Y0 = 1 / math.sqrt(4 * math.pi)
    def run(inp, out, gain, deg=3, feats=f):
        w = np.zeros(816)
        w[0 * 32 + inp] = 1.0          # W1 row 0 picks input `inp`
        w[512 + 5 * 16 + 0] = 1.0      # W2 row 5 picks h1[0]
        w[768 + out * 16 + 5] = gain   # W3 row `out` picks h2[5]
        sc = _neural_scene(rng, n, weights=w, feats=feats, base=np.zeros((n, 3)), deg=deg)
        return oracle.appearance_forward(sc, d)[1]
    res = run(0, 1, 2.5)               # the constant degree-0 input acts as the bias
    assert np.allclose(res[:, 1], math.tanh(2.5 * Y0), atol=1e-15) and np.all(res[:, [0, 2]] == 0)
    res = run(16 + 2 * 3, 2, 1.7)      # sin f_3 (ReLU keeps the positive part)
    assert np.allclose(res[:, 2], np.tanh(1.7 * np.maximum(np.sin(f[:, 3]), 0)), atol=1e-15)
    res = run(17 + 2 * 6, 0, -0.8)     # cos f_6
    assert np.allclose(res[:, 0], np.tanh(-0.8 * np.maximum(np.cos(f[:, 6]), 0)), atol=1e-15)
    res = run(17, 0, 1.0, feats=np.zeros((n, 8)))   # f = 0 encodes to (sin, cos) = (0, 1)
    assert np.allclose(res[:, 0], math.tanh(1.0), atol=1e-15)
    res = run(16, 0, 1.0, feats=np.zeros((n, 8)))
    assert np.all(res == 0)
    c1 = math.sqrt(3 / (4 * math.pi))
    res = run(2, 0, 1.0)               # Y_1^0 = c1 * z
    assert np.allclose(res[:, 0], np.tanh(np.maximum(c1 * d[:, 2], 0)), atol=1e-15)
    res = run(9, 0, 1.0, deg=2)        # a degree-3 input is inactive at degree 2
    assert np.all(res == 0)


def test_mlp_matches_numpy_matmul(oracle):
    rng = np.random.default_rng(11)
    n = 50
    sc = _neural_scene(rng, n)
    d = _dirs(rng, n)
    col, _ = oracle.appearance_forward(sc, d, deg=2)
    W1 = sc.mlp_weights[:512].reshape(16, 32); W2 = sc.mlp_weights[512:768].reshape(16, 16)
    W3 = sc.mlp_weights[768:].reshape(3, 16)
    Y = np.stack([oracle.sh_basis(v) for v in d]); Y[:, 9:] = 0
    enc = np.stack([np.sin(sc.features), np.cos(sc.features)], -1).reshape(n, 16)
    x = np.concatenate([Y, enc], 1)
    out = np.tanh(np.maximum(np.maximum(x @ W1.T, 0) @ W2.T, 0) @ W3.T)
    assert np.allclose(col, np.maximum(sc.base_color + 0.5 + out, 0), atol=1e-14)


def test_inactive_inputs_get_zero_weight_gradient(oracle):
    rng = np.random.default_rng(12)
    n = 64
    sc = _neural_scene(rng, n, deg=1)
    g = oracle.appearance_backward(sc, _dirs(rng, n), rng.standard_normal((n, 3)))
    dW1 = g.mlp_weights[:512].reshape(16, 32)
    assert np.all(dW1[:, 4:16] == 0)            # degrees 2 and 3 inactive at degree 1
    assert np.abs(dW1[:, :4]).max() > 0 and np.abs(dW1[:, 16:]).max() > 0


# ------------------------------------------------------------------------------ footprint + blend

def test_single_gaussian_footprint_and_colour(oracle):
    cam = scenes.identity_camera(64, 64, 64.0, background=(0.1, 0.2, 0.3))
    s, z, logit = 0.2, 3.0, 1.5
    base = np.array([0.3, -0.1, 0.2])
    sc = one_gaussian_scene([0.05, -0.03, z], math.log(s), logit, base)
    fwd, _ = oracle.render(sc, cam)
    o = 1 / (1 + math.exp(-logit))
    u, v = 64 * 0.05 / z + 32, 64 * -0.03 / z + 32
    jj = np.array([[1 + (0.05 / z) ** 2, 0.05 * -0.03 / z ** 2], [0.05 * -0.03 / z ** 2, 1 + (0.03 / z) ** 2]])
    cov = (s * 64 / z) ** 2 * jj + 0.3 * np.eye(2)
    Q = np.linalg.inv(cov)
    ii, jj_ = np.meshgrid(np.arange(64) + 0.5, np.arange(64) + 0.5)
    dx, dy = ii - u, jj_ - v
    alpha = o * np.exp(-0.5 * (Q[0, 0] * dx * dx + 2 * Q[0, 1] * dx * dy + Q[1, 1] * dy * dy))
    alpha = np.where(alpha >= 1 / 255, np.minimum(alpha, 0.99), 0.0)
    c = np.maximum(base + 0.5, 0)
    ref = c[:, None, None] * alpha + (1 - alpha) * np.array(cam.background)[:, None, None]
    assert np.abs(fwd.image - ref).max() < 1e-13
    assert np.abs(fwd.final_T - (1 - alpha)).max() < 1e-13
    # mass of the truncated Gaussian: sum_p alpha(p) ~ 2 pi sqrt(det cov) (o - 1/255)
    mass = 2 * math.pi * math.sqrt(np.linalg.det(cov)) * (o - 1 / 255)
    assert abs(alpha.sum() - mass) / mass < 2e-3
    assert abs((1 - fwd.final_T).sum() - mass) / mass < 2e-3


def _two_gaussians(cam, z1, z2, o1=0.7, o2=0.6):
    lg = lambda o: math.log(o / (1 - o))
    return SimpleNamespace(
        means=np.array([[0.0, 0, z1], [0.0, 0, z2]]), log_scales=np.full((2, 3), math.log(0.5)),
        quats=np.array([[1.0, 0, 0, 0]] * 2), opacity_logits=np.array([lg(o1), lg(o2)]),
        base_color=np.array([[0.4, 0.0, -0.2], [-0.3, 0.3, 0.1]]), app=0, active_degree=0,
        sh_rest=np.zeros((2, 15, 3)), features=None, mlp_weights=None)


def test_two_gaussian_closed_form_and_depth_swap(oracle):
    cam = scenes.identity_camera(16, 16, 16.0)
    cam.cx = cam.cy = 8.5      # pixel (8, 8) centre sits exactly on the optical axis
    for z1, z2 in ((2.0, 3.0), (3.0, 2.0)):
        sc = _two_gaussians(cam, z1, z2)
        fwd, _ = oracle.render(sc, cam)
        c = np.maximum(sc.base_color + 0.5, 0)
        front, back = (0, 1) if z1 < z2 else (1, 0)
        a = {0: 0.7, 1: 0.6}
        ref = c[front] * a[front] + c[back] * a[back] * (1 - a[front])
        assert np.allclose(fwd.image[:, 8, 8], ref, atol=1e-14)
        assert abs(fwd.final_T[8, 8] - (1 - 0.7) * (1 - 0.6)) < 1e-15
        assert fwd.n_contrib[8, 8] == 2


def test_alpha_clamp_and_early_stop(oracle):
    cam = scenes.identity_camera(16, 16, 16.0)
    cam.cx = cam.cy = 8.5
    sc = _two_gaussians(cam, 2.0, 3.0, o1=0.9999, o2=0.9999)
    # a third opaque Gaussian behind the two: T would fall to ~1e-6 < 1e-4, so it is cut
    for k in ("means", "log_scales", "quats", "base_color"):
        setattr(sc, k, np.concatenate([getattr(sc, k), getattr(sc, k)[1:2]], 0))
    sc.means[2, 2] = 4.0
    sc.base_color[2] = [0.5, 0.5, 0.5]
    sc.opacity_logits = np.append(sc.opacity_logits, sc.opacity_logits[1])
    sc.sh_rest = np.zeros((3, 15, 3))
    fwd, _ = oracle.render(sc, cam)
    c = np.maximum(sc.base_color + 0.5, 0)
    # both are clamped to alpha = 0.99: the second contributes 0.99 * 0.01 (<= 1 %)
    assert np.allclose(fwd.image[:, 8, 8], 0.99 * c[0] + 0.99 * 0.01 * c[1], atol=1e-15)
    assert fwd.n_contrib[8, 8] == 2 and abs(fwd.final_T[8, 8] - 1e-4) < 1e-15


def _min_quadratic_over_box(A, B, C, x0, x1, y0, y1):
    """min of A x^2 + 2 B x y + C y^2 over the box [x0,x1] x [y0,y1] (coordinates relative to the
    centre), by the textbook case split: the origin if inside, else the best of the four edges."""
    if x0 <= 0 <= x1 and y0 <= 0 <= y1:
        return 0.0
    best = math.inf
    for y in (y0, y1):                      # horizontal edges: minimise over x, clamp
        x = min(max(-B * y / A, x0), x1)
        best = min(best, A * x * x + 2 * B * x * y + C * y * y)
    for x in (x0, x1):                      # vertical edges
        y = min(max(-B * x / C, y0), y1)
        best = min(best, A * x * x + 2 * B * x * y + C * y * y)
    return best


def _instances_by_definition(fwd, cam, slack):
    """(tile, depth_bits, index) for every tile whose box of pixel centres the alpha >= 1/255 ellipse
    (conic form <= tau (1 + slack)) meets, straight from that definition."""
    gx, gy = (cam.width + 15) // 16, (cam.height + 15) // 16
    pre = fwd.pre
    out = []
    for g in np.nonzero(pre.valid)[0]:
        A, B, C = pre.conic[g]
        u, v = pre.mean2d[g]
        tau = 2 * math.log(255 * pre.opacity[g]) * (1 + slack)
        for ty in range(gy):
            for tx in range(gx):
                x0, x1 = 16 * tx + 0.5 - u, min(16 * tx + 15.5, cam.width - 0.5) - u
                y0, y1 = 16 * ty + 0.5 - v, min(16 * ty + 15.5, cam.height - 0.5) - v
                if _min_quadratic_over_box(A, B, C, x0, x1, y0, y1) <= tau:
                    out.append((ty * gx + tx, int(pre.depth_bits[g]), int(g)))
    return sorted(out)


def test_tiles_sort_and_ranges_by_brute_force(oracle):
    w = scenes.config1(400)
    cam = w.cameras[0]
    fwd, _ = oracle.render(w.scene, cam)
    got = [(int(k >> np.uint64(32)), int(k & np.uint64(0xFFFFFFFF)), int(v)) for k, v in zip(fwd.keys, fwd.vals)]
    assert fwd.P == len(got) and got == sorted(got)
    # lower bound: every tile that holds a pixel centre inside the ellipse (those are the pairs that
    # can blend); upper bound: every tile whose box of pixel centres the ellipse, padded by 5e-5 in
    # tau, meets at all (the span rule may drop a tile the ellipse only grazes between pixel centres)
    pre, gx = fwd.pre, (cam.width + 15) // 16
    ii, jj = np.meshgrid(np.arange(cam.width) + 0.5, np.arange(cam.height) + 0.5)
    must = set()
    for g in np.nonzero(pre.valid)[0]:
        dx, dy = ii - pre.mean2d[g, 0], jj - pre.mean2d[g, 1]
        A, B, C = pre.conic[g]
        ys, xs = np.nonzero(A * dx * dx + 2 * B * dx * dy + C * dy * dy <= 2 * math.log(255 * pre.opacity[g]))
        must |= {((y // 16) * gx + x // 16, int(pre.depth_bits[g]), int(g)) for y, x in zip(ys.tolist(), xs.tolist())}
    may = set(_instances_by_definition(fwd, cam, 5e-5))
    assert len(must) > 500 and must <= set(got) <= may
    assert len(may) - len(got) <= 0.02 * len(got)       # ... and it drops few of those
    assert len(got) < 0.99 * int(((fwd.rect[:, 2] - fwd.rect[:, 0]) * (fwd.rect[:, 3] - fwd.rect[:, 1])).sum())
    # ranges partition [0, P) and every instance lies inside its tile's range
    tiles = np.array([t for t, _, _ in got])
    for t in range(fwd.ranges.shape[0]):
        s, e = fwd.ranges[t]
        assert np.all(tiles[s:e] == t)
        assert e - s == (tiles == t).sum()
    assert fwd.ranges[:, 1].astype(np.int64).sum() - fwd.ranges[:, 0].astype(np.int64).sum() == fwd.P


def test_coverage_invariant_and_tiled_equals_brute(oracle):
    """Every (pixel, Gaussian) pair with alpha >= 1/255 is inside that pixel's tile list, and
    the tiled image equals the no-tiles definition bit for bit."""
    w = scenes.config1(300)
    cam = w.cameras[0]
    fwd, _ = oracle.render(w.scene, cam)
    pre = fwd.pre
    gx = (cam.width + 15) // 16
    lists = [set(fwd.vals[s:e].tolist()) for s, e in fwd.ranges]
    ii, jj = np.meshgrid(np.arange(cam.width) + 0.5, np.arange(cam.height) + 0.5)
    checked = 0
    for g in np.nonzero(pre.valid)[0]:
        dx, dy = ii - pre.mean2d[g, 0], jj - pre.mean2d[g, 1]
        A, B, Cc = pre.conic[g]
        alpha = pre.opacity[g] * np.exp(-0.5 * (A * dx * dx + Cc * dy * dy) - B * dx * dy)
        ys, xs = np.nonzero(alpha >= 1 / 255)
        for y, x in zip(ys, xs):
            assert g in lists[(y // 16) * gx + x // 16]
            checked += 1
    assert checked > 1000
    img, T = oracle.blend_brute(cam, pre.visible, pre.depth_bits, pre.mean2d, pre.conic, pre.opacity, fwd.color)
    assert np.array_equal(img, fwd.image) and np.array_equal(T, fwd.final_T)


def test_blend_invariants(oracle):
    w = scenes.config1()
    cam = w.cameras[0]
    fwd, _ = oracle.render(w.scene, cam)
    assert np.all(fwd.final_T >= 1e-4 * 0.999) and np.all(fwd.final_T <= 1)
    assert np.all(1 - fwd.final_T >= 0) and np.all(1 - fwd.final_T <= 1)
    lens = (fwd.ranges[:, 1] - fwd.ranges[:, 0]).reshape(4, 4)
    assert np.all(fwd.n_contrib <= np.kron(lens, np.ones((16, 16), np.uint32)))
    # transmittance is monotone: dropping the far half of every list can only raise final_T
    half = fwd.ranges.copy(); half[:, 1] = fwd.ranges[:, 0] + (fwd.ranges[:, 1] - fwd.ranges[:, 0]) // 2
    part = oracle.blend_forward(cam, fwd.vals, half, fwd.pre.mean2d, fwd.pre.conic, fwd.pre.opacity, fwd.color)
    assert np.all(part.final_T >= fwd.final_T)
    # colours are >= 0 and the weights sum to 1 - T: image <= max colour * (1 - T)
    assert np.all(fwd.image <= fwd.color.max() * (1 - fwd.final_T)[None] + 1e-12)


def test_integer_stage_f32_agrees_with_double(oracle):
    w = scenes.config1()
    cam = w.cameras[0]
    fwd, _ = oracle.render(w.scene, cam)
    pre = fwd.pre
    f32 = lambda a: a.astype(np.float32)
    rect, tt, P = oracle.tile_spans_f32(pre.valid, f32(pre.mean2d), f32(pre.chol), f32(pre.ext), cam.width, cam.height)
    assert (tt != fwd.tiles_touched).sum() <= 3      # fp32 rounding may flip a tile at a box edge, rarely
    assert abs(P - fwd.P) <= 6
    keys, vals, ranges = oracle.sorted_instances_f32(rect, tt, f32(pre.mean2d), f32(pre.chol), f32(pre.ext),
                                                     pre.depth_bits, cam.width, cam.height, P)
    assert len(vals) == P and np.all(np.diff(keys.astype(np.int64) >> 32) >= 0)


def test_oracle_output_has_not_drifted(oracle):
    """The oracle's summary numbers on small seeded scenes equal the stored ones (written by
    tests/golden/make_oracle_regression.py from the oracle alone): its arithmetic is changed on purpose or not
    at all."""
    import importlib.util
    here = os.path.dirname(__file__)
    spec = importlib.util.spec_from_file_location("make_oracle_regression", os.path.join(here, "golden", "make_oracle_regression.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = {}
    for line in open(os.path.join(here, "golden", "oracle_regression.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split("=")
            stored[k.strip()] = float(v)
    now = mod.summary()
    assert set(now) == set(stored)
    for k, v in now.items():
        assert abs(v - stored[k]) <= 1e-9 * max(1.0, abs(stored[k])), k
