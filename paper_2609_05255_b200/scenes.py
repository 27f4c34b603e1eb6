"""Seeded synthetic scenes and cameras.

This module only draws random inputs (numpy ``default_rng(PCG64(seed))``) with the
shapes and value distributions of the paper's workloads.  It contains none of the
method's arithmetic and is the one module that both the CUDA path's tests/bench and
the CPU oracle's tests may import.

All float arrays are float32, fp16 arrays are float32 draws rounded to nearest-even.
Camera frame: +x right, +y down, +z forward.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

APP_SH = 0
APP_NEURAL = 1
APP_SV = 2          # Spherical Voronoi (Eq. 3)
SV_SITES = 7

# Layer sizes of the shared decoder (Sec. 4, "two hidden layers of 16 neurons, three
# outputs", 32 inputs): 32*16 + 16*16 + 16*3 = 816 weights, no biases.
MLP_IN, MLP_HIDDEN, MLP_OUT, NUM_FEATURES = 32, 16, 3, 8
MLP_NUM_WEIGHTS = MLP_IN * MLP_HIDDEN + MLP_HIDDEN * MLP_HIDDEN + MLP_HIDDEN * MLP_OUT

# 1/sqrt(4 pi): the generator draws a "DC" coefficient and stores base_color = Y0 * DC,
# i.e. the paper's interface with the constant folded into the base colour (Eq. 2).
_Y0 = 0.5 / math.sqrt(math.pi)


@dataclass
class Camera:
    width: int
    height: int
    fx: float
    fy: float
    cx: float
    cy: float
    w2c: np.ndarray  # [3,4] float32 row-major [R|t], x_cam = R x_world + t
    near_plane: float = 0.2
    far_plane: float = 1.0e10
    background: tuple = (0.0, 0.0, 0.0)


@dataclass
class Scene:
    means: np.ndarray           # [n,3] f32
    log_scales: np.ndarray      # [n,3] f32
    quats: np.ndarray           # [n,4] f32 (w,x,y,z), not normalised by the caller
    opacity_logits: np.ndarray  # [n]   f32
    base_color: np.ndarray      # [n,3] f32
    app: int = APP_SH
    active_degree: int = 3
    sh_rest: Optional[np.ndarray] = None      # [n,15,3] f32
    features: Optional[np.ndarray] = None     # [n,8]  f16
    mlp_weights: Optional[np.ndarray] = None  # [816]  f16: W1[16][32], W2[16][16], W3[3][16]
    color_activation: int = 0                 # 0 ReLU(x+0.5), 1 softplus(x+0.5) beta 10, 2 sigmoid(4x), 3 clamp(x+0.5,0,1)
    sv_sites: Optional[np.ndarray] = None     # [n,7,7] f32: per site (a_r, a_g, a_b, s_x, s_y, s_z, log tau)
    mlp_hidden: int = 0                       # decoder variant: neurons per hidden layer (0 = the default 16)
    mlp_layers: int = 0                       # decoder variant: hidden layers (0 = the default 2)
    separate_pass: int = 0                    # 1: ask the library for its unfused reference path (same results)
    decoder_precision: int = 0                # 1: the decoder's products on plain fp16 operands (the paper's precision)

    @property
    def n(self) -> int:
        return int(self.means.shape[0])


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def identity_camera(width: int, height: int, focal: float, **kw) -> Camera:
    w2c = np.zeros((3, 4), np.float32)
    w2c[:, :3] = np.eye(3, dtype=np.float32)
    return Camera(width, height, float(focal), float(focal), width / 2.0, height / 2.0, w2c, **kw)


def orbit_camera(width: int, height: int, theta: float, radius: float = 5.0,
                 fov_half_deg: float = 30.0, **kw) -> Camera:
    """Camera on the circle (r cos t, 0, r sin t) looking at the origin, +y down."""
    eye = np.array([radius * math.cos(theta), 0.0, radius * math.sin(theta)], np.float64)
    f = -eye / np.linalg.norm(eye)
    r = np.cross(f, np.array([0.0, -1.0, 0.0]))
    r /= np.linalg.norm(r)
    down = np.cross(f, r)
    R = np.stack([r, down, f], 0)
    t = -R @ eye
    w2c = np.concatenate([R, t[:, None]], 1).astype(np.float32)
    focal = (width / 2.0) / math.tan(math.radians(fov_half_deg))
    return Camera(width, height, float(np.float32(focal)), float(np.float32(focal)),
                  width / 2.0, height / 2.0, w2c, **kw)


def orbit_cameras(width: int, height: int, count: int, radius: float = 5.0) -> List[Camera]:
    return [orbit_camera(width, height, 2.0 * math.pi * k / count, radius) for k in range(count)]


def _random_quats(rng, n):
    return _f32(rng.standard_normal((n, 4)))


def draw_sh_appearance(rng, n):
    dc = rng.normal(0.5, 0.1, (n, 3))
    base_color = _f32(_Y0 * dc)
    sh_rest = _f32(rng.normal(0.0, 0.05, (n, 15, 3)))
    return base_color, sh_rest


def draw_neural_appearance(rng, n, hidden: int = MLP_HIDDEN, layers: int = 2, num_features: int = NUM_FEATURES):
    """Features and Xavier-uniform weights of a decoder with `layers` hidden layers of `hidden` neurons;
    num_features = 8 (frequency encoded) or 16 (raw).  The defaults are the paper's decoder."""
    dc = rng.normal(0.5, 0.1, (n, 3))
    base_color = _f32(_Y0 * dc)
    features = _f32(rng.normal(0.0, 0.1, (n, num_features))).astype(np.float16)
    weights = []
    shapes = [(hidden, MLP_IN)] + [(hidden, hidden)] * (layers - 1) + [(MLP_OUT, hidden)]
    for fan_out, fan_in in shapes:
        bound = math.sqrt(6.0 / (fan_in + fan_out))
        weights.append(rng.uniform(-bound, bound, (fan_out, fan_in)).reshape(-1))
    mlp_weights = _f32(np.concatenate(weights)).astype(np.float16)
    return base_color, features, mlp_weights


def fibonacci_sites(count: int) -> np.ndarray:
    """`count` directions spread over the sphere on a Fibonacci lattice."""
    k = np.arange(count) + 0.5
    z = 1.0 - 2.0 * k / count
    phi = math.pi * (1.0 + math.sqrt(5.0)) * k
    r = np.sqrt(1.0 - z * z)
    return np.stack([r * np.cos(phi), r * np.sin(phi), z], 1)


def draw_sv_appearance(rng, n):
    """Spherical Voronoi: 7 sites per Gaussian, each (colour a [3], unnormalised direction s [3], log-temperature t).
    Sites start on a shared Fibonacci lattice (as the paper initialises them) and are perturbed and rescaled so
    that normalisation, temperatures and colours all matter."""
    dc = rng.normal(0.5, 0.1, (n, 3))
    base_color = _f32(_Y0 * dc)
    sites = np.empty((n, SV_SITES, 7))
    sites[:, :, 0:3] = rng.normal(0.0, 0.15, (n, SV_SITES, 3))
    lattice = fibonacci_sites(SV_SITES)[None] + rng.normal(0.0, 0.25, (n, SV_SITES, 3))
    sites[:, :, 3:6] = lattice * rng.uniform(0.5, 2.0, (n, SV_SITES, 1))
    sites[:, :, 6] = rng.normal(0.5, 0.5, (n, SV_SITES))
    return base_color, _f32(sites)


def _attach_appearance(rng, n, app, geom) -> Scene:
    if app == APP_SH:
        base_color, sh_rest = draw_sh_appearance(rng, n)
        return Scene(*geom, base_color=base_color, app=APP_SH, active_degree=3, sh_rest=sh_rest)
    if app == APP_SV:
        base_color, sites = draw_sv_appearance(rng, n)
        return Scene(*geom, base_color=base_color, app=APP_SV, active_degree=3, sv_sites=sites)
    base_color, features, weights = draw_neural_appearance(rng, n)
    return Scene(*geom, base_color=base_color, app=APP_NEURAL, active_degree=3,
                 features=features, mlp_weights=weights)


def box_scene(n: int, half_xy: float, z_lo: float, z_hi: float, log_scale_mean: float,
              log_scale_std: float, logit_std: float, app: int, seed: int) -> Scene:
    """Uniform box in front of an identity camera (configs 1 and 2)."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    means = np.empty((n, 3))
    means[:, 0:2] = rng.uniform(-half_xy, half_xy, (n, 2))
    means[:, 2] = rng.uniform(z_lo, z_hi, n)
    log_scales = rng.normal(log_scale_mean, log_scale_std, (n, 3))
    quats = _random_quats(rng, n)
    logits = rng.normal(0.0, logit_std, n)
    geom = (_f32(means), _f32(log_scales), quats, _f32(logits))
    return _attach_appearance(rng, n, app, geom)


def _random_rotations(rng, k):
    q = rng.standard_normal((k, 4))
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    w, x, y, z = q.T
    R = np.empty((k, 3, 3))
    R[:, 0, 0] = 1 - 2 * (y * y + z * z); R[:, 0, 1] = 2 * (x * y - w * z); R[:, 0, 2] = 2 * (x * z + w * y)
    R[:, 1, 0] = 2 * (x * y + w * z); R[:, 1, 1] = 1 - 2 * (x * x + z * z); R[:, 1, 2] = 2 * (y * z - w * x)
    R[:, 2, 0] = 2 * (x * z - w * y); R[:, 2, 1] = 2 * (y * z + w * x); R[:, 2, 2] = 1 - 2 * (x * x + y * y)
    return R


def clustered_scene(n: int, clusters: int, log_scale_mean: float, log_scale_std: float,
                    app: int, seed: int, deep: bool = False, logit_std: float = 1.5,
                    shell_fraction: float = 0.1, shell_radius: float = 20.0) -> Scene:
    """90 % anisotropic clusters + 10 % background shell (configs 3 and 4).

    ``deep=False``: cluster centres uniform in a ball of radius 2 (config 3).
    ``deep=True``: centres = uniform direction x radius log-uniform in [0.5, 45] (config 4).
    """
    rng = np.random.default_rng(np.random.PCG64(seed))
    n_shell = int(round(shell_fraction * n))
    n_cl = n - n_shell
    dirs = rng.standard_normal((clusters, 3))
    dirs /= np.linalg.norm(dirs, axis=1, keepdims=True)
    if deep:
        rad = np.exp(rng.uniform(math.log(0.5), math.log(45.0), clusters))
    else:
        rad = 2.0 * rng.uniform(0.0, 1.0, clusters) ** (1.0 / 3.0)
    centres = dirs * rad[:, None]
    rot = _random_rotations(rng, clusters)
    sig = 0.3 * np.exp(rng.normal(0.0, 0.5, (clusters, 3)))
    member = rng.integers(0, clusters, n_cl)
    local = rng.standard_normal((n_cl, 3)) * sig[member]
    pts = centres[member] + np.einsum("nij,nj->ni", rot[member], local)
    sh = rng.standard_normal((n_shell, 3))
    sh *= shell_radius / np.linalg.norm(sh, axis=1, keepdims=True)
    means = np.concatenate([pts, sh], 0)
    perm = rng.permutation(n)  # no spatial order in memory, like a densified scene
    means = means[perm]
    log_scales = rng.normal(log_scale_mean, log_scale_std, (n, 3))
    quats = _random_quats(rng, n)
    logits = rng.normal(0.0, logit_std, n)
    geom = (_f32(means), _f32(log_scales), quats, _f32(logits))
    return _attach_appearance(rng, n, app, geom)


def upstream_gradient(cam: Camera, seed: int) -> np.ndarray:
    """dL/dimage ~ N(0,1), [3,H,W] f32."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    return _f32(rng.standard_normal((3, cam.height, cam.width)))


def unit_directions(n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(np.random.PCG64(seed))
    d = rng.standard_normal((n, 3))
    d /= np.linalg.norm(d, axis=1, keepdims=True)
    return _f32(d)


def color_gradient(n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(np.random.PCG64(seed))
    return _f32(rng.standard_normal((n, 3)))


# ---------------------------------------------------------------------------------------
# The five benchmark configurations (seed = 1000 + config number).
# ---------------------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    scene: Scene
    cameras: List[Camera] = field(default_factory=list)


def config1(n: int = 1000) -> Workload:
    """Tiny SH scene, 64x64, identity camera."""
    scene = box_scene(n, 1.0, 2.0, 4.0, -3.0, 0.5, 1.0, APP_SH, seed=1001)
    return Workload("config1_tiny_sh", scene, [identity_camera(64, 64, 64.0)])


def config2(n: int = 100_000, app: int = APP_NEURAL) -> Workload:
    """Neural appearance, 100k Gaussians, 512x512, identity camera."""
    scene = box_scene(n, 3.0, 2.0, 8.0, -3.0, 0.5, 1.0, app, seed=1002)
    return Workload("config2_neural_100k", scene, [identity_camera(512, 512, 512.0)])


def config3(app: int, n: int = 1_000_000, width: int = 1256, height: int = 828,
            views: int = 8) -> Workload:
    """1M Gaussians in 64 clusters + shell, 8 orbit cameras."""
    scene = clustered_scene(n, 64, -4.0, 0.7, app, seed=1003)
    tag = {APP_SH: "sh", APP_SV: "sv"}.get(app, "neural")
    return Workload(f"config3_1M_{tag}", scene, orbit_cameras(width, height, views))


def config4(n: int = 3_000_000, width: int = 1920, height: int = 1080, views: int = 16) -> Workload:
    """3M Gaussians, 256 clusters with depth range 1-50, neural appearance, 16 orbit cameras."""
    scene = clustered_scene(n, 256, -4.5, 0.8, APP_NEURAL, seed=1004, deep=True)
    return Workload("config4_3M_neural", scene, orbit_cameras(width, height, views))


def decoder_variant(n: int, hidden: int, layers: int, num_features: int, seed: int = 1006):
    """Appearance-sweep inputs for a decoder variant of the paper's architecture table."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    geom = (np.zeros((n, 3), np.float32), np.zeros((n, 3), np.float32),
            np.zeros((n, 4), np.float32), np.zeros((n,), np.float32))
    base_color, features, weights = draw_neural_appearance(rng, n, hidden, layers, num_features)
    scene = Scene(*geom, base_color=base_color, app=APP_NEURAL, active_degree=3, features=features,
                  mlp_weights=weights, mlp_hidden=hidden, mlp_layers=layers)
    return scene, unit_directions(n, 2006), color_gradient(n, 3006)


def config5(n: int, app: int):
    """Appearance-stage sweep inputs: scene appearance parameters, unit directions, dL/dcolor."""
    rng = np.random.default_rng(np.random.PCG64(1005))
    geom = (np.zeros((n, 3), np.float32), np.zeros((n, 3), np.float32),
            np.zeros((n, 4), np.float32), np.zeros((n,), np.float32))
    scene = _attach_appearance(rng, n, app, geom)
    return scene, unit_directions(n, 2005), color_gradient(n, 3005)
