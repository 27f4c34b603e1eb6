"""ctypes front end of the CPU oracle (``gs_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's
``cpu_baseline`` / ``--impl reference`` legs.  The product path never imports it, and this
module imports nothing from the CUDA package.

Scenes and cameras are duck-typed: any object with the attributes ``means, log_scales, quats,
opacity_logits, base_color, app, active_degree, sh_rest | features + mlp_weights`` and
``width, height, fx, fy, cx, cy, w2c, near_plane, far_plane, background``.  All floating-point
inputs are widened to float64 exactly (fp16 and fp32 are subsets of fp64).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gs_oracle.cpp")
_LIB = os.path.join(_HERE, "libgs_oracle.so")
_lib = None

TILE = 16


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no FMA contraction, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.gso_num_mlp_weights.restype = C.c_int
        _lib.gso_mlp_macs.restype = C.c_int
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops use (all host cores unless OMP_NUM_THREADS says otherwise)."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _dp(a):
    return _p(a, C.c_double)


def cam_array(cam) -> np.ndarray:
    c = np.zeros(23, np.float64)
    c[0], c[1] = cam.width, cam.height
    c[2:6] = cam.fx, cam.fy, cam.cx, cam.cy
    c[6:18] = np.asarray(cam.w2c, np.float64).reshape(12)
    c[18], c[19] = cam.near_plane, cam.far_plane
    c[20:23] = cam.background
    return c


# ------------------------------------------------------------------------------------------
# thin wrappers, one per exported function
# ------------------------------------------------------------------------------------------

def sh_basis(d):
    d = _f64(d); Y = np.zeros(16)
    lib().gso_sh_basis(_dp(d), _dp(Y))
    return Y


def sh_basis_grad(d):
    d = _f64(d); G = np.zeros((16, 3))
    lib().gso_sh_basis_grad(_dp(d), _dp(G))
    return G


def quat_to_rot(q):
    q = _f64(q); R = np.zeros((3, 3))
    lib().gso_quat_to_rot(_dp(q), _dp(R))
    return R


def mlp_macs(fold: bool) -> int:
    return lib().gso_mlp_macs(int(fold))


def num_mlp_weights() -> int:
    return lib().gso_num_mlp_weights()


def decoder_arch(scene):
    """(hidden, layers, nfeat) of a scene's decoder; the default is the paper's 16 / 2 / 8."""
    return (int(getattr(scene, "mlp_hidden", 0) or 16), int(getattr(scene, "mlp_layers", 0) or 2),
            int(scene.features.shape[1]))


def decoder_num_weights(hidden: int, layers: int) -> int:
    return int(lib().gso_decoder_num_weights(C.c_int(hidden), C.c_int(layers)))


def decoder_macs(hidden: int, layers: int, fold: bool) -> int:
    return int(lib().gso_decoder_macs(C.c_int(hidden), C.c_int(layers), C.c_int(1 if fold else 0)))


def decoder_forward(scene, dirs, deg=None):
    """Colour of the neural model for any of the decoder architectures of the paper's architecture table."""
    hidden, layers, nfeat = decoder_arch(scene)
    dirs = _f64(dirs); n = dirs.shape[0]
    color = np.zeros((n, 3))
    lib().gso_decoder_forward(C.c_int64(n), C.c_int(hidden), C.c_int(layers), C.c_int(nfeat),
                              C.c_int(scene.active_degree if deg is None else deg), C.c_int(_act(scene)),
                              _dp(_f64(scene.base_color)), _dp(_f64(scene.features)), _dp(_f64(scene.mlp_weights)),
                              _dp(dirs), _dp(color))
    return color


def decoder_backward(scene, dirs, g_color, deg=None):
    hidden, layers, nfeat = decoder_arch(scene)
    dirs, g_color = _f64(dirs), _f64(g_color); n = dirs.shape[0]
    o = SimpleNamespace(base_color=np.zeros((n, 3)), features=np.zeros((n, nfeat)),
                        mlp_weights=np.zeros(decoder_num_weights(hidden, layers)), dirs=np.zeros((n, 3)))
    lib().gso_decoder_backward(C.c_int64(n), C.c_int(hidden), C.c_int(layers), C.c_int(nfeat),
                               C.c_int(scene.active_degree if deg is None else deg), C.c_int(_act(scene)),
                               _dp(_f64(scene.base_color)), _dp(_f64(scene.features)), _dp(_f64(scene.mlp_weights)),
                               _dp(dirs), _dp(g_color), _dp(o.base_color), _dp(o.features), _dp(o.mlp_weights), _dp(o.dirs))
    return o


ACT_RELU, ACT_SOFTPLUS, ACT_SIGMOID, ACT_HARD_SIGMOID = 0, 1, 2, 3


def _act(scene) -> int:
    return int(getattr(scene, "color_activation", 0))


def color_act(act: int, x: float) -> float:
    """phi(x), x = c0 + A(d) (Sec. 3.1): 0 ReLU(x + 0.5), 1 softplus(x + 0.5) with beta = 10, 2 sigmoid(4x),
    3 clamp(x + 0.5, 0, 1)."""
    f = lib().gso_color_act
    f.restype = C.c_double
    return float(f(C.c_int(act), C.c_double(x)))


def color_act_grad(act: int, x: float) -> float:
    f = lib().gso_color_act_grad
    f.restype = C.c_double
    return float(f(C.c_int(act), C.c_double(x)))


def neural_fold(scene):
    """Export step of the viewer (App. C.3): [n,16] pre-activations of the first layer from the features,
    the constant degree-0 input and their 17 weight columns, in double (not yet rounded to fp16)."""
    n = scene.means.shape[0]
    pre = np.zeros((n, 16))
    lib().gso_neural_fold(C.c_int64(n), _dp(_f64(scene.features)), _dp(_f64(scene.mlp_weights)), _dp(pre))
    return pre


def neural_prepass(scene, pre, eye, deg=None):
    """Per-frame colour of every Gaussian from the folded pre-activations and the camera position `eye`."""
    n = scene.means.shape[0]
    color = np.zeros((n, 3))
    lib().gso_neural_prepass(C.c_int64(n), C.c_int(scene.active_degree if deg is None else deg), C.c_int(_act(scene)),
                             _dp(_f64(scene.means)),
                             _dp(_f64(scene.base_color)), _dp(_f64(pre)), _dp(_f64(scene.mlp_weights)), _dp(_f64(eye)),
                             _dp(color))
    return color


def rgba8(color, opacity):
    """The prepass output texel: colour clamped to [0,1] and opacity, each to 8 bits, round to nearest."""
    c = np.clip(np.concatenate([np.asarray(color, np.float64), np.asarray(opacity, np.float64)[:, None]], 1), 0.0, 1.0)
    return np.floor(c * 255.0 + 0.5).astype(np.uint8)


def adam_step(param, grad, m, v, lr, beta1=0.9, beta2=0.999, eps=1e-15, step=1):
    """One Adam step with one learning rate per column (App. C.1).  param, grad, m, v: [rows, cols] (or
    [cols] for a single row); lr: [cols].  Returns new (param, m, v) as float64 arrays of the input shape."""
    shape = np.shape(param)
    lr = _f64(np.atleast_1d(lr))
    cols = lr.shape[0]
    p2, g2 = _f64(param).reshape(-1, cols).copy(), _f64(grad).reshape(-1, cols)
    m2, v2 = _f64(m).reshape(-1, cols).copy(), _f64(v).reshape(-1, cols).copy()
    lib().gso_adam_step(C.c_int64(p2.shape[0]), C.c_int(cols), _dp(p2), _dp(np.ascontiguousarray(g2)), _dp(m2), _dp(v2),
                        _dp(lr), C.c_double(beta1), C.c_double(beta2), C.c_double(eps), C.c_int64(step))
    return p2.reshape(shape), m2.reshape(shape), v2.reshape(shape)


def preprocess(means, log_scales, quats, opacity_logits, cam):
    means, log_scales, quats, logits = _f64(means), _f64(log_scales), _f64(quats), _f64(opacity_logits)
    n = means.shape[0]
    o = SimpleNamespace(
        mean2d=np.zeros((n, 2)), cov2d=np.zeros((n, 3)), conic=np.zeros((n, 3)), opacity=np.zeros(n),
        extent=np.zeros((n, 2)), depth32=np.zeros(n, np.float32), dir=np.zeros((n, 3)),
        valid=np.zeros(n, np.uint8), visible=np.zeros(n, np.uint8), rect_px=np.zeros((n, 4), np.int32))
    cam_a = cam_array(cam)
    lib().gso_preprocess(C.c_int64(n), _dp(means), _dp(log_scales), _dp(quats), _dp(logits), _dp(cam_a),
                         _dp(o.mean2d), _dp(o.cov2d), _dp(o.conic), _dp(o.opacity), _dp(o.extent),
                         _p(o.depth32, C.c_float), _dp(o.dir), _p(o.valid, C.c_uint8),
                         _p(o.visible, C.c_uint8), _p(o.rect_px, C.c_int32))
    o.depth_bits = o.depth32.view(np.uint32)
    return o


def _app_args(scene):
    sh = _f64(scene.sh_rest) if scene.app == 0 else (_f64(scene.sv_sites) if scene.app == 2 else None)
    ft = _f64(scene.features) if scene.app == 1 else None
    wt = _f64(scene.mlp_weights) if scene.app == 1 else None
    return _f64(scene.base_color), sh, ft, wt


def _is_variant(scene) -> bool:
    return scene.app == 1 and decoder_arch(scene) != (16, 2, 8)


def appearance_forward(scene, dirs, mask=None, deg=None):
    if _is_variant(scene):      # a decoder of another size: the generic decoder, masked rows left at zero
        keep = np.ones(len(dirs), bool) if mask is None else np.asarray(mask) > 0
        color = np.zeros((len(dirs), 3))
        color[keep] = decoder_forward(scene_rows(scene, keep), _f64(dirs)[keep], deg)
        return color, np.zeros((len(dirs), 3))
    base, sh, ft, wt = _app_args(scene)
    dirs = _f64(dirs); n = dirs.shape[0]
    color, resid = np.zeros((n, 3)), np.zeros((n, 3))
    deg = scene.active_degree if deg is None else deg
    m = None if mask is None else np.ascontiguousarray(mask, np.uint8)
    lib().gso_appearance_forward(C.c_int64(n), C.c_int(scene.app), C.c_int(deg), C.c_int(_act(scene)), _dp(base), _dp(sh),
                                 _dp(ft), _dp(wt), _dp(dirs), _p(m, C.c_uint8), _dp(color), _dp(resid))
    return color, resid


def scene_rows(scene, keep):
    """The appearance parameters of the Gaussians selected by the boolean array `keep` (decoder shared)."""
    return SimpleNamespace(app=scene.app, active_degree=scene.active_degree, base_color=np.asarray(scene.base_color)[keep],
                           features=np.asarray(scene.features)[keep], mlp_weights=scene.mlp_weights,
                           mlp_hidden=getattr(scene, "mlp_hidden", 0), mlp_layers=getattr(scene, "mlp_layers", 0),
                           color_activation=_act(scene))


def appearance_backward(scene, dirs, g_color, mask=None, deg=None):
    if _is_variant(scene):
        n = len(dirs)
        keep = np.ones(n, bool) if mask is None else np.asarray(mask) > 0
        g = decoder_backward(scene_rows(scene, keep), _f64(dirs)[keep], _f64(g_color)[keep], deg)
        nfeat = scene.features.shape[1]
        o = SimpleNamespace(base_color=np.zeros((n, 3)), dirs=np.zeros((n, 3)), sh_rest=None, sv_sites=None,
                            features=np.zeros((n, nfeat)), mlp_weights=g.mlp_weights)
        o.base_color[keep], o.dirs[keep], o.features[keep] = g.base_color, g.dirs, g.features
        return o
    base, sh, ft, wt = _app_args(scene)
    dirs, g_color = _f64(dirs), _f64(g_color); n = dirs.shape[0]
    deg = scene.active_degree if deg is None else deg
    m = None if mask is None else np.ascontiguousarray(mask, np.uint8)
    o = SimpleNamespace(base_color=np.zeros((n, 3)), dirs=np.zeros((n, 3)), sh_rest=None,
                        features=None, mlp_weights=None, sv_sites=None)
    if scene.app == 0:
        o.sh_rest = np.zeros((n, 15, 3))
    elif scene.app == 2:
        o.sv_sites = np.zeros((n, 7, 7))
    else:
        o.features = np.zeros((n, 8)); o.mlp_weights = np.zeros(num_mlp_weights())
    lib().gso_appearance_backward(C.c_int64(n), C.c_int(scene.app), C.c_int(deg), C.c_int(_act(scene)), _dp(base), _dp(sh),
                                  _dp(ft), _dp(wt), _dp(dirs), _p(m, C.c_uint8), _dp(g_color),
                                  _dp(o.base_color), _dp(o.sv_sites if scene.app == 2 else o.sh_rest), _dp(o.features),
                                  _dp(o.mlp_weights), _dp(o.dirs))
    return o


def mlp_kink_margin(scene, dirs, deg=None):
    """[n]: smallest |pre-activation| among the 32 hidden units of the default decoder, per Gaussian."""
    dirs = _f64(dirs); n = dirs.shape[0]
    out = np.zeros(n)
    lib().gso_mlp_kink_margin(C.c_int64(n), C.c_int(scene.active_degree if deg is None else deg),
                              _dp(_f64(scene.features)), _dp(_f64(scene.mlp_weights)), _dp(dirs), _dp(out))
    return out


def _tile_spans(suffix, dtype, ctype, valid, mean2d, chol, ext, width, height):
    valid = np.ascontiguousarray(valid, np.uint8)
    m = np.ascontiguousarray(mean2d, dtype); c = np.ascontiguousarray(chol, dtype)
    e = np.ascontiguousarray(ext, dtype)
    n = valid.shape[0]
    assert m.shape == (n, 2) and c.shape == (n, 3) and e.shape == (n, 4)
    rect = np.zeros((n, 4), np.int32); tt = np.zeros(n, np.uint32)
    f = getattr(lib(), "gso_tile_spans_" + suffix)
    f.restype = C.c_int64
    P = f(C.c_int64(n), _p(valid, C.c_uint8), _p(m, ctype), _p(c, ctype), _p(e, ctype), C.c_int(width),
          C.c_int(height), _p(rect, C.c_int32), _p(tt, C.c_uint32))
    return rect, tt, int(P)


def _sorted_instances(suffix, dtype, ctype, rect, tt, mean2d, chol, ext, depth_bits, width, height, P):
    rect = np.ascontiguousarray(rect, np.int32); tt = np.ascontiguousarray(tt, np.uint32)
    m = np.ascontiguousarray(mean2d, dtype); c = np.ascontiguousarray(chol, dtype)
    e = np.ascontiguousarray(ext, dtype); db = np.ascontiguousarray(depth_bits, np.uint32)
    gx, gy = (width + TILE - 1) // TILE, (height + TILE - 1) // TILE
    keys = np.zeros(P, np.uint64); vals = np.zeros(P, np.uint32)
    ranges = np.zeros((gx * gy, 2), np.uint32)
    getattr(lib(), "gso_sorted_instances_" + suffix)(
        C.c_int64(rect.shape[0]), _p(rect, C.c_int32), _p(tt, C.c_uint32), _p(m, ctype), _p(c, ctype), _p(e, ctype),
        _p(db, C.c_uint32), C.c_int(width), C.c_int(height), C.c_int64(P), _p(keys, C.c_uint64), _p(vals, C.c_uint32))
    lib().gso_tile_ranges(C.c_int64(P), _p(keys, C.c_uint64), C.c_int(gx * gy), _p(ranges, C.c_uint32))
    return keys, vals, ranges


def tile_spans_f32(valid, mean2d, chol, ext, width, height):
    """Integer stage on fp32 per-Gaussian values (from either side): bounding tile rectangle, tiles
    the alpha >= 1/255 ellipse meets, pair count.  chol = (la, lb, lc), ext = (ex, ey, tau, -)."""
    return _tile_spans("f32", np.float32, C.c_float, valid, mean2d, chol, ext, width, height)


def sorted_instances_f32(rect, tt, mean2d, chol, ext, depth_bits, width, height, P):
    return _sorted_instances("f32", np.float32, C.c_float, rect, tt, mean2d, chol, ext, depth_bits, width, height, P)


def tile_spans_f64(valid, mean2d, chol, ext, width, height):
    return _tile_spans("f64", np.float64, C.c_double, valid, mean2d, chol, ext, width, height)


def sorted_instances_f64(rect, tt, mean2d, chol, ext, depth_bits, width, height, P):
    return _sorted_instances("f64", np.float64, C.c_double, rect, tt, mean2d, chol, ext, depth_bits, width, height, P)


def cholesky_of_conic(conic):
    """(la, lb, lc) with conic = [[la^2, la lb], [la lb, lb^2 + lc^2]]."""
    conic = np.asarray(conic, np.float64)
    with np.errstate(invalid="ignore", divide="ignore"):
        la = np.sqrt(conic[:, 0]); lb = conic[:, 1] / la
        lc = np.sqrt(np.maximum(conic[:, 2] - lb * lb, 0.0))
    out = np.stack([la, lb, lc], 1)
    out[~np.isfinite(out).all(1)] = 0
    return out


def blend_forward(cam, vals, ranges, mean2d, conic, opacity, color):
    W, H = cam.width, cam.height
    bg = _f64(cam.background)
    o = SimpleNamespace(image=np.zeros((3, H, W)), final_T=np.zeros((H, W)),
                        n_contrib=np.zeros((H, W), np.uint32), fragile=np.zeros((H, W), np.uint8),
                        fragile_pos=np.zeros((H, W), np.int32))
    vals = np.ascontiguousarray(vals, np.uint32); ranges = np.ascontiguousarray(ranges, np.uint32)
    lib().gso_blend_forward(C.c_int(W), C.c_int(H), _dp(bg), _p(vals, C.c_uint32), _p(ranges, C.c_uint32),
                            _dp(_f64(mean2d)), _dp(_f64(conic)), _dp(_f64(opacity)), _dp(_f64(color)),
                            _dp(o.image), _dp(o.final_T), _p(o.n_contrib, C.c_uint32),
                            _p(o.fragile, C.c_uint8), _p(o.fragile_pos, C.c_int32))
    return o


def set_stop_window(width=1e-8):
    """Half-width of the window around T (1 - alpha) = 1e-4 in which a stop is flagged fragile (default 1e-8)."""
    lib().gso_set_stop_window(C.c_double(width))


def blend_pixel_records(px, py, vals, mean2d, conic, opacity, color):
    """What one pixel (centre px, py) records from the ordered list `vals`: the entries it composites and the
    ghosts (pairs it leaves out although they sit within tolerance of a blend threshold), in list order."""
    vals = np.ascontiguousarray(vals, np.uint32)
    cap = 2 * len(vals) + 4
    o = SimpleNamespace(g=np.zeros(cap, np.uint32), pos=np.zeros(cap, np.int32), alpha=np.zeros(cap), T=np.zeros(cap),
                        clamped=np.zeros(cap, np.uint8), ghost=np.zeros(cap, np.uint8))
    f = lib().gso_blend_pixel_records
    f.restype = C.c_int64
    k = int(f(C.c_double(px), C.c_double(py), _p(vals, C.c_uint32), C.c_int64(len(vals)), _dp(_f64(mean2d)),
              _dp(_f64(conic)), _dp(_f64(opacity)), _dp(_f64(color)), C.c_int64(cap), _p(o.g, C.c_uint32),
              _p(o.pos, C.c_int32), _dp(o.alpha), _dp(o.T), _p(o.clamped, C.c_uint8), _p(o.ghost, C.c_uint8)))
    assert k <= cap
    for nm in ("g", "pos", "alpha", "T", "clamped", "ghost"):
        setattr(o, nm, getattr(o, nm)[:k])
    return o


def blend_brute(cam, visible, depth_bits, mean2d, conic, opacity, color):
    W, H = cam.width, cam.height
    bg = _f64(cam.background)
    image = np.zeros((3, H, W)); final_T = np.zeros((H, W))
    visible = np.ascontiguousarray(visible, np.uint8); db = np.ascontiguousarray(depth_bits, np.uint32)
    lib().gso_blend_brute(C.c_int64(visible.shape[0]), C.c_int(W), C.c_int(H), _dp(bg),
                          _p(visible, C.c_uint8), _p(db, C.c_uint32), _dp(_f64(mean2d)), _dp(_f64(conic)),
                          _dp(_f64(opacity)), _dp(_f64(color)), _dp(image), _dp(final_T))
    return image, final_T


def blend_backward(cam, vals, ranges, mean2d, conic, opacity, color, G, with_abs=False):
    W, H = cam.width, cam.height
    bg = _f64(cam.background)
    n = np.asarray(opacity).shape[0]
    vals = np.ascontiguousarray(vals, np.uint32); ranges = np.ascontiguousarray(ranges, np.uint32)
    o = SimpleNamespace(color=np.zeros((n, 3)), opacity=np.zeros(n), conic=np.zeros((n, 3)),
                        mean2d=np.zeros((n, 2)), abs_sum=np.zeros((n, 9)) if with_abs else None,
                        flip_sum=np.zeros((n, 9)) if with_abs else None)
    lib().gso_blend_backward(C.c_int64(n), C.c_int(W), C.c_int(H), _dp(bg), C.c_int64(vals.shape[0]),
                             _p(vals, C.c_uint32), _p(ranges, C.c_uint32), _dp(_f64(mean2d)),
                             _dp(_f64(conic)), _dp(_f64(opacity)), _dp(_f64(color)), _dp(_f64(G)),
                             _dp(o.color), _dp(o.opacity), _dp(o.conic), _dp(o.mean2d), _dp(o.abs_sum),
                             _dp(o.flip_sum))
    return o


def preprocess_backward(means, log_scales, quats, opacity_logits, cam, visible, g_mean2d, g_conic,
                        g_opacity, g_dir):
    means, log_scales, quats, logits = _f64(means), _f64(log_scales), _f64(quats), _f64(opacity_logits)
    n = means.shape[0]
    visible = np.ascontiguousarray(visible, np.uint8)
    o = SimpleNamespace(means=np.zeros((n, 3)), log_scales=np.zeros((n, 3)), quats=np.zeros((n, 4)),
                        opacity_logits=np.zeros(n))
    cam_a = cam_array(cam)
    lib().gso_preprocess_backward(C.c_int64(n), _dp(means), _dp(log_scales), _dp(quats), _dp(logits),
                                  _dp(cam_a), _p(visible, C.c_uint8), _dp(_f64(g_mean2d)),
                                  _dp(_f64(g_conic)), _dp(_f64(g_opacity)), _dp(_f64(g_dir)),
                                  _dp(o.means), _dp(o.log_scales), _dp(o.quats), _dp(o.opacity_logits))
    return o


# ------------------------------------------------------------------------------------------
# The whole path, composed in the paper's order: preprocess (projection + fused colour) ->
# tile assignment -> sort -> blend -> blend backward -> appearance backward -> preprocess
# backward.
# ------------------------------------------------------------------------------------------

def render_forward(scene, cam):
    pre = preprocess(scene.means, scene.log_scales, scene.quats, scene.opacity_logits, cam)
    chol = cholesky_of_conic(pre.conic)
    with np.errstate(divide="ignore", invalid="ignore"):
        tau = np.where(pre.valid > 0, 2.0 * np.log(255.0 * pre.opacity), 0.0)
    ext = np.concatenate([pre.extent, tau[:, None], np.zeros_like(tau)[:, None]], 1)
    rect, tiles_touched, P = tile_spans_f64(pre.valid, pre.mean2d, chol, ext, cam.width, cam.height)
    pre.visible = (tiles_touched > 0).astype(np.uint8)      # visible = meets at least one tile
    pre.chol, pre.ext = chol, ext
    color, resid = appearance_forward(scene, pre.dir, mask=pre.visible)
    keys, vals, ranges = sorted_instances_f64(rect, tiles_touched, pre.mean2d, chol, ext, pre.depth_bits,
                                              cam.width, cam.height, P)
    bl = blend_forward(cam, vals, ranges, pre.mean2d, pre.conic, pre.opacity, color)
    return SimpleNamespace(pre=pre, color=color, residual=resid, rect=rect, tiles_touched=tiles_touched,
                           P=P, keys=keys, vals=vals, ranges=ranges, image=bl.image, final_T=bl.final_T,
                           n_contrib=bl.n_contrib, fragile=bl.fragile, fragile_pos=bl.fragile_pos)


def render_backward(scene, cam, fwd, G, with_abs=False):
    pre = fwd.pre
    g2 = blend_backward(cam, fwd.vals, fwd.ranges, pre.mean2d, pre.conic, pre.opacity, fwd.color, G,
                        with_abs=with_abs)
    ga = appearance_backward(scene, pre.dir, g2.color, mask=pre.visible)
    gp = preprocess_backward(scene.means, scene.log_scales, scene.quats, scene.opacity_logits, cam,
                             pre.visible, g2.mean2d, g2.conic, g2.opacity, ga.dirs)
    return SimpleNamespace(means=gp.means, log_scales=gp.log_scales, quats=gp.quats,
                           opacity_logits=gp.opacity_logits, base_color=ga.base_color,
                           sh_rest=ga.sh_rest, features=ga.features, mlp_weights=ga.mlp_weights, sv_sites=ga.sv_sites,
                           blend=g2, dirs=ga.dirs)


def render(scene, cam, G=None, with_abs=False):
    fwd = render_forward(scene, cam)
    grads = render_backward(scene, cam, fwd, G, with_abs=with_abs) if G is not None else None
    return fwd, grads
