"""Parity of the viewer-side kernels (gs_neural_fold, gs_neural_prepass) against the oracle: the folded
pre-activations as half-precision values, the unquantised colour within what half-precision operands
allow, and the RGBA8 texels against the texels the oracle makes of its own colour."""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes

pytestmark = pytest.mark.gpu


def _scene(n, seed):
    w = scenes.config2(n=n)
    sc = w.scene
    rng = np.random.default_rng(seed)
    sc.features = rng.normal(0, 0.6, sc.features.shape).astype(np.float16)
    return sc, w.cameras[0]


def _run(sc, cam, deg, want_color=True):
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    dev = ctx.device
    sc.active_degree = deg
    ds = api.upload_scene(sc, dev)
    n = ds.n
    pre = torch.full((max(n, 1), 16), float("nan"), device=dev, dtype=torch.float16)
    rgba = torch.full((max(n, 1), 4), 77, device=dev, dtype=torch.uint8)
    color = torch.full((max(n, 1), 3), float("nan"), device=dev) if want_color else None
    api.gs_neural_fold(ctx, ds, pre)
    api.gs_neural_prepass(ctx, ds, pre, api.make_camera(cam), rgba, color)
    torch.cuda.synchronize()
    out = pre.cpu().numpy()[:n], rgba.cpu().numpy()[:n], (color.cpu().numpy()[:n] if want_color else None)
    ctx.close()
    return out


def _eye(cam):
    R, t = np.asarray(cam.w2c, np.float64)[:, :3], np.asarray(cam.w2c, np.float64)[:, 3]
    return -R.T @ t


@pytest.mark.parametrize("deg", [3, 1])
def test_fold_and_prepass_match_oracle(oracle, deg):
    sc, cam = _scene(10_007, 21)                       # ragged: the last warp holds 23 Gaussians
    cam = scenes.orbit_camera(cam.width, cam.height, 0.7)
    pre, rgba, color = _run(sc, cam, deg)
    want_pre = oracle.neural_fold(sc)
    # fp32 accumulation, then one rounding to half: within one half-precision ulp of the rounded exact value
    err = np.abs(pre.astype(np.float64) - want_pre)
    assert np.all(err <= 2.0 ** -10 * np.abs(want_pre) + 1e-6)
    # per frame, on the GPU's own pre-activations: half-precision operands (2^-11 relative each) in three layers
    want = oracle.neural_prepass(sc, pre.astype(np.float64), _eye(cam), deg=deg)
    assert np.abs(color - want).max() < 4e-3 and np.abs(color - want).mean() < 4e-4
    o = 1 / (1 + np.exp(-sc.opacity_logits.astype(np.float64)))
    texel = oracle.rgba8(want, o)
    diff = np.abs(rgba.astype(int) - texel.astype(int))
    assert diff.max() <= 1 and (diff[:, :3] != 0).mean() < 0.1       # a colour may land on the other side of a rounding step
    assert (diff[:, 3] != 0).mean() < 1e-3
    # the texel is the GPU's own colour, quantised exactly
    assert np.array_equal(rgba[:, :3], np.floor(np.clip(color.astype(np.float64), 0, 1) * 255 + 0.5).astype(np.uint8))


def test_prepass_degree_zero_and_no_colour_output(oracle):
    sc, cam = _scene(999, 22)
    pre, rgba, color = _run(sc, cam, 0)
    want = np.maximum(sc.base_color.astype(np.float64) + 0.5, 0)
    assert np.abs(color - want).max() < 1e-6
    pre2, rgba2, none = _run(sc, cam, 0, want_color=False)
    assert none is None and np.array_equal(rgba, rgba2)


def test_prepass_at_full_size_agrees_with_the_training_decoder(oracle):
    """1M Gaussians: the viewer's colour against the colour the training-side separate-pass decoder gives for the
    same directions (two different code paths of this library; the oracle ties each to the definition at small n)."""
    import torch
    from paper_2609_05255_b200 import api
    sc = scenes.config3(scenes.APP_NEURAL).scene
    cam = scenes.orbit_cameras(1256, 828, 8)[3]
    ctx = api.Context(0)
    dev = ctx.device
    ds = api.upload_scene(sc, dev)
    n = ds.n
    pre = torch.empty((n, 16), device=dev, dtype=torch.float16)
    rgba = torch.empty((n, 4), device=dev, dtype=torch.uint8)
    color = torch.empty((n, 3), device=dev)
    api.gs_neural_fold(ctx, ds, pre)
    api.gs_neural_prepass(ctx, ds, pre, api.make_camera(cam), rgba, color)
    eye = torch.tensor(_eye(cam), device=dev, dtype=torch.float32)
    d = ds.means - eye
    d = (d / d.norm(dim=1, keepdim=True)).contiguous()
    ref = torch.empty((n, 3), device=dev)
    api.gs_appearance_forward(ctx, ds, d, ref)
    torch.cuda.synchronize()
    assert float((color - ref).abs().max()) < 6e-3 and float((color - ref).abs().mean()) < 5e-4
    # sampled Gaussians against the oracle, one by one
    idx = np.random.default_rng(0).choice(n, 2000, replace=False)
    rows = ("means", "log_scales", "quats", "opacity_logits", "base_color", "features")
    sub = scenes.Scene(**{k: (getattr(sc, k)[idx] if k in rows else getattr(sc, k)) for k in sc.__dataclass_fields__})
    want = oracle.neural_prepass(sub, oracle.neural_fold(sub), _eye(cam))
    assert np.abs(color.cpu().numpy()[idx] - want).max() < 6e-3
    ctx.close()


@pytest.mark.parametrize("act", [1, 2, 3])
def test_prepass_with_other_colour_activations(oracle, act):
    sc, cam = _scene(4_001, 30 + act)
    sc.color_activation = act
    sc.base_color = np.random.default_rng(act).uniform(-0.8, 0.8, sc.base_color.shape).astype(np.float32)
    pre, rgba, color = _run(sc, cam, 3)
    want = oracle.neural_prepass(sc, pre.astype(np.float64), _eye(cam), deg=3)
    assert np.abs(color - want).max() < 4e-3
    assert np.abs(want - np.maximum(sc.base_color + 0.5, 0)).max() > 1e-2
    texel = oracle.rgba8(want, 1 / (1 + np.exp(-sc.opacity_logits.astype(np.float64))))
    assert np.abs(rgba.astype(int) - texel.astype(int)).max() <= 1
