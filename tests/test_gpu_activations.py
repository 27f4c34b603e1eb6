"""The colour activations of Sec. 3.1 other than the baseline ReLU, through the CUDA path: the
separate-pass decode (forward and backward) and the whole fused step, each against the oracle with the
same rules as the baseline cases."""
from types import SimpleNamespace

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from gpu_helpers import grad_mismatch, run_gpu
import test_gpu_parity as small

pytestmark = pytest.mark.gpu

ACTS = {"softplus": 1, "sigmoid": 2, "hard_sigmoid": 3}


@pytest.mark.parametrize("app", [scenes.APP_SH, scenes.APP_NEURAL])
@pytest.mark.parametrize("act", list(ACTS))
def test_separate_pass_decode(oracle, app, act):
    import torch
    from paper_2609_05255_b200 import api
    n = 6_011
    sc, dirs, gcol = scenes.config5(n, app)
    sc.color_activation = ACTS[act]
    rng = np.random.default_rng(ACTS[act])
    sc.base_color = rng.uniform(-0.8, 0.8, sc.base_color.shape).astype(np.float32)      # both kinks of the clamp in range
    ctx = api.Context(0)
    ds = api.upload_scene(sc, ctx.device)
    d = torch.from_numpy(dirs).to(ctx.device); gc = torch.from_numpy(gcol).to(ctx.device)
    color = torch.empty((n, 3), device=ctx.device)
    api.gs_appearance_forward(ctx, ds, d, color)
    grads = api.alloc_grads(n, app, ctx.device)
    gd = torch.empty((n, 3), device=ctx.device)
    api.gs_appearance_backward(ctx, ds, d, gc, grads, gd)
    torch.cuda.synchronize()
    ref_c, _ = oracle.appearance_forward(sc, dirs)
    ref = oracle.appearance_backward(sc, dirs, gcol)
    assert np.abs(color.cpu().numpy() - ref_c).max() < 2e-5
    assert np.abs(ref_c - np.maximum(sc.base_color + 0.5, 0)).max() > 1e-2               # not the baseline's colours
    # a pre-activation within 1e-5 of a kink of the clamp may take the other one-sided derivative
    near_kink = np.zeros((n, 3), bool)
    if act == "hard_sigmoid":
        near_kink = (np.abs(ref_c) < 1e-5) | (np.abs(ref_c - 1) < 1e-5)
    assert (grad_mismatch(grads.base_color.cpu().numpy(), ref.base_color) & ~near_kink).sum() == 0
    rows = ~near_kink.any(1)
    assert grad_mismatch(gd.cpu().numpy()[rows], ref.dirs[rows]).sum() == 0
    if app == scenes.APP_SH:
        assert grad_mismatch(grads.sh_rest.cpu().numpy()[rows], ref.sh_rest[rows]).sum() == 0
    else:
        assert grad_mismatch(grads.features.cpu().numpy()[rows], ref.features[rows]).sum() == 0
        if rows.all():
            assert grad_mismatch(grads.mlp_weights.cpu().numpy(), ref.mlp_weights).sum() == 0
    ctx.close()


CASES = {f"{app_name}_{act}": (app, code) for app_name, app in (("sh", scenes.APP_SH), ("neural", scenes.APP_NEURAL))
         for act, code in ACTS.items()}


@pytest.fixture(scope="module", params=list(CASES))
def fused(request, oracle):
    app, code = CASES[request.param]
    w = scenes.config2(n=8_009, app=app)
    w.scene.color_activation = code
    cam = w.cameras[0]
    G = scenes.upstream_gradient(cam, 99)
    gpu = run_gpu(w.scene, cam, G)
    fwd, grads = oracle.render(w.scene, cam, G, with_abs=True)
    m2, co, col = (a.astype(np.float64) for a in (gpu.mean2d, gpu.conic_opacity, gpu.color))
    for a in (m2, co, col):
        a[~gpu.visible] = 0
    iso = oracle.blend_forward(cam, gpu.sorted_vals, gpu.tile_ranges, m2, co[:, :3], co[:, 3], col)
    iso_g = oracle.blend_backward(cam, gpu.sorted_vals, gpu.tile_ranges, m2, co[:, :3], co[:, 3], col, G, with_abs=True)
    r = SimpleNamespace(w=w, cam=cam, G=G, gpu=gpu, fwd=fwd, grads=grads, iso=iso, iso_g=iso_g)
    return {request.param: r}, request.param


def test_fused_step_floats_and_image(fused, oracle):
    results, name = fused
    small.test_per_gaussian_floats(results, name)
    small.test_image(results, name)


def test_fused_step_gradients(fused, oracle):
    results, name = fused
    small.test_parameter_gradients(results, oracle, name)
