"""The Spherical Voronoi appearance model (Eq. 3) through the CUDA path: the separate-pass decode, forward
and backward, and the whole fused step, each against the oracle with the same rules as the other models."""
from types import SimpleNamespace

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from gpu_helpers import grad_mismatch, run_gpu
import test_gpu_parity as small

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("deg", [3, 0])
@pytest.mark.parametrize("act", [0, 2])
def test_separate_pass_decode(oracle, deg, act):
    import torch
    from paper_2609_05255_b200 import api
    n = 10_037
    sc, dirs, gcol = scenes.config5(n, scenes.APP_SV)
    sc.active_degree, sc.color_activation = deg, act
    ctx = api.Context(0)
    ds = api.upload_scene(sc, ctx.device)
    d = torch.from_numpy(dirs).to(ctx.device); gc = torch.from_numpy(gcol).to(ctx.device)
    color = torch.empty((n, 3), device=ctx.device)
    api.gs_appearance_forward(ctx, ds, d, color)
    grads = api.alloc_grads(n, scenes.APP_SV, ctx.device)
    grads.sv_sites.fill_(float("nan"))
    gd = torch.empty((n, 3), device=ctx.device)
    api.gs_appearance_backward(ctx, ds, d, gc, grads, gd)
    torch.cuda.synchronize()
    ref_c, ref_A = oracle.appearance_forward(sc, dirs)
    ref = oracle.appearance_backward(sc, dirs, gcol)
    assert np.abs(color.cpu().numpy() - ref_c).max() < 2e-5
    if deg:
        assert np.abs(ref_A).max() > 0.05
    assert grad_mismatch(grads.base_color.cpu().numpy(), ref.base_color).sum() == 0
    assert grad_mismatch(gd.cpu().numpy(), ref.dirs).sum() == 0
    assert grad_mismatch(grads.sv_sites.cpu().numpy(), ref.sv_sites).sum() == 0
    ctx.close()


@pytest.fixture(scope="module")
def fused(oracle):
    w = scenes.config2(n=12_013, app=scenes.APP_SV)
    cam = w.cameras[0]
    G = scenes.upstream_gradient(cam, 123)
    gpu = run_gpu(w.scene, cam, G)
    fwd, grads = oracle.render(w.scene, cam, G, with_abs=True)
    m2, co, col = (a.astype(np.float64) for a in (gpu.mean2d, gpu.conic_opacity, gpu.color))
    for a in (m2, co, col):
        a[~gpu.visible] = 0
    iso = oracle.blend_forward(cam, gpu.sorted_vals, gpu.tile_ranges, m2, co[:, :3], co[:, 3], col)
    iso_g = oracle.blend_backward(cam, gpu.sorted_vals, gpu.tile_ranges, m2, co[:, :3], co[:, 3], col, G, with_abs=True)
    r = SimpleNamespace(w=w, cam=cam, G=G, gpu=gpu, fwd=fwd, grads=grads, iso=iso, iso_g=iso_g)
    return {"sv": r}, "sv"


def test_fused_step_floats_integers_and_image(fused, oracle):
    results, name = fused
    small.test_per_gaussian_floats(results, name)
    small.test_integer_stage_bit_exact(results, oracle, name)
    small.test_image(results, name)


def test_fused_step_gradients(fused, oracle):
    results, name = fused
    small.test_blend_backward_2d_gradients(results, name)
    small.test_parameter_gradients(results, oracle, name)
