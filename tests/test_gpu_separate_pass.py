"""The unfused reference path of the rendering step (Sec. 4 "CUDA Implementation", App. D "Fusion"): the
appearance model evaluated as passes of its own around the rasterizer, exchanging directions, colours and
their gradients through global memory.  It must give what the fused step gives (the paper's own validation of
its fused kernels), and it is the way a decoder of another size goes through the whole step: those are
checked against the oracle."""
import copy

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from gpu_helpers import GRAD_ATOL, check_bound, grad_mismatch, grad_names, image_mismatch, run_gpu

pytestmark = pytest.mark.gpu

INT_FIELDS = ("depth_key", "rect", "tiles_touched", "depth_order", "sorted_tiles", "sorted_vals", "tile_ranges", "n_contrib")


@pytest.mark.parametrize("app", [scenes.APP_SH, scenes.APP_NEURAL, scenes.APP_SV], ids=["sh", "neural", "sv"])
def test_unfused_step_equals_fused_step(app):
    w = scenes.config2(n=12_011, app=app)
    cam = w.cameras[0]
    G = scenes.upstream_gradient(cam, 7)
    fused = run_gpu(w.scene, cam, G)
    sc = copy.copy(w.scene)
    sc.separate_pass = 1
    unfused = run_gpu(sc, cam, G)
    for nm in INT_FIELDS:
        assert np.array_equal(getattr(fused, nm), getattr(unfused, nm)), nm
    vis = fused.visible
    assert vis.sum() > 5_000
    assert np.abs(fused.color[vis] - unfused.color[vis]).max() < 1e-5
    assert np.abs(fused.image - unfused.image).max() < 1e-5
    for nm in grad_names(app):
        a, b = getattr(fused.grads, nm), getattr(unfused.grads, nm)
        # both runs sum the blend's atomics in their own order: the rule of the parity tests, between the two
        bad = grad_mismatch(a, b)
        check_bound(f"unfused_vs_fused_app{app}", "between two runs", "outside_literal_rule", int(bad.sum()), parameter=nm)
        assert np.abs(a - b).max() <= max(2e-3 * np.abs(a).max(), GRAD_ATOL), nm
        if nm != "mlp_weights":
            assert np.all(b[~vis] == 0), nm        # culled Gaussians: exact zeros from the separate passes too


def test_unfused_step_with_nan_appearance_on_a_culled_gaussian():
    """A Gaussian that is culled never reaches the appearance passes: its parameters may hold anything."""
    w = scenes.config2(n=3_001, app=scenes.APP_NEURAL)
    cam = w.cameras[0]
    G = scenes.upstream_gradient(cam, 8)
    sc = copy.copy(w.scene)
    sc.separate_pass = 1
    sc.means = sc.means.copy(); sc.features = sc.features.copy(); sc.base_color = sc.base_color.copy()
    sc.means[5] = (0.0, 0.0, -3.0)                       # behind the camera
    sc.features[5] = np.float16("nan"); sc.base_color[5] = np.nan
    out = run_gpu(sc, cam, G)
    assert not out.visible[5]
    for nm in grad_names(scenes.APP_NEURAL):
        assert np.isfinite(getattr(out.grads, nm)).all(), nm
    assert np.isfinite(out.image).all()


@pytest.mark.parametrize("arch", [(16, 1, 8), (32, 2, 8), (16, 2, 16), (16, 3, 8)], ids=lambda a: "h%d_l%d_f%d" % a)
def test_decoder_variant_through_the_whole_step(oracle, arch):
    hidden, layers, nfeat = arch
    case = "variant_step_h%d_l%d_f%d" % arch
    w = scenes.config2(n=20_011, app=scenes.APP_NEURAL)      # the size of the fused parity tests: same tolerances
    cam = w.cameras[0]
    sc = w.scene
    rng = np.random.default_rng(np.random.PCG64(4242))
    _, sc.features, sc.mlp_weights = scenes.draw_neural_appearance(rng, sc.n, hidden, layers, nfeat)
    sc.mlp_hidden, sc.mlp_layers = hidden, layers
    G = scenes.upstream_gradient(cam, 9)
    gpu = run_gpu(sc, cam, G)
    fwd, grads = oracle.render(sc, cam, G)
    same_vis = gpu.visible == fwd.pre.visible.astype(bool)
    assert (~same_vis).sum() <= 2
    both = gpu.visible & same_vis
    assert np.abs(gpu.color[both] - fwd.color[both]).max() < 2e-5
    assert image_mismatch(gpu.image, fwd.image, fwd.fragile).sum() == 0
    # the appearance passes in isolation: the oracle's decoder fed with the GPU's own dL/dcolor
    vis = gpu.visible.astype(np.uint8)
    ga = oracle.appearance_backward(sc, fwd.pre.dir, gpu.g2d[:, 0:3].astype(np.float64), mask=vis)
    gp = oracle.preprocess_backward(sc.means, sc.log_scales, sc.quats, sc.opacity_logits, cam, vis,
                                    gpu.g2d[:, 7:9], gpu.g2d[:, 4:7], gpu.g2d[:, 3], ga.dirs)
    ref = dict(means=gp.means, log_scales=gp.log_scales, quats=gp.quats, opacity_logits=gp.opacity_logits,
               base_color=ga.base_color, features=ga.features, mlp_weights=ga.mlp_weights)
    assert gpu.grads.features.shape == (sc.n, nfeat) and gpu.grads.mlp_weights.shape == ref["mlp_weights"].shape
    for nm in grad_names(scenes.APP_NEURAL):
        got = getattr(gpu.grads, nm)
        bad = grad_mismatch(got, ref[nm])
        if nm != "mlp_weights":
            bad[~same_vis] = False
            check_bound(case, "per-Gaussian backward", "outside_literal_rule", int(bad.sum()), parameter=nm)
        else:
            assert np.abs(got - ref[nm]).max() <= 2e-4 * np.abs(ref[nm]).max()
    # end to end against the oracle's own gradients, by the rule of the fused parity tests
    for nm in grad_names(scenes.APP_NEURAL):
        got, want = getattr(gpu.grads, nm), getattr(grads, nm)
        bad = grad_mismatch(got, want)
        d = np.abs(got - want)
        if nm != "mlp_weights":
            bad[~same_vis] = False; d[~same_vis] = 0
        check_bound(case, "end to end", "outside_literal_rule", int(bad.sum()), parameter=nm)
        assert d.max() <= max(1e-2 * np.abs(want).max(), GRAD_ATOL), nm
        if nm != "mlp_weights":
            assert np.all(got[~gpu.visible] == 0)


@pytest.mark.parametrize("app", [scenes.APP_SH, scenes.APP_NEURAL, scenes.APP_SV], ids=["sh", "neural", "sv"])
@pytest.mark.parametrize("n", [0, 1, 33, 130])
def test_unfused_step_on_tiny_scenes(oracle, app, n):
    w = scenes.config2(n=max(n, 1), app=app)
    sc, cam = w.scene, w.cameras[0]
    if n == 0:
        for f in ("means", "log_scales", "quats", "opacity_logits", "base_color", "sh_rest", "features", "sv_sites"):
            if getattr(sc, f) is not None:
                setattr(sc, f, getattr(sc, f)[:0])
    sc.separate_pass = 1
    sc.color_activation = 1                      # softplus, to go through the activation argument too
    G = scenes.upstream_gradient(cam, 12)
    gpu = run_gpu(sc, cam, G)
    fwd, grads = oracle.render(sc, cam, G)
    assert image_mismatch(gpu.image, fwd.image, fwd.fragile).sum() == 0
    if n == 0:
        return
    for nm in grad_names(app):
        got, want = getattr(gpu.grads, nm), getattr(grads, nm)
        assert np.abs(got - want).max() <= max(2e-3 * np.abs(want).max(), GRAD_ATOL), nm


def test_workspace_covers_the_separate_passes():
    from paper_2609_05255_b200 import api
    n = 100_000
    # backward scratch: [n,12] + three [n,3] arrays, each rounded up to 256 bytes
    assert api.gs_workspace_bytes(n, 64, 64, 0) >= n * (12 + 9) * 4


@pytest.mark.parametrize("app", [scenes.APP_SH, scenes.APP_SV], ids=["sh", "sv"])
@pytest.mark.parametrize("n", [32, 128, 160, 4096, 4128, 75_776, 75_777])
def test_bulk_copy_decode_at_warp_and_block_boundaries(oracle, app, n):
    """The separate-pass kernels of the explicit models move whole 32-row slabs by bulk copies and a ragged last
    warp by plain loads: sizes that end exactly on a warp, on a block, one warp past a block, and (75 776 = 592 x
    128) exactly one block per persistent CTA and one Gaussian more."""
    import torch
    from paper_2609_05255_b200 import api
    sc, dirs, gcol = scenes.config5(n, app)
    ctx = api.Context(0)
    ds = api.upload_scene(sc, ctx.device)
    d = torch.from_numpy(dirs).to(ctx.device); gc = torch.from_numpy(gcol).to(ctx.device)
    color = torch.full((n, 3), float("nan"), device=ctx.device)
    api.gs_appearance_forward(ctx, ds, d, color)
    grads = api.alloc_grads_for(ds, ctx.device)
    rows = grads.sh_rest if app == scenes.APP_SH else grads.sv_sites
    rows.fill_(float("nan")); grads.base_color.fill_(float("nan"))
    gd = torch.full((n, 3), float("nan"), device=ctx.device)
    api.gs_appearance_backward(ctx, ds, d, gc, grads, gd)
    torch.cuda.synchronize()
    api.gs_async_status(ctx)
    ref_c, _ = oracle.appearance_forward(sc, dirs)
    ref = oracle.appearance_backward(sc, dirs, gcol)
    assert np.abs(color.cpu().numpy() - ref_c).max() < 2e-5
    assert grad_mismatch(grads.base_color.cpu().numpy(), ref.base_color).sum() == 0
    assert grad_mismatch(gd.cpu().numpy(), ref.dirs).sum() == 0
    assert grad_mismatch(rows.cpu().numpy(), ref.sh_rest if app == scenes.APP_SH else ref.sv_sites).sum() == 0
    ctx.close()
