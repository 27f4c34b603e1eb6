"""The separate-pass forward and backward of the default decoder (Eq. 5-7) on tcgen05.mma with the accumulators in tensor memory
(gs_set_decoder_engine(ctx, GS_ENGINE_TCGEN05)) against the oracle, element by element: split operands within the
2e-5 of the default kernel, plain fp16 operands within their own stated bound; sizes that give every persistent CTA
(8 per SM on 148 SMs, 128 Gaussians per tile) a second and a third tile and a ragged last one, the sweep's sizes up
to 10M, tiny and empty inputs, partly active input bands, the other colour activations, and the engine as
the (masked, in-place) appearance pass of the unfused rendering step.  After every run the context's status is read: no bounded wait
on the MMAs' mbarrier ran out."""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from conftest import record_parity
from gpu_helpers import run_gpu
from test_gpu_half_precision import COLOR_ATOL as HALF_COLOR_ATOL
from test_gpu_decode_at_size import _check as check_decode

pytestmark = pytest.mark.gpu

WAVE = 8 * 148 * 128      # Gaussians one full wave of the kernel's CTAs takes per trip


def _forward(n, precision=0, deg=None, act=0, engine=1):
    import torch
    from paper_2609_05255_b200 import api
    sc, dirs, _ = scenes.config5(n, scenes.APP_NEURAL)
    sc.decoder_precision = precision
    sc.color_activation = act
    if deg is not None:
        sc.active_degree = deg
    ctx = api.Context(0)
    api.gs_set_decoder_engine(ctx, engine)
    ds = api.upload_scene(sc, ctx.device)
    d = torch.from_numpy(dirs).to(ctx.device)
    color = torch.full((n, 3), float("nan"), device=ctx.device)
    api.gs_appearance_forward(ctx, ds, d, color)
    torch.cuda.synchronize()
    api.gs_async_status(ctx)
    out = color.cpu().numpy()
    ctx.close()
    return sc, dirs, out


@pytest.mark.parametrize("n", [1, 31, 129, 4_099, WAVE + 1, 2 * WAVE, 2 * WAVE + 127, 1_000_000, 3_000_000, 10_000_000])
def test_tcgen05_forward_split_operands(oracle, n):
    sc, dirs, got = _forward(n)
    ref, _ = oracle.appearance_forward(sc, dirs)
    err = float(np.abs(got - ref).max())
    record_parity(f"decode_tcgen05_split_{n}", "decode vs oracle", color_max_err=err)
    assert np.all(np.isfinite(got)) and err < 2e-5, err


@pytest.mark.parametrize("n", [4_099, 2 * WAVE + 127, 1_000_000])
def test_tcgen05_forward_plain_fp16_operands(oracle, n):
    sc, dirs, got = _forward(n, precision=1)
    ref, _ = oracle.appearance_forward(sc, dirs)
    err = float(np.abs(got - ref).max())
    record_parity(f"decode_tcgen05_half_{n}", "half precision", color_max_err=err)
    assert 1e-6 < err < HALF_COLOR_ATOL, err


def test_tcgen05_forward_empty_and_disabled_residual(oracle):
    import torch
    from paper_2609_05255_b200 import api
    sc, dirs, got = _forward(5_003, deg=0)            # residual disabled: no product at all, colour = activation(c0 + 0.5)
    ref, _ = oracle.appearance_forward(sc, dirs)
    assert np.abs(got - ref).max() < 1e-6
    ctx = api.Context(0)
    api.gs_set_decoder_engine(ctx, api.GS_ENGINE_TCGEN05)
    sc0, dirs0, _ = scenes.config5(0, scenes.APP_NEURAL)
    ds = api.upload_scene(sc0, ctx.device)
    api.gs_appearance_forward(ctx, ds, torch.empty((0, 3), device=ctx.device), torch.empty((0, 3), device=ctx.device))
    torch.cuda.synchronize()
    with pytest.raises(api.GsError):
        api.gs_set_decoder_engine(ctx, 7)
    ctx.close()


@pytest.mark.parametrize("deg,act", [(1, 0), (2, 1), (3, 2), (3, 3)])
def test_tcgen05_forward_bands_and_activations(oracle, deg, act):
    sc, dirs, got = _forward(40_003, deg=deg, act=act)
    ref, _ = oracle.appearance_forward(sc, dirs)
    assert np.abs(got - ref).max() < 2e-5


def test_tcgen05_equals_warp_mma_within_rounding():
    _, _, a = _forward(300_001, engine=0)
    _, _, b = _forward(300_001, engine=1)
    assert np.abs(a - b).max() < 2e-6                 # same operands and products; only the order of the fp32 sums differs


def test_tcgen05_engine_in_the_unfused_step(oracle):
    """The engine as the appearance pass of the rendering step (GsScene.separate_pass): masked by the tiles-touched
    array, colours in place over the directions.  Integers identical and colours as close to the oracle as with the
    fused kernel."""
    import copy
    from paper_2609_05255_b200 import api
    w = scenes.config3(scenes.APP_NEURAL, n=30_000, width=320, height=208, views=1)
    sc = copy.copy(w.scene)
    sc.separate_pass = 1
    got = run_gpu(sc, w.cameras[0], decoder_engine=api.GS_ENGINE_TCGEN05)
    fused = run_gpu(w.scene, w.cameras[0])
    ref = oracle.render_forward(w.scene, w.cameras[0])
    vis = got.tiles_touched > 0
    assert vis.sum() > 10_000
    for name in ("tiles_touched", "rect", "depth_order", "sorted_vals", "tile_ranges", "n_contrib"):
        assert np.array_equal(getattr(got, name), getattr(fused, name)), name
    assert np.abs(got.color[vis] - fused.color[vis]).max() < 2e-6
    assert np.abs(got.image - fused.image).max() < 1e-5
    both = vis & (ref.tiles_touched > 0)
    assert np.abs(got.color[both] - ref.color[both]).max() < 2e-5


# The backward on the same engine (recompute, data gradients, and the weight gradients as products over the 128
# Gaussians of a tile accumulated in tensor memory), held to the rules of the warp-level kernel's test: per-Gaussian
# gradients by the literal rule except rows at a ReLU kink that the oracle names, weight gradients over the other rows.
# 3 CTAs per SM x 148 SMs x 128 Gaussians = one trip of the backward's persistent grid.
WAVE_BWD = 3 * 148 * 128


@pytest.mark.parametrize("n", [1, 129, 4_099, WAVE_BWD + 1, 2 * WAVE_BWD + 127, 1_000_000, 3_000_000, 10_000_000])
def test_tcgen05_backward_split_operands(oracle, n):
    check_decode(oracle, "neural_split", n, engine=1)


@pytest.mark.parametrize("n", [4_099, 2 * WAVE_BWD + 127, 1_000_000])
def test_tcgen05_backward_plain_fp16_operands(oracle, n):
    check_decode(oracle, "neural_half", n, engine=1)
