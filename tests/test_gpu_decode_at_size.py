"""The separate-pass appearance decode (the appearance-stage sweep: colour decode forward + backward only, random
unit directions) compared with the oracle element by element AT THE SIZES THE SWEEP IS TIMED ON - 1M, 3M and 10M
Gaussians - for degree-3 SH, Spherical Voronoi, the neural decoder with split operands and with plain fp16
operands; and at sizes that make every CTA of the persistent grids take a second and a third full trip (and one
Gaussian more), so that the later bulk loads of both slabs, both barrier phases and the accumulation of the
decoder-weight gradient across trips are all checked against the oracle, not only against themselves."""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from conftest import record_parity
from gpu_helpers import grad_mismatch
from test_gpu_half_precision import COLOR_ATOL as HALF_COLOR_ATOL, check_gradient as check_half_gradient

pytestmark = pytest.mark.gpu

MODELS = {"sh": (scenes.APP_SH, 0), "sv": (scenes.APP_SV, 0), "neural_split": (scenes.APP_NEURAL, 0),
          "neural_half": (scenes.APP_NEURAL, 1)}

# Colours: 2e-5 absolute (split / explicit models).  Per-Gaussian gradients: the literal rule, 1e-3 relative or 1e-5
# absolute, no exceptions for the explicit models; for the neural decoder a Gaussian whose hidden pre-activation sits
# within fp32 rounding of the ReLU kink may take the other branch - measured at most 3 rows in 10M, bounded at 1e-6
# of the rows.  Decoder-weight gradients (each the sum of n signed terms, accumulated in fp32 per CTA): the literal
# rule for all but a few of the 816 (bounded per size below, from the measured counts) and no element off by more
# than 1e-5 of the largest one.
KINK_ROW_FRACTION = 1e-6
WEIGHTS_OFF = {1_000_000: 8, 3_000_000: 8, 10_000_000: 8}
WEIGHTS_OFF_DEFAULT = 8
WEIGHT_MAX_REL = 1e-5


def _decode(app, precision, n):
    import torch
    from paper_2609_05255_b200 import api
    sc, dirs, gcol = scenes.config5(n, app)
    sc.decoder_precision = precision
    ctx = api.Context(0)
    ds = api.upload_scene(sc, ctx.device)
    d = torch.from_numpy(dirs).to(ctx.device); gc = torch.from_numpy(gcol).to(ctx.device)
    color = torch.full((n, 3), float("nan"), device=ctx.device)
    api.gs_appearance_forward(ctx, ds, d, color)
    grads = api.alloc_grads_for(ds, ctx.device)
    for t in (grads.base_color, grads.sh_rest, grads.sv_sites, grads.features, grads.mlp_weights):
        if t is not None:
            t.fill_(float("nan"))
    gd = torch.full((n, 3), float("nan"), device=ctx.device)
    api.gs_appearance_backward(ctx, ds, d, gc, grads, gd)
    torch.cuda.synchronize()
    api.gs_async_status(ctx)                  # no bounded wait of a bulk-copy kernel ran out
    cp = lambda t: None if t is None else t.cpu().numpy()
    out = dict(color=cp(color), base_color=cp(grads.base_color), dirs=cp(gd), sh_rest=cp(grads.sh_rest),
               sv_sites=cp(grads.sv_sites), features=cp(grads.features), mlp_weights=cp(grads.mlp_weights))
    ctx.close()
    del color, grads, gd, d, gc, ds
    torch.cuda.empty_cache()
    return sc, dirs, gcol, out


def _check(oracle, model, n):
    app, precision = MODELS[model]
    sc, dirs, gcol, got = _decode(app, precision, n)
    ref_c, _ = oracle.appearance_forward(sc, dirs)
    ref = oracle.appearance_backward(sc, dirs, gcol)
    case = f"decode_{model}_{n}"
    err_c = float(np.abs(got["color"] - ref_c).max())
    assert np.all(np.isfinite(got["color"]))
    if precision == 1:
        assert err_c < HALF_COLOR_ATOL, err_c
        for nm in ("base_color", "features", "dirs", "mlp_weights"):
            check_half_gradient(got[nm], getattr(ref, nm), nm)
        record_parity(case, "half precision", color_max_err=err_c)
        return
    assert err_c < 2e-5, err_c
    rows = {"sh": ["sh_rest"], "sv": ["sv_sites"], "neural_split": ["features"]}[model]
    counts = {}
    for nm in ["base_color", "dirs"] + rows:
        bad = grad_mismatch(got[nm], getattr(ref, nm))
        bad_rows = int(bad.reshape(n, -1).any(1).sum())
        counts[nm + "_rows_off"] = bad_rows
        limit = int(KINK_ROW_FRACTION * n) + (3 if app == scenes.APP_NEURAL else 0)
        assert bad_rows <= (limit if app == scenes.APP_NEURAL else 0), f"{nm}: {bad_rows} of {n} rows off"
    if app == scenes.APP_NEURAL:
        w_got, w_ref = got["mlp_weights"].astype(np.float64), ref.mlp_weights
        off = int(grad_mismatch(w_got, w_ref).sum())
        rel = float(np.abs(w_got - w_ref).max() / np.abs(w_ref).max())
        counts.update(weights_off=off, weights_max_rel_to_largest=rel)
        assert off <= WEIGHTS_OFF.get(n, WEIGHTS_OFF_DEFAULT), f"{off} of 816 weight gradients outside the literal rule"
        assert rel <= WEIGHT_MAX_REL, rel
    record_parity(case, "decode vs oracle", color_max_err=err_c, **counts)


@pytest.mark.parametrize("n", [1_000_000, 3_000_000, 10_000_000])
@pytest.mark.parametrize("model", list(MODELS))
def test_decode_at_the_sweep_sizes(oracle, model, n):
    _check(oracle, model, n)


# 592 and 444 CTAs are the persistent grids of these kernels on a 148-SM part (4 and 3 resident CTAs per SM), 128
# Gaussians per CTA and trip: k full trips for every CTA, and one Gaussian more.
@pytest.mark.parametrize("n", [592 * 128 * 2, 592 * 128 * 2 + 1, 592 * 128 * 3, 592 * 128 * 3 + 1,
                               444 * 128 * 2, 444 * 128 * 2 + 1, 444 * 128 * 3 + 1])
@pytest.mark.parametrize("model", ["sh", "sv", "neural_split"])
def test_decode_on_whole_trips_of_the_persistent_grids(oracle, model, n):
    _check(oracle, model, n)
