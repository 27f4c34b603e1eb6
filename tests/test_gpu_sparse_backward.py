"""The preprocess backward of the neural model spends arithmetic only on the Gaussians that received a gradient
(k_bwd_flags + k_preprocess_bwd_sparse): the others - culled, or listed in tiles but composited by no pixel - get
exact zeros.  Checked here: an upstream gradient that is zero outside a small window, so that almost every visible
Gaussian is skipped and the few that are not fill less than one batch per CTA; an upstream gradient that is zero
everywhere; a visible Gaussian with a zero gradient and non-finite appearance parameters; sizes around the batch and
flag-word boundaries (128 Gaussians per batch, 32 per flag word, 4096 per scan round); the same through the unfused
path, whose projection-only backward uses the same two kernels.  Every case against the oracle by the literal rule,
with exact zeros where the oracle has zeros."""
import copy

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from gpu_helpers import grad_mismatch, grad_names, run_gpu

pytestmark = pytest.mark.gpu


def _window_gradient(cam, seed, x0, y0, size):
    G = scenes.upstream_gradient(cam, seed)
    W = np.zeros_like(G)
    W[:, y0:y0 + size, x0:x0 + size] = G[:, y0:y0 + size, x0:x0 + size]
    return W


def _check(oracle, sc, cam, G, allow=0.002):
    gpu = run_gpu(sc, cam, G)
    fwd, ref = oracle.render(sc, cam, G)
    skipped = 0
    for nm in grad_names(sc.app):
        got, want = getattr(gpu.grads, nm), getattr(ref, nm)
        assert np.all(np.isfinite(got)), nm
        if nm != "mlp_weights":
            zero_rows = ~np.asarray(want != 0).reshape(len(want), -1).any(1)
            assert np.all(np.asarray(got).reshape(len(got), -1)[zero_rows] == 0), nm     # exact zeros, not small numbers
            skipped = max(skipped, int(zero_rows.sum()))
        bad = grad_mismatch(got, want)
        assert bad.mean() <= allow, (nm, int(bad.sum()))
    return gpu, skipped


@pytest.mark.parametrize("n", [127, 129, 4_095, 4_097, 30_000])
def test_gradient_in_a_small_window(oracle, n):
    w = scenes.config3(scenes.APP_NEURAL, n=n, width=320, height=208, views=1)
    cam = w.cameras[0]
    G = _window_gradient(cam, 3, 150, 90, 24)
    gpu, skipped = _check(oracle, w.scene, cam, G)
    assert skipped > 0.5 * n                                   # most Gaussians took the short way


def test_zero_upstream_gradient_gives_exact_zeros(oracle):
    w = scenes.config3(scenes.APP_NEURAL, n=20_011, width=320, height=208, views=1)
    cam = w.cameras[0]
    gpu = run_gpu(w.scene, cam, np.zeros((3, cam.height, cam.width), np.float32))
    for nm in grad_names(w.scene.app):
        assert np.all(getattr(gpu.grads, nm) == 0), nm


def test_skipped_gaussian_with_non_finite_appearance(oracle):
    """A listed Gaussian that receives no gradient is never decoded: non-finite features leave its row and the
    decoder-weight gradient finite (the forward's colour of that Gaussian is not finite, so it is put where no pixel
    with a gradient sees it)."""
    w = scenes.config3(scenes.APP_NEURAL, n=10_007, width=320, height=208, views=1)
    cam = w.cameras[0]
    G = _window_gradient(cam, 5, 8, 8, 16)
    base = run_gpu(w.scene, cam, G)
    quiet = np.flatnonzero(base.visible & ~np.asarray(base.g2d[:, :9] != 0).any(1))
    assert len(quiet) > 100
    sc = copy.copy(w.scene)
    sc.features = w.scene.features.copy()
    victim = int(quiet[len(quiet) // 2])
    sc.features[victim] = np.float16(np.inf)
    gpu = run_gpu(sc, cam, G)
    if not np.asarray(gpu.g2d[victim, :9] != 0).any():          # still without a gradient (its colour reached no such pixel)
        for nm in grad_names(sc.app):
            assert np.all(np.isfinite(getattr(gpu.grads, nm))), nm
        assert np.all(gpu.grads.features[victim] == 0)


def test_unfused_path_uses_the_same_kernels(oracle):
    w = scenes.config3(scenes.APP_NEURAL, n=12_013, width=320, height=208, views=1)
    cam = w.cameras[0]
    sc = copy.copy(w.scene)
    sc.separate_pass = 1
    _check(oracle, sc, cam, _window_gradient(cam, 7, 100, 60, 40))


@pytest.mark.parametrize("arch", [(16, 1, 8), (16, 3, 8), (32, 2, 8), (16, 2, 16), (32, 3, 16)], ids=lambda a: "h%d_l%d_f%d" % a)
@pytest.mark.parametrize("n", [129, 30_000])
def test_decoder_variants_work_on_the_flagged_gaussians_only(oracle, arch, n):
    """A decoder of another size runs through the step unfused, and its backward (the tcgen05 kernels) gathers the
    Gaussians that received a gradient into tiles of 128: same check, gradient in a small window, rows of 8 and of 16
    features."""
    hidden, layers, nfeat = arch
    w = scenes.config3(scenes.APP_NEURAL, n=n, width=320, height=208, views=1)
    cam = w.cameras[0]
    sc = w.scene
    rng = np.random.default_rng(np.random.PCG64(777))
    _, sc.features, sc.mlp_weights = scenes.draw_neural_appearance(rng, sc.n, hidden, layers, nfeat)
    sc.mlp_hidden, sc.mlp_layers = hidden, layers
    gpu, skipped = _check(oracle, sc, cam, _window_gradient(cam, 3, 150, 90, 24))
    assert skipped > 0.5 * n
    assert gpu.grads.features.shape == (n, nfeat)


def test_decoder_variant_with_a_zero_upstream_gradient(oracle):
    w = scenes.config3(scenes.APP_NEURAL, n=5_003, width=320, height=208, views=1)
    cam = w.cameras[0]
    sc = w.scene
    rng = np.random.default_rng(np.random.PCG64(778))
    _, sc.features, sc.mlp_weights = scenes.draw_neural_appearance(rng, sc.n, 32, 2, 16)
    sc.mlp_hidden, sc.mlp_layers = 32, 2
    gpu = run_gpu(sc, cam, np.zeros((3, cam.height, cam.width), np.float32))
    for nm in grad_names(sc.app):
        assert np.all(getattr(gpu.grads, nm) == 0), nm
