"""Pins of the oracle's viewer-side evaluation of the neural model (App. C.3): the folded first layer
must reproduce the full decoder exactly, costs the 560 multiply-accumulates the paper prints, and its
fp16 storage moves the colour by less than the bound the arithmetic gives."""
import numpy as np

from paper_2609_05255_b200 import scenes


def _scene(n=500, seed=3):
    w = scenes.config2(n=n)
    sc = w.scene
    rng = np.random.default_rng(seed)
    sc.features = rng.normal(0, 0.6, sc.features.shape).astype(np.float16)     # well away from zero
    return sc


def test_folded_evaluation_equals_the_full_decoder(oracle):
    sc = _scene()
    eye = np.array([0.3, -0.2, -1.0])
    d = sc.means.astype(np.float64) - eye
    d /= np.linalg.norm(d, axis=1, keepdims=True)
    for deg in (1, 2, 3):
        full = oracle.appearance_forward(sc, d, deg=deg)
        col = full[0] if isinstance(full, tuple) else full
        pre = oracle.neural_fold(sc)
        got = oracle.neural_prepass(sc, pre, eye, deg=deg)
        assert np.abs(got - col).max() < 1e-12
    # degree 0: no residual at all
    assert np.allclose(oracle.neural_prepass(sc, pre, eye, deg=0), np.maximum(sc.base_color.astype(np.float64) + 0.5, 0))


def test_pre_activations_are_the_seventeen_view_independent_columns(oracle):
    sc = _scene(50)
    W1 = sc.mlp_weights[:512].astype(np.float64).reshape(16, 32)
    f = sc.features.astype(np.float64)
    enc = np.stack([np.sin(f), np.cos(f)], 2).reshape(len(f), 16)        # (sin f_j, cos f_j) interleaved
    want = 0.5 / np.sqrt(np.pi) * W1[:, 0][None] + enc @ W1[:, 16:].T
    assert np.abs(oracle.neural_fold(sc) - want).max() < 1e-13
    # what is left per frame: 15 direction columns padded to 16, then the two later layers (printed: 560)
    assert 16 * 16 + 16 * 16 + 16 * 3 == 560 == oracle.mlp_macs(True) and oracle.mlp_macs(False) == 816


def test_half_precision_storage_moves_the_colour_within_its_bound(oracle):
    sc = _scene()
    eye = np.zeros(3)
    pre = oracle.neural_fold(sc)
    exact = oracle.neural_prepass(sc, pre, eye)
    rounded = oracle.neural_prepass(sc, pre.astype(np.float16).astype(np.float64), eye)
    # |d pre| <= 2^-11 |pre|; two ReLU layers and tanh are 1-Lipschitz, so the colour moves by at most
    # ||W3|| ||W2|| times the norm of the perturbation
    W = sc.mlp_weights.astype(np.float64)
    W2, W3 = W[512:768].reshape(16, 16), W[768:].reshape(3, 16)
    bound = np.linalg.norm(W3, 2) * np.linalg.norm(W2, 2) * np.linalg.norm(pre * 2.0 ** -11, axis=1)
    assert np.all(np.abs(rounded - exact).max(1) <= bound + 1e-15)
    assert np.abs(rounded - exact).max() < 2e-3
    # and the 8-bit texel rarely notices
    a, b = oracle.rgba8(exact, np.full(len(exact), 0.5)), oracle.rgba8(rounded, np.full(len(exact), 0.5))
    assert np.abs(a.astype(int) - b.astype(int)).max() <= 1 and (a != b).mean() < 0.05
    assert np.all(a[:, 3] == 128)


def test_rgba8_rounds_to_nearest_and_saturates(oracle):
    c = np.array([[0.0, 1.0, 2.5], [0.5, 0.25, 0.999], [1 / 510 - 1e-9, 1 / 510 + 1e-9, -0.1]])
    got = oracle.rgba8(c, np.array([0.0, 1.0, 0.5]))
    assert got.tolist() == [[0, 255, 255, 0], [128, 64, 255, 255], [0, 1, 0, 128]]
