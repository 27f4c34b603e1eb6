"""Pins of the oracle's decoder with the architecture as a parameter (App. D, architecture table): the MAC
counts the paper prints for every configuration, agreement with the fixed-size decoder (an independent second
statement of Eq. 5-7) for the default architecture, numpy matrix products, and finite differences."""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes

VARIANTS = [(16, 1, 8), (16, 3, 8), (32, 2, 8), (16, 2, 16), (16, 2, 8)]


def test_mac_counts_of_the_architecture_table(oracle):
    # MAC/G as the viewer evaluates the model: the first layer is folded wherever that pays off (16 neurons)
    assert oracle.decoder_macs(16, 1, True) == 304
    assert oracle.decoder_macs(16, 3, True) == 816
    assert oracle.decoder_macs(32, 2, False) == 2144          # "lists the full count": folding would double the payload
    assert oracle.decoder_macs(16, 2, True) == 560            # the default, and F = 16 without frequency encoding
    assert oracle.decoder_macs(16, 2, False) == 816 == oracle.decoder_num_weights(16, 2)
    assert oracle.decoder_num_weights(32, 2) == 2144 and oracle.decoder_num_weights(16, 1) == 560


def test_default_architecture_equals_the_fixed_size_decoder(oracle):
    sc, dirs, gcol = scenes.config5(300, scenes.APP_NEURAL)
    sc.features = np.random.default_rng(2).normal(0, 0.7, sc.features.shape).astype(np.float16)
    for deg in (0, 1, 3):
        a = oracle.appearance_forward(sc, dirs, deg=deg)[0]
        b = oracle.decoder_forward(sc, dirs, deg=deg)
        assert np.abs(a - b).max() < 1e-14
        ga, gb = oracle.appearance_backward(sc, dirs, gcol, deg=deg), oracle.decoder_backward(sc, dirs, gcol, deg=deg)
        for nm in ("base_color", "features", "mlp_weights", "dirs"):
            assert np.abs(getattr(ga, nm) - getattr(gb, nm)).max() < 1e-12, nm


@pytest.mark.parametrize("hidden,layers,nfeat", VARIANTS)
def test_forward_is_the_chain_of_matrix_products(oracle, hidden, layers, nfeat):
    sc, dirs, _ = scenes.decoder_variant(64, hidden, layers, nfeat)
    W = sc.mlp_weights.astype(np.float64)
    assert len(W) == oracle.decoder_num_weights(hidden, layers)
    Y = np.stack([oracle.sh_basis(d) for d in dirs])
    f = sc.features.astype(np.float64)
    enc = np.stack([np.sin(f), np.cos(f)], 2).reshape(len(f), 16) if nfeat == 8 else f
    h = np.concatenate([Y, enc], 1)
    off, nin = 0, 32
    for _ in range(layers):
        h = np.maximum(h @ W[off:off + hidden * nin].reshape(hidden, nin).T, 0)
        off += hidden * nin; nin = hidden
    A = np.tanh(h @ W[off:].reshape(3, hidden).T)
    want = np.maximum(sc.base_color.astype(np.float64) + 0.5 + A, 0)
    assert np.abs(oracle.decoder_forward(sc, dirs) - want).max() < 1e-13


@pytest.mark.parametrize("hidden,layers,nfeat", VARIANTS[:4])
def test_gradients_by_finite_differences(oracle, hidden, layers, nfeat):
    sc, dirs, gcol = scenes.decoder_variant(12, hidden, layers, nfeat)
    sc.features = np.random.default_rng(3).normal(0, 0.5, sc.features.shape).astype(np.float16)
    out = oracle.decoder_backward(sc, dirs, gcol)

    def loss():
        return float((oracle.decoder_forward(sc, dirs) * gcol).sum())

    h = 1e-6
    rng = np.random.default_rng(4)
    W0 = sc.mlp_weights.astype(np.float64)
    for k in rng.choice(len(W0), 40, replace=False):
        vals = []
        for sgn in (+1, -1):
            W = W0.copy(); W[k] += sgn * h
            sc.mlp_weights = W
            vals.append(loss())
        fd = (vals[0] - vals[1]) / (2 * h)
        assert abs(fd - out.mlp_weights[k]) < 2e-6 * max(1.0, abs(fd)), k
    sc.mlp_weights = W0
    F0 = sc.features.astype(np.float64)
    for _ in range(20):
        i, j = rng.integers(12), rng.integers(nfeat)
        vals = []
        for sgn in (+1, -1):
            F = F0.copy(); F[i, j] += sgn * h
            sc.features = F
            vals.append(loss())
        fd = (vals[0] - vals[1]) / (2 * h)
        assert abs(fd - out.features[i, j]) < 2e-6 * max(1.0, abs(fd))
    sc.features = F0
    d0 = dirs.astype(np.float64)
    for _ in range(10):
        i, c = rng.integers(12), rng.integers(3)
        vals = []
        for sgn in (+1, -1):
            d = d0.copy(); d[i, c] += sgn * h
            vals.append(float((oracle.decoder_forward(sc, d) * gcol).sum()))
        fd = (vals[0] - vals[1]) / (2 * h)
        assert abs(fd - out.dirs[i, c]) < 2e-6 * max(1.0, abs(fd))


@pytest.mark.parametrize("arch", [(32, 1, 16), (16, 3, 8)], ids=lambda a: "h%d_l%d_f%d" % a)
def test_whole_step_with_a_variant_against_finite_differences(oracle, arch):
    """The oracle's rendering step composes projection, appearance and blend; with a decoder of another size the
    composition calls the generic decoder.  Central differences of the image loss pin that composition: features,
    decoder weights and means (whose gradient carries the direction term of the decoder)."""
    import test_oracle_gradients as og
    hidden, layers, nfeat = arch
    sc = og.tiny_scene(1, seed=31)
    rng = np.random.default_rng(77)
    sc.features = rng.normal(0, 0.7, (sc.means.shape[0], nfeat))
    sc.mlp_weights = rng.uniform(-0.6, 0.6, oracle.decoder_num_weights(hidden, layers))
    sc.mlp_hidden, sc.mlp_layers = hidden, layers
    cam = og.tiny_cam(None)
    G = np.random.default_rng(98).standard_normal((3, cam.height, cam.width))
    fwd, grads = oracle.render(sc, cam, G)
    assert fwd.pre.visible.sum() >= 10
    assert grads.features.shape == (sc.means.shape[0], nfeat)
    assert grads.mlp_weights.shape == (oracle.decoder_num_weights(hidden, layers),)
    for name, stride in (("features", 1), ("mlp_weights", 7), ("means", 1), ("base_color", 1)):
        checked, skipped, bad, worst, gmax = og.fd_check(oracle, sc, cam, G, [name], stride=stride)[name]
        assert gmax > 1e-3, (name, gmax)
        assert bad == 0, (name, checked, skipped, bad, worst)
        assert skipped <= 0.1 * (checked + skipped), (name, checked, skipped)
