"""Pins of the oracle's Spherical Voronoi residual (Eq. 3, App. B): facts the definition fixes - the weights
are a softmax (convex combination, a single site or equal colours give a constant), the sites only matter
through their direction, sharp temperatures give the nearest site's colour (the Voronoi partition), the
common-interface identity of App. B - numpy evaluated by hand, and finite differences of every gradient."""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes


def _scene(n=60, seed=4):
    sc, dirs, gcol = scenes.config5(n, scenes.APP_SV)
    return sc, dirs, gcol


def _residual(oracle, sc, dirs):
    return oracle.appearance_forward(sc, dirs)[1]


def test_matches_the_definition_written_out_in_numpy(oracle):
    sc, dirs, _ = _scene()
    S = sc.sv_sites.astype(np.float64)
    a, raw, t = S[:, :, 0:3], S[:, :, 3:6], S[:, :, 6]
    s = raw / np.linalg.norm(raw, axis=2, keepdims=True)
    rho = np.linalg.norm(s - dirs[:, None, :], axis=2)
    logit = -np.exp(t) * rho
    w = np.exp(logit - logit.max(1, keepdims=True)); w /= w.sum(1, keepdims=True)
    want = (w[:, :, None] * a).sum(1)
    got = _residual(oracle, sc, dirs)
    assert np.abs(got - want).max() < 1e-14
    col = oracle.appearance_forward(sc, dirs)[0]
    assert np.abs(col - np.maximum(sc.base_color.astype(np.float64) + 0.5 + want, 0)).max() < 1e-14


def test_convex_combination_and_constant_cases(oracle):
    sc, dirs, _ = _scene()
    a = sc.sv_sites[:, :, 0:3].astype(np.float64)
    A = _residual(oracle, sc, dirs)
    assert np.all(A <= a.max(1) + 1e-12) and np.all(A >= a.min(1) - 1e-12)       # weights >= 0 and sum to one
    # equal site colours: the residual is that colour whatever the direction (a single effective site)
    sc.sv_sites[:, :, 0:3] = sc.sv_sites[:, :1, 0:3]
    assert np.abs(_residual(oracle, sc, dirs) - sc.sv_sites[:, 0, 0:3]).max() < 1e-12
    # App. B: sum_i w_i (c0 + a_i) = c0 + A: shifting every site colour by c moves the residual by c
    sc2, dirs2, _ = _scene()
    A0 = _residual(oracle, sc2, dirs2)
    sc2.sv_sites[:, :, 0:3] += np.float32(0.25)
    assert np.abs(_residual(oracle, sc2, dirs2) - (A0 + 0.25)).max() < 1e-6


def test_sites_matter_through_their_direction_only(oracle):
    sc, dirs, _ = _scene()
    A0 = _residual(oracle, sc, dirs)
    sc.sv_sites[:, :, 3:6] *= np.float32(4.0)              # exact in fp32: same normalised sites
    assert np.abs(_residual(oracle, sc, dirs) - A0).max() < 1e-12


def test_sharp_temperatures_give_the_voronoi_partition(oracle):
    sc, dirs, _ = _scene(200)
    sc.sv_sites[:, :, 6] = np.float32(6.0)                 # tau = e^6: the softmax is all but a hard arg-min
    S = sc.sv_sites.astype(np.float64)
    s = S[:, :, 3:6] / np.linalg.norm(S[:, :, 3:6], axis=2, keepdims=True)
    rho = np.linalg.norm(s - dirs[:, None, :], axis=2)
    order = np.sort(rho, 1)
    clear = order[:, 1] - order[:, 0] > 0.05              # a clear nearest site
    nearest = S[np.arange(len(S)), rho.argmin(1), 0:3]
    assert clear.sum() > 100
    assert np.abs(_residual(oracle, sc, dirs) - nearest)[clear].max() < 1e-6


def test_gradients_by_finite_differences(oracle):
    sc, dirs, gcol = _scene(25)
    out = oracle.appearance_backward(sc, dirs, gcol)

    def loss(scene, d):
        return float((oracle.appearance_forward(scene, d)[0] * gcol).sum())

    h = 1e-6
    S0 = sc.sv_sites.astype(np.float64)
    rng = np.random.default_rng(0)
    for _ in range(60):                                     # random site parameters
        i, k, p = rng.integers(25), rng.integers(7), rng.integers(7)
        vals = []
        for sgn in (+1, -1):
            S = S0.copy(); S[i, k, p] += sgn * h
            sc.sv_sites = S
            vals.append(loss(sc, dirs))
        fd = (vals[0] - vals[1]) / (2 * h)
        assert abs(fd - out.sv_sites[i, k, p]) < 1e-6 * max(1.0, abs(fd)), (i, k, p, fd, out.sv_sites[i, k, p])
    sc.sv_sites = S0
    for _ in range(20):                                     # the direction, as a free vector
        i, c = rng.integers(25), rng.integers(3)
        vals = []
        for sgn in (+1, -1):
            d = dirs.astype(np.float64).copy(); d[i, c] += sgn * h
            vals.append(loss(sc, d))
        fd = (vals[0] - vals[1]) / (2 * h)
        assert abs(fd - out.dirs[i, c]) < 1e-6 * max(1.0, abs(fd))
    # a site's gradient has no component along the site (only its direction matters)
    raw = S0[:, :, 3:6]
    assert np.abs((out.sv_sites[:, :, 3:6] * raw).sum(2)).max() < 1e-12


def test_degree_zero_disables_the_residual(oracle):
    sc, dirs, gcol = _scene(10)
    sc.active_degree = 0
    col, A = oracle.appearance_forward(sc, dirs)
    assert not A.any() and np.allclose(col, np.maximum(sc.base_color.astype(np.float64) + 0.5, 0))
    out = oracle.appearance_backward(sc, dirs, gcol)
    assert not out.sv_sites.any() and not out.dirs.any()
