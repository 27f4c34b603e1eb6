"""Pins for the oracle outputs that set the tolerances of the GPU parity tests: `fragile`, `fragile_pos`, the ghost
records, `abs_sum` and `flip_sum`.  A mistake that inflates any of them would silently loosen every image and
gradient comparison, so each is fixed here on hand-built pixels: the pair that sits near a threshold of the blend
rule (alpha = 1/255, T (1 - alpha) = 1e-4, raw alpha = 0.99) is placed there on purpose, which entries are flagged
and which are ghosts is written down as literals, and the sums of |terms| are formed by the few lines of numpy
below from the definition of the blend backward.

Windows under test: |255 alpha - 1| < 1e-4, |T (1 - alpha) - 1e-4| < 1e-8, |raw - 0.99| < 0.99e-4.
"""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes


def _cam(w=1, h=1, bg=(0.0, 0.0, 0.0)):
    return scenes.identity_camera(w, h, 8.0, background=bg)


def _centred(alphas, colors=None):
    """Gaussians centred on pixel (0, 0) of a one-tile image: the falloff is exp(0) = 1 there, so the pair's raw
    alpha IS the opacity, to the last bit."""
    n = len(alphas)
    mean2d = np.full((n, 2), 0.5)
    conic = np.tile([1.0, 0.0, 1.0], (n, 1))
    color = np.tile([0.2, 0.5, 0.8], (n, 1)) if colors is None else np.asarray(colors, np.float64)
    return mean2d, conic, np.asarray(alphas, np.float64), color


def _forward(oracle, cam, mean2d, conic, opacity, color):
    n = len(opacity)
    ranges = np.zeros((((cam.width + 15) // 16) * ((cam.height + 15) // 16), 2), np.uint32)
    ranges[0] = (0, n)
    return oracle.blend_forward(cam, np.arange(n, dtype=np.uint32), ranges, mean2d, conic, opacity, color), ranges


# ---------------------------------------------------------------------------------------- fragile, fragile_pos

@pytest.mark.parametrize("delta,fragile,composited", [(+5e-5, True, True), (-5e-5, True, False),
                                                      (+5e-4, False, True), (-5e-4, False, False)])
def test_fragile_window_at_the_alpha_threshold(oracle, delta, fragile, composited):
    a = (1.0 + delta) / 255.0
    cam = _cam()
    fwd, _ = _forward(oracle, cam, *_centred([0.3, 0.2, a, 0.4]))
    assert bool(fwd.fragile[0, 0]) == fragile
    assert fwd.fragile_pos[0, 0] == (2 if fragile else -1)
    T = 0.7 * 0.8 * ((1 - a) if composited else 1.0) * 0.6
    assert fwd.final_T[0, 0] == pytest.approx(T, rel=1e-14)
    assert fwd.n_contrib[0, 0] == 4


@pytest.mark.parametrize("delta,fragile", [(+5e-9, True), (-5e-9, True), (+5e-8, False), (-5e-8, False)])
def test_fragile_window_at_the_transmittance_stop(oracle, delta, fragile):
    T3 = (1.0 * (1.0 - 0.9)) * (1.0 - 0.9) * (1.0 - 0.9)      # after three entries of alpha 0.9
    a4 = 1.0 - (1e-4 + delta) / T3
    cam = _cam()
    fwd, _ = _forward(oracle, cam, *_centred([0.9, 0.9, 0.9, a4, 0.5]))
    assert bool(fwd.fragile[0, 0]) == fragile
    assert fwd.fragile_pos[0, 0] == (3 if fragile else -1)
    # the stop itself follows the plain rule: the fourth entry is composited iff T (1 - alpha) >= 1e-4
    assert fwd.n_contrib[0, 0] == (4 if delta > 0 else 3)       # the 0.5 behind it always stops


@pytest.mark.parametrize("delta,fragile", [(+5e-5, True), (-5e-5, True), (+5e-4, False), (-5e-4, False)])
def test_fragile_window_at_the_alpha_clamp(oracle, delta, fragile):
    cam = _cam()
    fwd, _ = _forward(oracle, cam, *_centred([0.25, 0.99 * (1.0 + delta), 0.5]))
    assert bool(fwd.fragile[0, 0]) == fragile
    assert fwd.fragile_pos[0, 0] == (1 if fragile else -1)
    a = min(0.99, 0.99 * (1.0 + delta))
    assert fwd.final_T[0, 0] == pytest.approx(0.75 * (1 - a) * 0.5, rel=1e-13)


def test_fragile_pos_is_the_first_flagged_position_and_other_pixels_stay_clean(oracle):
    # two pairs near thresholds in pixel (0, 0): positions 1 and 3; pixel (1, 0) sees other alphas and is clean
    cam = _cam(2, 1)
    m, q, o, c = _centred([0.3, (1 + 2e-5) / 255, 0.2, 0.99 * (1 - 1e-5), 0.1])
    fwd, _ = _forward(oracle, cam, m, q, o, c)
    assert fwd.fragile[0, 0] == 1 and fwd.fragile_pos[0, 0] == 1
    assert fwd.fragile[0, 1] == 0 and fwd.fragile_pos[0, 1] == -1


# ---------------------------------------------------------------------------------------- ghost records

def test_no_ghost_without_a_near_threshold_pair(oracle):
    m, q, o, c = _centred([0.3, 0.001, 0.2, 0.995, 0.4])      # one skipped pair, one clamped pair, none near
    r = oracle.blend_pixel_records(0.5, 0.5, np.arange(5), m, q, o, c)
    assert r.pos.tolist() == [0, 2, 3, 4] and r.ghost.tolist() == [0, 0, 0, 0]
    assert r.clamped.tolist() == [0, 0, 1, 0]
    assert r.alpha.tolist() == [0.3, 0.2, 0.99, 0.4]
    assert np.allclose(r.T, [1.0, 0.7, 0.56, 0.0056], rtol=1e-14)


def test_ghost_of_a_pair_just_below_the_alpha_threshold(oracle):
    a = (1 - 5e-5) / 255
    m, q, o, c = _centred([0.3, a, 0.2])
    r = oracle.blend_pixel_records(0.5, 0.5, np.arange(3), m, q, o, c)
    assert r.pos.tolist() == [0, 1, 2] and r.ghost.tolist() == [0, 1, 0]
    assert r.alpha[1] == a and r.T[1] == pytest.approx(0.7, rel=1e-15)
    assert r.T[2] == pytest.approx(0.7, rel=1e-15)            # the ghost did not dim what lies behind it
    # 5e-4 below: outside the window, no record at all
    m, q, o, c = _centred([0.3, (1 - 5e-4) / 255, 0.2])
    r = oracle.blend_pixel_records(0.5, 0.5, np.arange(3), m, q, o, c)
    assert r.pos.tolist() == [0, 2] and r.ghost.tolist() == [0, 0]


def test_ghosts_of_a_stop_within_the_window(oracle):
    T3 = (1.0 * (1.0 - 0.9)) * (1.0 - 0.9) * (1.0 - 0.9)
    a4 = 1.0 - (1e-4 - 5e-9) / T3
    m, q, o, c = _centred([0.9, 0.9, 0.9, a4, 0.5, 0.5])
    r = oracle.blend_pixel_records(0.5, 0.5, np.arange(6), m, q, o, c)
    # the stopping pair is the one ghost: behind it 0.5 takes the transmittance to 5e-5, clearly below the window
    assert r.pos.tolist() == [0, 1, 2, 3] and r.ghost.tolist() == [0, 0, 0, 1]
    assert r.alpha[3] == a4 and r.T[3] == pytest.approx(T3, rel=1e-15)
    # a pair behind it that keeps the transmittance inside the window is walked over as a ghost too
    a4 = 1.0 - (1e-4 - 1e-10) / T3
    tiny = 4e-3                                                # >= 1/255, so it is evaluated ...
    m, q, o, c = _centred([0.9, 0.9, 0.9, a4, tiny, 0.5])
    r = oracle.blend_pixel_records(0.5, 0.5, np.arange(6), m, q, o, c)
    assert (1e-4 - 1e-10) * (1 - tiny) < 1e-4 - 1e-8          # ... it leaves the window, so the chain ends at once
    assert r.pos.tolist() == [0, 1, 2, 3] and r.ghost.tolist() == [0, 0, 0, 1]
    # 5e-8 below the threshold: a plain stop, no ghost
    a4 = 1.0 - (1e-4 - 5e-8) / T3
    m, q, o, c = _centred([0.9, 0.9, 0.9, a4, 0.5])
    r = oracle.blend_pixel_records(0.5, 0.5, np.arange(5), m, q, o, c)
    assert r.pos.tolist() == [0, 1, 2] and r.ghost.tolist() == [0, 0, 0]


# ---------------------------------------------------------------------------------------- abs_sum, flip_sum

def _pixel_terms(px, py, rows, G, bg, ghosts=(), flip_from=None, flip_clamped=()):
    """The nine per-Gaussian terms (colour 3, opacity, conic A B C, mean u v) one pixel sends to each entry of
    `rows` = [(mean, (A, B, C), opacity, colour)], from the definition of the blend backward: with T_i the
    transmittance in front of entry i and S_i the light arriving from behind it,
      d/dcolour = alpha T G,  d/dalpha = G . (T c - S / (1 - alpha)),  d/dopacity = exp(power) d/dalpha,
      d/dpower = alpha d/dalpha,  d/d(A, B, C) = (-dx^2/2, -dx dy, -dy^2/2) d/dpower,
      d/d(u, v) = (A dx + B dy, B dx + C dy) d/dpower; a clamped alpha passes nothing to opacity and power.
    `ghosts`: positions the plain rule leaves out (they enter neither T nor S) but whose would-be terms count for
    the flip allowance; `flip_from`: first flagged position; `flip_clamped`: clamped entries whose clamp is within
    the window.  Returns (terms [n,9] of the composited entries, |terms| [n,9], flip [n,9])."""
    n = len(rows)
    alpha, T, power, clamped, comp = np.zeros(n), np.zeros(n), np.zeros(n), np.zeros(n, bool), np.zeros(n, bool)
    t = 1.0
    for i, (mean, (A, B, C), o, col) in enumerate(rows):
        dx, dy = px - mean[0], py - mean[1]
        power[i] = -0.5 * (A * dx * dx + C * dy * dy) - B * dx * dy
        raw = o * np.exp(power[i])
        alpha[i], clamped[i], T[i] = min(0.99, raw), raw > 0.99, t
        if i in ghosts or alpha[i] < 1 / 255:
            continue
        if t * (1 - alpha[i]) < 1e-4:
            break
        comp[i] = True
        t *= 1 - alpha[i]
    S = t * np.asarray(bg, np.float64)
    terms, flip = np.zeros((n, 9)), np.zeros((n, 9))
    for i in range(n - 1, -1, -1):
        if not (comp[i] or i in ghosts):
            continue
        mean, (A, B, C), o, col = rows[i]
        col = np.asarray(col, np.float64)
        dx, dy = px - mean[0], py - mean[1]
        v = np.zeros(9)
        v[0:3] = alpha[i] * T[i] * G
        dalpha = float(G @ (T[i] * col - S / (1 - alpha[i])))
        dpower = alpha[i] * dalpha
        geo = np.array([np.exp(power[i]) * dalpha, -0.5 * dx * dx * dpower, -dx * dy * dpower, -0.5 * dy * dy * dpower,
                        dpower * (A * dx + B * dy), dpower * (B * dx + C * dy)])
        real = v.copy()
        if not clamped[i]:
            v[3:] = geo; real[3:] = geo
        elif i in flip_clamped:
            v[3:] = geo                                      # fp32 might not clamp: allowance only
        if comp[i]:
            terms[i] = real
            S = S + col * alpha[i] * T[i]
        if flip_from is not None and i >= flip_from:
            flip[i] = np.abs(v)
    return terms, np.abs(terms), flip


def _rows_for(alphas_at_00, offsets, colors):
    """Three-entry list with off-centre means; opacities chosen so that pixel (0,0) sees exactly `alphas_at_00`."""
    rows = []
    conics = [(0.9, 0.2, 0.7), (0.5, -0.1, 0.6), (0.3, 0.05, 0.4)]
    for a, off, col, q in zip(alphas_at_00, offsets, colors, conics):
        mean = (0.5 - off[0], 0.5 - off[1])
        power = -0.5 * (q[0] * off[0] ** 2 + q[2] * off[1] ** 2) - q[1] * off[0] * off[1]
        rows.append((mean, q, a / np.exp(power), col))
    return rows


def _backward(oracle, cam, rows, G):
    mean2d = np.array([r[0] for r in rows]); conic = np.array([r[1] for r in rows])
    opacity = np.array([r[2] for r in rows]); color = np.array([r[3] for r in rows])
    fwd, ranges = _forward(oracle, cam, mean2d, conic, opacity, color)
    g = oracle.blend_backward(cam, np.arange(len(rows), dtype=np.uint32), ranges, mean2d, conic, opacity, color, G,
                              with_abs=True)
    got = np.concatenate([g.color, g.opacity[:, None], g.conic, g.mean2d], 1)
    return fwd, got, g.abs_sum, g.flip_sum


COLORS = [(0.9, 0.1, 0.3), (0.2, 0.7, 0.4), (0.5, 0.5, 0.1)]
OFFSETS = [(0.6, -0.4), (-0.8, 0.3), (0.2, 0.9)]


def test_abs_sum_is_the_sum_of_absolute_terms_and_flip_sum_is_zero_without_a_near_pair(oracle):
    cam = _cam(3, 2, bg=(0.3, 0.1, 0.6))
    rng = np.random.default_rng(5)
    G = rng.standard_normal((3, 2, 3))
    rows = _rows_for([0.45, 0.3, 0.6], OFFSETS, COLORS)
    fwd, got, abs_sum, flip_sum = _backward(oracle, cam, rows, G)
    assert fwd.fragile.sum() == 0
    want, want_abs = np.zeros((3, 9)), np.zeros((3, 9))
    for y in range(2):
        for x in range(3):
            t, a, _ = _pixel_terms(x + 0.5, y + 0.5, rows, G[:, y, x], cam.background)
            want += t; want_abs += a
    assert np.allclose(got, want, rtol=1e-12, atol=1e-15)
    assert np.allclose(abs_sum, want_abs, rtol=1e-12, atol=1e-15)
    assert np.all(abs_sum >= np.abs(got) - 1e-15) and (abs_sum > np.abs(got) * 1.01).any()   # signs do cancel here
    assert np.all(flip_sum == 0)


@pytest.mark.parametrize("case", ["alpha_above", "alpha_below_ghost", "clamp_above", "clamp_below"])
def test_flip_sum_counts_the_flagged_pair_and_everything_behind_it_in_that_pixel_only(oracle, case):
    cam = _cam(3, 2, bg=(0.3, 0.1, 0.6))
    rng = np.random.default_rng(6)
    G = rng.standard_normal((3, 2, 3))
    mid = {"alpha_above": (1 + 5e-5) / 255, "alpha_below_ghost": (1 - 5e-5) / 255,
           "clamp_above": 0.99 * (1 + 5e-5), "clamp_below": 0.99 * (1 - 5e-5)}[case]
    rows = _rows_for([0.45, mid, 0.6], OFFSETS, COLORS)       # position 1 of pixel (0, 0) sits near a threshold
    fwd, got, abs_sum, flip_sum = _backward(oracle, cam, rows, G)
    assert fwd.fragile.sum() == 1 and fwd.fragile[0, 0] == 1 and fwd.fragile_pos[0, 0] == 1
    want, want_abs, want_flip = np.zeros((3, 9)), np.zeros((3, 9)), np.zeros((3, 9))
    for y in range(2):
        for x in range(3):
            flagged = (x, y) == (0, 0)
            t, a, f = _pixel_terms(x + 0.5, y + 0.5, rows, G[:, y, x], cam.background,
                                   ghosts=(1,) if flagged and case == "alpha_below_ghost" else (),
                                   flip_from=1 if flagged else None,
                                   flip_clamped=(1,) if flagged and case == "clamp_above" else ())
            want += t; want_abs += a; want_flip += f
    assert np.allclose(got, want, rtol=1e-12, atol=1e-15)
    assert np.allclose(abs_sum, want_abs, rtol=1e-12, atol=1e-15)
    assert np.allclose(flip_sum, want_flip, rtol=1e-12, atol=1e-18)
    assert np.all(flip_sum[0] == 0)                           # the entry in front of the flagged pair is safe
    assert flip_sum[1, :3].min() > 0 and flip_sum[2, :3].min() > 0
    assert flip_sum[1, 3] > 0       # also where the pair is clamped in double: fp32 might not clamp, so its opacity
                                    # and conic terms belong to the allowance although they are not in the gradient


def test_flip_sum_of_a_stop_within_the_window(oracle):
    cam = _cam()
    T3 = (1.0 * (1.0 - 0.9)) * (1.0 - 0.9) * (1.0 - 0.9)
    a4 = 1.0 - (1e-4 - 5e-9) / T3
    alphas = [0.9, 0.9, 0.9, a4, 0.5]
    cols = [(0.9, 0.1, 0.3), (0.2, 0.7, 0.4), (0.5, 0.5, 0.1), (0.3, 0.3, 0.9), (0.6, 0.2, 0.2)]
    rows = [((0.5, 0.5), (1.0, 0.0, 1.0), a, c) for a, c in zip(alphas, cols)]
    G = np.array([0.7, -1.1, 0.4]).reshape(3, 1, 1)
    fwd, got, abs_sum, flip_sum = _backward(oracle, cam, rows, G)
    assert fwd.fragile[0, 0] == 1 and fwd.fragile_pos[0, 0] == 3 and fwd.n_contrib[0, 0] == 3
    # the plain rule stopped at position 3: the three entries in front of it are all there is
    t, a, _ = _pixel_terms(0.5, 0.5, rows[:3], G[:, 0, 0], cam.background)
    assert np.allclose(got[:3], t, rtol=1e-12, atol=1e-18) and np.allclose(abs_sum[:3], a, rtol=1e-12, atol=1e-18)
    assert np.all(got[3:] == 0) and np.all(abs_sum[3:] == 0)
    # entries 0..2 are in front of the flagged pair: no allowance; the stopping pair gets its would-be terms
    assert np.all(flip_sum[:3] == 0) and np.all(flip_sum[4] == 0)
    want = np.zeros(9)
    S = fwd.final_T[0, 0] * np.asarray(cam.background, np.float64)
    want[0:3] = np.abs(a4 * T3 * G[:, 0, 0])
    want[3] = abs(float(G[:, 0, 0] @ (T3 * np.asarray(cols[3]) - S / (1 - a4))))
    assert np.allclose(flip_sum[3], want, rtol=1e-12, atol=1e-18)


# ---------------------------------------------------------------------------------------- ReLU margin of the decoder

def test_kink_margin_is_the_smallest_hidden_pre_activation(oracle):
    """Hand-set weights: with f = 0 the input cos f_0 is exactly 1, W1 routes it to hidden unit o with gain
    0.1 (o + 1), W2 is diagonal with one negative and one small entry.  The 32 pre-activations are then known in
    closed form; the margin is the smallest of their absolute values.  Degree 0 disables the residual: no decision."""
    n = 3
    w = np.zeros(816)
    for o in range(16):
        w[o * 32 + 17] = 0.1 * (o + 1)                  # W1[o][cos f_0]
        w[512 + o * 16 + o] = 1.0                       # W2 diagonal
    w[512 + 3 * 16 + 3] = -0.5                          # unit 3 of layer 2: pre-activation -0.5 * 0.4 = -0.2
    w[512 + 5 * 16 + 5] = 0.01                          # unit 5 of layer 2: 0.01 * 0.6 = 0.006, the smallest
    sc = scenes.Scene(np.zeros((n, 3), np.float32), np.zeros((n, 3), np.float32), np.zeros((n, 4), np.float32),
                      np.zeros(n, np.float32), np.zeros((n, 3), np.float32), app=scenes.APP_NEURAL, active_degree=3,
                      features=np.zeros((n, 8)), mlp_weights=w)
    d = np.array([[0.0, 0.0, 1.0], [1.0, 0.0, 0.0], [0.6, 0.0, 0.8]])
    m = oracle.mlp_kink_margin(sc, d)
    assert np.allclose(m, 0.006, rtol=1e-13)
    w[512 + 5 * 16 + 5] = 1.0
    assert np.allclose(oracle.mlp_kink_margin(sc, d), 0.1, rtol=1e-13)       # now the first unit of layer 1
    w[7 * 32 + 17] = -3e-7                                                    # a unit just below its kink
    m = oracle.mlp_kink_margin(sc, d)
    assert np.allclose(m, 0.0, atol=3.1e-7) and np.all(m <= 3e-7)           # layer 2 sees relu(-3e-7) = 0 there
    assert np.all(np.isinf(oracle.mlp_kink_margin(sc, d, deg=0)))
