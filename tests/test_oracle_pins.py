"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with a retyped copy of itself: each
uses a closed form (logistic / hyperbolic functions for 2- and 3-level
alphabets, binary entropy), an identity (Proposition 1), a limit (the Remark
of Sec. IV-A), finite differences of Q_d built from the CPMF (Lemma 1 and the
derived alpha- and rate-derivatives), a brute-force search on tiny inputs, or
a library routine (numpy integer matmul).
"""
import math

import numpy as np
import pytest

import oracle
from paper_2501_09849_b200 import inputs

# Parameter grid of Figs. 1-2: b = 3 (levels -4..3), q = 0.1, alpha in {100, 300, 500, 700}.
FIG_Q, FIG_LO, FIG_HI = 0.1, -4, 3
FIG_ALPHAS = (100.0, 300.0, 500.0, 700.0)

f32 = np.float32


def qd_from_cpmf(theta, q, lo, hi, alpha, window=0):
    """Q_d assembled outside the oracle's soft(): sum of CPMF times levels, double inputs."""
    P = oracle.cpmf(theta, q, lo, hi, alpha, window)
    return float(np.dot(P, np.arange(lo, hi + 1, dtype=np.float64) * q))


# ------------------------------------------------------------------ CPMF (Sec. IV-A, Eq. (4))
@pytest.mark.parametrize("alpha", FIG_ALPHAS + (1.0, 1e4))
def test_cpmf_is_a_distribution(alpha):
    for theta in np.linspace(-0.6, 0.5, 23):
        P = oracle.cpmf(theta, FIG_Q, FIG_LO, FIG_HI, alpha)
        assert P.shape == (8,)
        assert np.all(P >= 0.0)
        assert abs(P.sum() - 1.0) < 1e-14
        assert np.argmax(P) == int(np.clip(round(theta / FIG_Q), FIG_LO, FIG_HI)) - FIG_LO or \
            abs(theta / FIG_Q - math.floor(theta / FIG_Q) - 0.5) < 1e-9


def test_cpmf_two_levels_is_the_logistic_function():
    # levels {0, q}: P(q | theta) = 1 / (1 + exp(-alpha q (2 theta - q)))
    q, alpha = 0.3, 17.0
    for theta in (-0.4, 0.0, 0.1, 0.15, 0.2, 0.9):
        P = oracle.cpmf(theta, q, 0, 1, alpha)
        expect = 1.0 / (1.0 + math.exp(-alpha * q * (2.0 * theta - q)))
        assert P[1] == pytest.approx(expect, rel=1e-13, abs=1e-300)
        assert P[0] == pytest.approx(1.0 - expect, rel=1e-12, abs=1e-15)


def test_cpmf_ratio_of_neighbours():
    # P_i / P_j = exp(-alpha ((theta-iq)^2 - (theta-jq)^2)) for any pair: catches an index or sign slip.
    q, alpha, theta, lo, hi = 0.07, 40.0, 0.11, -3, 5
    P = oracle.cpmf(theta, q, lo, hi, alpha)
    for i in range(lo, hi + 1):
        for j in range(lo, hi + 1):
            expect = math.exp(-alpha * ((theta - i * q) ** 2 - (theta - j * q) ** 2))
            assert P[i - lo] / P[j - lo] == pytest.approx(expect, rel=1e-11)


# ------------------------------------------------------------------ Q_d (Sec. IV-B, Eq. (8))
def test_soft_three_levels_closed_form():
    # levels {-q, 0, q}: Q_d = q * 2 e^{-a} sinh(2 alpha q theta) / (1 + 2 e^{-a} cosh(2 alpha q theta)), a = alpha q^2
    q, alpha = f32(0.25), f32(9.0)
    x = np.linspace(-0.7, 0.7, 57).astype(f32)
    y = oracle.soft(x, q, -1, 1, alpha)
    qq, al = float(q), float(alpha)
    a = al * qq * qq
    t = 2.0 * al * qq * x.astype(np.float64)
    expect = qq * 2.0 * math.exp(-a) * np.sinh(t) / (1.0 + 2.0 * math.exp(-a) * np.cosh(t))
    np.testing.assert_allclose(y, expect, rtol=1e-12, atol=1e-15)


def test_soft_two_levels_closed_form_and_slope():
    # levels {0, q}: Q_d = q sigma(z), z = alpha q (2 theta - q); dQ_d/dtheta = 2 alpha q^2 sigma (1 - sigma)
    q, alpha = f32(0.5), f32(6.0)
    x = np.linspace(-0.5, 1.0, 31).astype(f32)
    y = oracle.soft(x, q, 0, 1, alpha)
    dth, dq, dal, var = oracle.partials(x, q, 0, 1, alpha)
    qq, al = float(q), float(alpha)
    s = 1.0 / (1.0 + np.exp(-al * qq * (2.0 * x.astype(np.float64) - qq)))
    np.testing.assert_allclose(y, qq * s, rtol=1e-13)
    np.testing.assert_allclose(dth, 2.0 * al * qq * qq * s * (1.0 - s), rtol=1e-11)
    np.testing.assert_allclose(var, qq * qq * s * (1.0 - s), rtol=1e-11)
    # d/dq [q sigma(alpha q (2 theta - q))] and d/dalpha, by hand
    th = x.astype(np.float64)
    np.testing.assert_allclose(dq, s + qq * s * (1 - s) * al * (2.0 * th - 2.0 * qq), rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(dal, qq * s * (1 - s) * qq * (2.0 * th - qq), rtol=1e-10, atol=1e-13)


def test_soft_is_odd_on_symmetric_alphabets():
    x = inputs.normal((501,), 0.3, seed=11)
    y1 = oracle.soft(x, f32(0.1), -3, 3, f32(80.0))
    y2 = oracle.soft(-x, f32(0.1), -3, 3, f32(80.0))
    np.testing.assert_allclose(y1, -y2, rtol=0, atol=1e-15)


def test_soft_saturates_outside_the_alphabet():
    y = oracle.soft(np.array([10.0, -10.0], dtype=f32), f32(0.1), -4, 3, f32(100.0))
    assert y[0] == pytest.approx(3 * float(f32(0.1)), abs=1e-12)
    assert y[1] == pytest.approx(-4 * float(f32(0.1)), abs=1e-12)


@pytest.mark.parametrize("alpha", (1e6, 1e8))
def test_soft_tends_to_nearest_level_for_large_alpha(alpha):
    # Remark of Sec. IV-A / end of Sec. IV-B: Q_p and Q_d approach the uniform quantizer as alpha grows.
    x = inputs.normal((4000,), 0.25, seed=5)
    q = f32(0.1)
    u = x.astype(np.float64) / float(q)
    away = np.abs(u - np.floor(u) - 0.5) > 0.05
    idx, _ = oracle.hard(x, q, FIG_LO, FIG_HI)
    y = oracle.soft(x, q, FIG_LO, FIG_HI, f32(alpha))
    np.testing.assert_allclose(y[away], idx[away] * float(q), rtol=0, atol=1e-9)


def test_midpoint_value_and_slope_for_large_alpha():
    # at theta = (k + 1/2) q the two nearest levels share the mass: Q_d = theta, dQ_d/dtheta -> alpha q^2 / 2
    q, alpha = f32(0.125), f32(4096.0)                      # exactly representable products
    x = (np.arange(-4, 3, dtype=np.float64) + 0.5) * float(q)
    x32 = x.astype(f32)
    assert np.array_equal(x32.astype(np.float64), x)
    y = oracle.soft(x32, q, FIG_LO, FIG_HI, alpha)
    dth, _, _, _ = oracle.partials(x32, q, FIG_LO, FIG_HI, alpha)
    np.testing.assert_allclose(y, x, rtol=0, atol=1e-14)
    np.testing.assert_allclose(dth, float(alpha) * float(q) ** 2 / 2.0, rtol=1e-12)


# ------------------------------------------------------------------ Proposition 1
@pytest.mark.parametrize("alpha", FIG_ALPHAS)
def test_proposition_1_variance_decomposition(alpha):
    x = np.linspace(-0.55, 0.45, 41).astype(f32)
    q = f32(FIG_Q)
    y = oracle.soft(x, q, FIG_LO, FIG_HI, f32(alpha))
    _, _, _, var = oracle.partials(x, q, FIG_LO, FIG_HI, f32(alpha))
    lev = np.arange(FIG_LO, FIG_HI + 1, dtype=np.float64) * float(q)
    for e, th in enumerate(x.astype(np.float64)):
        P = oracle.cpmf(th, float(q), FIG_LO, FIG_HI, float(f32(alpha)))
        lhs = float(np.sum(P * (th - lev) ** 2))            # E{(theta - Q_p)^2 | theta}
        assert lhs == pytest.approx((th - y[e]) ** 2 + var[e], rel=1e-11, abs=1e-18)


# ------------------------------------------------------------------ Lemma 1 and the derived d/dalpha
@pytest.mark.parametrize("alpha", FIG_ALPHAS)
@pytest.mark.parametrize("window", (0, 5))
def test_lemma_1_against_finite_differences(alpha, window):
    q, al = f32(FIG_Q), f32(alpha)
    # stay away from the points where the 5-level window switches (Q_d is discontinuous there)
    x = np.array([-0.52, -0.43, -0.31, -0.262, -0.13, -0.04, 0.0, 0.02, 0.13, 0.168, 0.31, 0.33, 0.41], dtype=f32)
    dth, dq, dal, _ = oracle.partials(x, q, FIG_LO, FIG_HI, al, window)
    qq, aa = float(q), float(al)
    for e, th in enumerate(x.astype(np.float64)):
        h = 1e-6
        fd_th = (qd_from_cpmf(th + h, qq, FIG_LO, FIG_HI, aa, window) - qd_from_cpmf(th - h, qq, FIG_LO, FIG_HI, aa, window)) / (2 * h)
        hq = 1e-7
        fd_q = (qd_from_cpmf(th, qq + hq, FIG_LO, FIG_HI, aa, window) - qd_from_cpmf(th, qq - hq, FIG_LO, FIG_HI, aa, window)) / (2 * hq)
        ha = 1e-3
        fd_a = (qd_from_cpmf(th, qq, FIG_LO, FIG_HI, aa + ha, window) - qd_from_cpmf(th, qq, FIG_LO, FIG_HI, aa - ha, window)) / (2 * ha)
        assert dth[e] == pytest.approx(fd_th, rel=2e-6, abs=1e-8)
        assert dq[e] == pytest.approx(fd_q, rel=2e-6, abs=1e-6)
        assert dal[e] == pytest.approx(fd_a, rel=2e-6, abs=1e-10)


def test_lemma_1_finite_differences_on_unsigned_and_wide_alphabets():
    cases = [(f32(0.25), 0, 15, f32(50.0)), (f32(0.03), -32, 31, f32(500.0)), (f32(0.0315), -127, 127, f32(1.0))]
    for q, lo, hi, al in cases:
        x = (inputs.normal((9,), 1.0, seed=3) * f32(q * (hi - lo) / 4)).astype(f32)
        dth, dq, dal, _ = oracle.partials(x, q, lo, hi, al)
        qq, aa = float(q), float(al)
        for e, th in enumerate(x.astype(np.float64)):
            h, hq, ha = 1e-6 * max(1.0, abs(th)), 1e-6 * qq, 1e-5 * aa
            fd_th = (qd_from_cpmf(th + h, qq, lo, hi, aa) - qd_from_cpmf(th - h, qq, lo, hi, aa)) / (2 * h)
            fd_q = (qd_from_cpmf(th, qq + hq, lo, hi, aa) - qd_from_cpmf(th, qq - hq, lo, hi, aa)) / (2 * hq)
            fd_a = (qd_from_cpmf(th, qq, lo, hi, aa + ha) - qd_from_cpmf(th, qq, lo, hi, aa - ha)) / (2 * ha)
            assert dth[e] == pytest.approx(fd_th, rel=1e-5, abs=1e-8)
            assert dq[e] == pytest.approx(fd_q, rel=1e-5, abs=1e-5)
            assert dal[e] == pytest.approx(fd_a, rel=1e-5, abs=1e-9)


@pytest.mark.parametrize("alpha", FIG_ALPHAS)
def test_slope_grows_away_from_the_nearest_level(alpha):
    # Property read off Fig. 1 (Sec. IV-B): dQ_d/dtheta increases as theta leaves its nearest level.
    # It is a property of the lattice of levels: with the figure's 8 levels and alpha = 100 (alpha q^2 = 1) the
    # missing levels beyond the ends bend the curve, so that alpha is checked on a 64-level alphabet instead.
    q = f32(FIG_Q)
    lo, hi = (FIG_LO, FIG_HI) if alpha > 100.0 else (-32, 31)
    for k in (-1, 0):
        for sign in (+1.0, -1.0):
            t = np.linspace(0.0, 0.49, 50)
            x = ((k + sign * t) * float(q)).astype(f32)
            dth, _, _, _ = oracle.partials(x, q, lo, hi, f32(alpha))
            assert np.all(np.diff(dth) > 0)


# ------------------------------------------------------------------ top-five truncation (Sec. VI-B.1)
def test_window_keeps_the_five_nearest_levels_and_renormalises():
    q, lo, hi, beta = 0.25, 0, 15, 3.0                     # small beta*q^2: the tails carry weight
    for theta in (-0.3, 0.0, 0.1, 0.6, 1.27, 2.0, 3.4, 3.7, 3.9, 5.0):
        full = oracle.cpmf(theta, q, lo, hi, beta)
        win = oracle.cpmf(theta, q, lo, hi, beta, 5)
        kept = np.flatnonzero(win)
        start = int(np.clip(round(theta / q) - 2, lo, hi - 4)) - lo
        assert list(kept) == list(range(start, start + 5))
        assert abs(win.sum() - 1.0) < 1e-14
        np.testing.assert_allclose(win[kept] / win[kept].sum(), full[kept] / full[kept].sum(), rtol=1e-13)
        # every kept entry is at least as probable as every dropped one
        dropped = np.setdiff1d(np.arange(16), kept)
        assert full[kept].min() >= full[dropped].max()


def test_window_tie_takes_the_lower_level():
    # theta exactly between levels 3 and 4: levels 1 and 6 are equally far; the lower one is kept
    win = oracle.cpmf(0.875, 0.25, 0, 15, 2.0, 5)
    assert list(np.flatnonzero(win)) == [1, 2, 3, 4, 5]


def test_window_not_smaller_than_alphabet_is_the_full_cpmf():
    a = oracle.cpmf(0.05, 0.1, -1, 1, 30.0, 5)
    b = oracle.cpmf(0.05, 0.1, -1, 1, 30.0, 0)
    assert np.array_equal(a, b)


# ------------------------------------------------------------------ hard index (uniform quantizer Q_u)
def test_hard_agrees_with_brute_force_nearest_level():
    for q, lo, hi, seed in ((0.02, -7, 7, 1), (0.25, 0, 15, 2), (0.7, -1, 1, 3), (0.011, -127, 127, 4)):
        x = inputs.normal((3000,), q * (hi - lo) / 3.0, seed=seed)
        if lo == 0:
            x = np.maximum(x, 0)
        idx, hist = oracle.hard(x, f32(q), lo, hi)
        lev = np.arange(lo, hi + 1, dtype=np.float64) * float(f32(q))
        dist = np.abs(x.astype(np.float64)[:, None] - lev[None, :])
        brute = np.argmin(dist, axis=1) + lo
        u = x.astype(np.float64) / float(f32(q))
        near_mid = np.abs(u - np.floor(u) - 0.5) < 1e-6
        assert np.array_equal(idx[~near_mid], brute[~near_mid])
        assert near_mid.sum() < 5
        assert hist.sum() == x.size
        assert np.array_equal(hist, np.bincount(idx - lo, minlength=hi - lo + 1).astype(np.uint64))


def test_hard_ties_clamp_and_nan():
    q = f32(0.5)
    x = np.array([0.25, 0.75, 1.25, -0.25, -0.75, 100.0, -100.0, np.inf, -np.inf, np.nan, 0.0, -0.0], dtype=f32)
    idx, hist = oracle.hard(x, q, -2, 3)
    # quotients .5, 1.5, 2.5, -.5, -1.5 round to the even neighbour
    assert list(idx) == [0, 2, 2, 0, -2, 3, -2, 3, -2, -2, 0, 0]      # NaN -> lo
    idx_u, _ = oracle.hard(np.array([np.nan, -3.0], dtype=f32), q, 2, 5)
    assert list(idx_u) == [2, 2]                       # NaN and values below the range -> lo
    assert hist.sum() == x.size


def test_hard_single_level_alphabet():
    idx, hist = oracle.hard(np.array([-1.0, 0.3, 7.0], dtype=f32), f32(0.1), 2, 2)
    assert list(idx) == [2, 2, 2] and list(hist) == [3]


# ------------------------------------------------------------------ entropy (Sec. III-A, Sec. V-C)
def test_entropy_closed_forms():
    H, p, n = oracle.entropy(np.full(16, 7, dtype=np.uint64))
    assert H == pytest.approx(4.0, abs=1e-14) and n == 112 and np.allclose(p, 1 / 16)
    H, p, n = oracle.entropy(np.array([0, 0, 9, 0], dtype=np.uint64))
    assert H == 0.0 and n == 9 and list(p) == [0, 0, 1, 0]
    H, _, _ = oracle.entropy(np.array([1, 3], dtype=np.uint64))
    assert H == pytest.approx(-(0.25 * math.log2(0.25) + 0.75 * math.log2(0.75)), abs=1e-15)
    H, _, _ = oracle.entropy(np.array([2, 1, 1], dtype=np.uint64))
    assert H == pytest.approx(1.5, abs=1e-15)
    H, _, n = oracle.entropy(np.zeros(5, dtype=np.uint64))
    assert H == 0.0 and n == 0


def test_entropy_matches_ideal_code_length_on_dyadic_counts():
    # dyadic probabilities: entropy equals the mean length of the optimal prefix code (Sec. V-C, Sec. VI-A)
    hist = np.array([8, 4, 2, 1, 1], dtype=np.uint64)
    lengths = np.array([1, 2, 3, 4, 4])
    H, p, _ = oracle.entropy(hist)
    assert H == pytest.approx(float(np.dot(p, lengths)), abs=1e-15)


# ------------------------------------------------------------------ backward (Sec. V-B) and the rate term
def test_backward_is_the_gradient_proxy_of_the_partials():
    x = inputs.normal((777,), 0.06, seed=8)
    g = inputs.normal((777,), 1.0, seed=9)
    q, lo, hi, al = f32(0.02), -7, 7, f32(50.0)
    out = oracle.backward(x, g, q, lo, hi, al)
    dth, dq, dal, _ = oracle.partials(x, q, lo, hi, al)
    gd = g.astype(np.float64)
    np.testing.assert_allclose(out["grad_x"], gd * dth, rtol=1e-15)
    assert out["grad_q"] == pytest.approx(math.fsum(gd * dq), rel=1e-12)
    assert out["grad_alpha"] == pytest.approx(math.fsum(gd * dal), rel=1e-12)
    assert out["abs_q"] == pytest.approx(math.fsum(np.abs(gd * dq)), rel=1e-12)
    assert out["abs_alpha"] == pytest.approx(math.fsum(np.abs(gd * dal)), rel=1e-12)


def test_backward_term_magnitude_scales_two_level_closed_form():
    # mag_q / mag_alpha (the floors of the reduced-sum tolerances) on levels {0, q}, where every moment is a
    # logistic expression: E = q s, Var = q^2 s (1 - s), Skew_u = E X^3 - E X E X^2 = q^3 s (1 - s),
    # s = sigma(alpha q (2 theta - q)).  A dropped 1/q, a missing term or a lost absolute value fails here.
    q, alpha = f32(0.5), f32(6.0)
    x = np.linspace(-0.5, 1.0, 31).astype(f32)
    g = inputs.normal((31,), 1.0, seed=21)
    out = oracle.backward(x, g, q, 0, 1, alpha)
    qq, al, th, ag = float(q), float(alpha), x.astype(np.float64), np.abs(g.astype(np.float64))
    s = 1.0 / (1.0 + np.exp(-al * qq * (2.0 * th - qq)))
    v = s * (1.0 - s)
    mag_q = math.fsum(ag * (qq * s + np.abs(2.0 * al * th) * qq * qq * v + 2.0 * al * qq ** 3 * v) / qq)
    mag_alpha = math.fsum(ag * (np.abs(2.0 * th) * qq * qq * v + qq ** 3 * v))
    assert out["mag_q"] == pytest.approx(mag_q, rel=1e-11)
    assert out["mag_alpha"] == pytest.approx(mag_alpha, rel=1e-11)
    # the three terms have mixed signs on this grid (theta < 0 and theta > 0), so the scales strictly exceed
    # the sums of |g * partial| and those exceed the signed sums
    assert out["mag_q"] > out["abs_q"] > abs(out["grad_q"])
    assert out["mag_alpha"] > out["abs_alpha"] > abs(out["grad_alpha"])


@pytest.mark.parametrize("window", (0, 5))
def test_backward_term_magnitude_scales_from_the_cpmf(window):
    # General alphabets: the three terms of Eq. (9b) and the two of dQ_d/dalpha rebuilt from the CPMF itself
    # (moments taken with numpy), and the identities  term sums = partials  that tie them to Lemma 1.
    x = inputs.normal((257,), 0.08, seed=12)
    g = inputs.normal((257,), 1.0, seed=13)
    q, lo, hi, al = f32(0.02), -7, 7, f32(50.0)
    out = oracle.backward(x, g, q, lo, hi, al, window)
    _, dq, dal, _ = oracle.partials(x, q, lo, hi, al, window)
    qq, a = float(q), float(al)
    lev = np.arange(lo, hi + 1, dtype=np.float64) * qq
    mq, ma = [], []
    for e in range(x.size):
        th, ge = float(x[e]), abs(float(g[e]))
        P = oracle.cpmf(th, qq, lo, hi, a, window)
        E = float(P @ lev)
        var = float(P @ (lev - E) ** 2)
        sk = float(P @ lev ** 3) - E * float(P @ lev ** 2)
        t_q = (E, 2.0 * a * th * var, -2.0 * a * sk)
        t_a = (2.0 * th * var, -sk)
        assert sum(t_q) / qq == pytest.approx(dq[e], rel=1e-9, abs=1e-12)
        assert sum(t_a) == pytest.approx(dal[e], rel=1e-9, abs=1e-15)
        mq.append(ge * sum(abs(t) for t in t_q) / qq)
        ma.append(ge * sum(abs(t) for t in t_a))
    assert out["mag_q"] == pytest.approx(math.fsum(mq), rel=1e-11)
    assert out["mag_alpha"] == pytest.approx(math.fsum(ma), rel=1e-11)


def test_backward_zero_rate_weight_and_uniform_probabilities_add_nothing():
    x = inputs.normal((300,), 0.06, seed=8)
    g = inputs.normal((300,), 1.0, seed=9)
    q, lo, hi, al = f32(0.02), -7, 7, f32(50.0)
    base = oracle.backward(x, g, q, lo, hi, al)["grad_x"]
    lp = np.random.default_rng(0).dirichlet(np.ones(15))
    np.testing.assert_array_equal(oracle.backward(x, g, q, lo, hi, al, 0, 0.0, lp)["grad_x"], base)
    uni = oracle.backward(x, g, q, lo, hi, al, 0, 0.01, np.full(15, 1 / 15))["grad_x"]
    np.testing.assert_allclose(uni, base, rtol=0, atol=1e-15)


@pytest.mark.parametrize("window", (0, 5))
def test_rate_term_is_the_derivative_of_total_bits_of_the_marginal_pmf(window):
    # Sec. V-C: total bits = n * H( (1/n) sum_i P(.|theta_i) ).  Its derivative w.r.t. one theta_i, by central
    # differences, must equal the oracle's rate term when the level probabilities are that marginal PMF.
    q, lo, hi, al = f32(0.25), 0, 7, f32(12.0)
    x = np.array([0.03, 0.31, 0.52, 0.9, 1.1, 1.26, 1.6, 0.02], dtype=f32)   # away from window switches
    n = x.size
    qq, aa = float(q), float(al)

    def total_bits(theta):
        mp = np.mean([oracle.cpmf(t, qq, lo, hi, aa, window) for t in theta], axis=0)
        nz = mp > 0
        return -n * float(np.sum(mp[nz] * np.log2(mp[nz])))

    th = x.astype(np.float64)
    mp = np.mean([oracle.cpmf(t, qq, lo, hi, aa, window) for t in th], axis=0)
    zero_g = np.zeros(n, dtype=f32)
    rate = oracle.backward(x, zero_g, q, lo, hi, al, window, 1.0, mp)["grad_x"]
    for i in range(n):
        h = 1e-6
        tp, tm = th.copy(), th.copy()
        tp[i] += h
        tm[i] -= h
        fd = (total_bits(tp) - total_bits(tm)) / (2 * h)
        assert rate[i] == pytest.approx(fd, rel=1e-5, abs=1e-7)
    # scaling with the rate weight, and clamping of log2 at -30 for empty levels
    half = oracle.backward(x, zero_g, q, lo, hi, al, window, 0.5, mp)["grad_x"]
    np.testing.assert_allclose(half, 0.5 * rate, rtol=1e-14)
    lp = np.zeros(8)
    lp[0] = 1.0                                            # log2: 0 for level 0, -30 for the others
    P = oracle.cpmf(float(x[1]), qq, lo, hi, aa, window)
    lev = np.arange(lo, hi + 1) * qq
    L = np.where(np.arange(8) == 0, 0.0, -30.0)
    expect = -2.0 * aa * (np.sum(P * L * lev) - np.sum(P * L) * np.sum(P * lev))
    got = oracle.backward(x[1:2], zero_g[1:2], q, lo, hi, al, window, 1.0, lp)["grad_x"][0]
    assert got == pytest.approx(expect, rel=1e-12)


# ------------------------------------------------------------------ index GEMMs (Sec. V-A)
def test_index_gemms_against_numpy_integer_matmul():
    M, K, N = 37, 53, 19
    A = inputs.uniform_indices((M, K), 0, 15, seed=1)
    As = inputs.uniform_indices((M, K), -128, 127, seed=2)
    W = inputs.uniform_indices((K, N), -7, 7, seed=3)
    G = inputs.uniform_indices((M, N), -127, 127, seed=4)
    assert A.dtype == np.uint8 and W.dtype == np.int8
    A64, As64, W64, G64 = (t.astype(np.int64) for t in (A, As, W, G))
    assert np.array_equal(oracle.gemm_fwd(A, W), A64 @ W64)
    assert np.array_equal(oracle.gemm_fwd(As, W), As64 @ W64)
    assert np.array_equal(oracle.gemm_dx(G, W), G64 @ W64.T)
    assert np.array_equal(oracle.gemm_dw(A, G), A64.T @ G64)
    assert np.array_equal(oracle.gemm_dw(As, G), As64.T @ G64)


def test_index_gemms_with_padded_leading_dimensions_and_uint8_above_127():
    M, K, N = 5, 20, 7
    Ap = np.zeros((M, 32), dtype=np.uint8)
    Ap[:, :K] = inputs.uniform_indices((M, K), 200, 255, seed=5)
    Wp = np.zeros((K, 16), dtype=np.int8)
    Wp[:, :N] = inputs.uniform_indices((K, N), -128, -100, seed=6)
    A, W = Ap[:, :K], Wp[:, :N]
    assert np.array_equal(oracle.gemm_fwd(A, W), A.astype(np.int64) @ W.astype(np.int64))


def test_one_hot_index_matrix_selects_rows():
    K, N = 6, 4
    W = inputs.uniform_indices((K, N), -7, 7, seed=7)
    A = np.zeros((K, K), dtype=np.uint8)
    A[np.arange(K), np.arange(K)[::-1]] = 1
    assert np.array_equal(oracle.gemm_fwd(A, W), W[::-1].astype(np.int64))


# ------------------------------------------------------------------ soft histogram / marginal PMF (Sec. V-C, Eq. (25))
def test_soft_histogram_is_the_sum_of_cpmfs_and_tends_to_the_count_histogram():
    x = inputs.normal((3001,), 0.2, seed=31)
    q, lo, hi = f32(0.1), -4, 3
    for window in (0, 5):
        s = oracle.mpmf(x, q, lo, hi, f32(40.0), window)
        assert s.sum() == pytest.approx(x.size, rel=1e-12)               # every CPMF sums to 1
        byhand = np.sum([oracle.cpmf(float(t), float(q), lo, hi, float(f32(40.0)), window) for t in x[:200]], axis=0)
        np.testing.assert_allclose(oracle.mpmf(x[:200], q, lo, hi, f32(40.0), window), byhand, rtol=1e-12)
    # Remark of Sec. IV-A: for large alpha all the mass sits on the nearest level -> the count histogram
    u = x.astype(np.float64) / float(q)
    away = np.abs(u - np.floor(u) - 0.5) > 0.02
    _, hist = oracle.hard(x[away], q, lo, hi)
    np.testing.assert_allclose(oracle.mpmf(x[away], q, lo, hi, f32(1e7)), hist.astype(np.float64), rtol=0, atol=1e-6)


def test_soft_histogram_two_levels_closed_form():
    q, alpha = f32(0.5), f32(6.0)
    x = inputs.normal((500,), 0.5, seed=32)
    s = oracle.mpmf(x, q, 0, 1, alpha)
    sig = 1.0 / (1.0 + np.exp(-float(alpha) * float(q) * (2.0 * x.astype(np.float64) - float(q))))
    assert s[1] == pytest.approx(sig.sum(), rel=1e-12) and s[0] == pytest.approx((1 - sig).sum(), rel=1e-12)


def test_gradient_digits_reconstruct_the_gradient_within_half_a_fine_step():
    # pins the two-digit expansion to its defining property: |g - (q1 i1 + q2 i2)| <= q2 / 2 inside the range,
    # digits within [-127, 127], and saturation outside
    rng = np.random.default_rng(3)
    g = rng.normal(0, 1e-2, 20000).astype(np.float32)
    absmax = float(np.abs(g).max())
    i1, i2, q1, q2 = oracle.gradient_digits(g, absmax)
    assert np.abs(i1).max() <= 127 and np.abs(i2).max() <= 127
    rec = np.float64(q1) * i1 + np.float64(q2) * i2
    assert np.abs(g.astype(np.float64) - rec).max() <= float(q2) / 2 * (1 + 1e-6)
    assert np.isclose(float(q2) * 254, float(q1), rtol=1e-6) and np.isclose(float(q1) * 127, absmax, rtol=1e-6)
    # a bound smaller than the data: both digits saturate with the sign of g
    i1s, i2s, _, _ = oracle.gradient_digits(np.array([1.0, -1.0], dtype=np.float32), 0.5)
    assert list(i1s) == [127, -127] and list(i2s) == [127, -127]
    # exact multiples of the coarse step have a zero fine digit
    i1m, i2m, q1m, _ = oracle.gradient_digits((np.arange(-5, 6) * np.float32(2.0 / 127)).astype(np.float32), 2.0)
    assert list(i1m) == list(range(-5, 6)) and not i2m.any()
