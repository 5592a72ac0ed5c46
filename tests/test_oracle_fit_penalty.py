"""Pins for the oracle's moments, moment-ratio fit, penalty and gradient."""
import math
from fractions import Fraction

import mpmath as mp
import numpy as np
import pytest
import scipy.optimize
import scipy.special

import gg_synth
from oracle import gg_oracle as o

mp.mp.dps = 50


# ------------------------------------------------------------------ moments
def test_moments_brute_force_exact_rationals():
    rng = np.random.default_rng(11)
    for n in (1, 2, 7, 64):
        x = (rng.standard_normal(n) * np.exp(rng.uniform(-20, 20, n))).astype(np.float32)
        s1 = sum(Fraction(abs(float(v))) for v in x)
        s2 = sum(Fraction(float(v)) ** 2 for v in x)
        g1, g2, cnt, bad = o.moments(x)
        assert cnt == n and bad == 0
        assert abs(Fraction(g1) - s1) <= s1 * Fraction(1, 10 ** 15)
        assert abs(Fraction(g2) - s2) <= s2 * Fraction(1, 10 ** 15)


def test_moments_count_nonfinite_and_skip_them():
    x = np.array([1.0, -2.0, np.inf, np.nan, 3.0], dtype=np.float32)
    s1, s2, n, bad = o.moments(x)
    assert (s1, s2, n, bad) == (6.0, 14.0, 5, 2)
    assert o.fit(x)[5] & o.FLAG_NONFINITE


# ---------------------------------------------------------------------- fit
@pytest.mark.parametrize("beta", [0.05001, 0.1, 0.3, 0.5, 0.8, 1.0, 1.3, 2.0, 4.0, 10.0, 19.99])
def test_fit_round_trip_from_exact_moments(beta):
    """Moments computed in 50 digits from the density's closed forms must give beta, alpha back."""
    alpha, n = 0.0123, 1000
    b = mp.mpf(beta)
    m1 = alpha * mp.gamma(2 / b) / mp.gamma(1 / b)
    m2 = alpha ** 2 * mp.gamma(3 / b) / mp.gamma(1 / b)
    bh, ah, fl = o.fit_from_moments(float(m1 * n), float(m2 * n), n)
    assert fl == 0
    # the ratio is flat at large beta: the round trip is limited by the rounding of the moments
    tol = 1e-12 if beta <= 4 else 1e-9
    assert bh == pytest.approx(beta, rel=tol)
    assert ah == pytest.approx(alpha, rel=tol)


def test_fit_agrees_with_an_independent_root_finder():
    """brentq on scipy's gammaln instead of bisection on libm's lgamma."""
    rng = np.random.default_rng(5)
    for _ in range(20):
        beta = float(np.exp(rng.uniform(math.log(0.1), math.log(8.0))))
        x = gg_synth.gg_host(rng, beta, 0.5, 4096).numpy()
        s1, s2, n, _ = o.moments(x)
        r = (s1 / n) ** 2 / (s2 / n)
        gl = scipy.special.gammaln
        f = lambda b: 2 * gl(2 / b) - gl(1 / b) - gl(3 / b) - math.log(r)
        root = scipy.optimize.brentq(f, 0.05, 20.0, xtol=1e-15, rtol=1e-15)
        bh, ah, fl = o.fit_from_moments(s1, s2, n)
        assert fl == 0
        assert bh == pytest.approx(root, rel=1e-11)
        # Eq. 2/3 identity: the fitted scale reproduces the second moment exactly
        assert o.variance(ah, bh) == pytest.approx(s2 / n, rel=1e-12)


def test_fit_tiny_and_degenerate_inputs():
    # x = {+1,-1}: ratio 1 > 3/4 -> clamped high
    b, a, *_rest, fl = o.fit(np.array([1, -1], dtype=np.float32))
    assert b == o.BETA_HI and fl == o.FLAG_BETA_CLAMPED_HI
    # x = {1,2,3}: ratio 36/(3*14) = 6/7 > 3/4 -> clamped high, alpha from Eq. 2
    b, a, s1, s2, n, fl = o.fit(np.array([1, 2, 3], dtype=np.float32))
    assert (s1, s2, n) == (6.0, 14.0, 3) and b == o.BETA_HI and fl == o.FLAG_BETA_CLAMPED_HI
    assert a == pytest.approx(math.sqrt(14 / 3) * math.sqrt(math.gamma(0.05) / math.gamma(0.15)), rel=1e-13)
    # one huge value among zeros: ratio 1/n -> clamped low
    x = np.zeros(10 ** 6, dtype=np.float32); x[0] = 1.0
    b, a, *_rest, fl = o.fit(x)
    assert b == o.BETA_LO and fl == o.FLAG_BETA_CLAMPED_LO
    # empty and all-zero segments
    for x in (np.zeros(0, np.float32), np.zeros(17, np.float32)):
        b, a, *_rest, fl = o.fit(x)
        assert (b, a) == (0.0, 0.0) and fl == o.FLAG_DEGENERATE


@pytest.mark.parametrize("beta", [0.5, 1.0, 1.3, 2.0])
def test_fit_recovers_parameters_of_library_samples(beta):
    rng = np.random.default_rng(int(beta * 100))
    alpha = gg_synth.alpha_for_std(0.02, beta)
    x = gg_synth.gg_host(rng, beta, alpha, 2_000_000).numpy()
    bh, ah, *_ = o.fit(x)
    assert bh == pytest.approx(beta, rel=0.02)
    assert ah == pytest.approx(alpha, rel=0.03)


# ------------------------------------------------------- penalty & gradient
def _mp_grad(x, beta, alpha, lam):
    if x == 0:
        return mp.mpf(0)
    g = mp.mpf(lam) * beta * abs(mp.mpf(x)) ** (mp.mpf(beta) - 1) / mp.mpf(alpha) ** mp.mpf(beta)
    return g if x > 0 else -g


@pytest.mark.parametrize("beta,alpha", [(0.5, 3e-4), (0.8, 1.1), (1.0, 0.02), (1.3, 0.014),
                                        (2.0, 0.03), (3.7, 0.5), (0.05, 1e-3), (20.0, 2.0)])
def test_penalty_grad_multiprecision(beta, alpha):
    lam = 1e-4
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(56) * alpha).astype(np.float32)
    x = np.concatenate([x, np.array([0.0, -0.0, 1e-45, -1e-45, 1.17549435e-38, 3.0e38, -3.0e38, 1.0],
                                    dtype=np.float32)])
    pen, g = o.penalty_grad(x, beta, alpha, lam)
    ref_pen = mp.mpf(0)
    for xi, gi in zip(x, g):
        ref = _mp_grad(float(xi), beta, alpha, lam)
        ref_pen += mp.mpf(lam) * (abs(mp.mpf(float(xi))) / mp.mpf(alpha)) ** mp.mpf(beta)
        if ref == 0:
            assert gi == 0.0
        elif abs(ref) > mp.mpf(2) ** 1023:
            assert math.isinf(gi) and (gi > 0) == (ref > 0)
        elif abs(ref) < mp.mpf(2) ** -1000:
            assert abs(gi) < 2.0 ** -999
        else:
            assert abs(mp.mpf(gi) - ref) <= abs(ref) * mp.mpf(10) ** -13
    if ref_pen < mp.mpf(2) ** 1023:
        assert abs(mp.mpf(pen) - ref_pen) <= ref_pen * mp.mpf(10) ** -13


def test_gradient_special_cases():
    rng = np.random.default_rng(4)
    x = (rng.standard_normal(64) * 0.02).astype(np.float32)
    lam, alpha = 1e-4, 0.02
    _, g2 = o.penalty_grad(x, 2.0, alpha, lam)          # Gaussian: linear in x
    np.testing.assert_allclose(g2, 2 * lam * x.astype(np.float64) / alpha ** 2, rtol=1e-14)
    _, g1 = o.penalty_grad(x, 1.0, alpha, lam)          # Laplace: constant magnitude
    np.testing.assert_allclose(g1, lam * np.sign(x.astype(np.float64)) / alpha, rtol=1e-14)
    # odd symmetry
    _, gm = o.penalty_grad(-x, 1.3, alpha, lam)
    _, gp = o.penalty_grad(x, 1.3, alpha, lam)
    np.testing.assert_array_equal(gm, -gp)


@pytest.mark.parametrize("beta", [0.6, 1.0, 1.7])
def test_gradient_is_the_derivative_of_the_penalty(beta):
    """Central differences of P with respect to one element at a time."""
    lam, alpha = 1e-4, 0.02
    x = np.array([0.013, -0.004, 0.05, -0.021], dtype=np.float32)
    _, g = o.penalty_grad(x, beta, alpha, lam)
    for i in range(len(x)):
        xp, xm = x.copy(), x.copy()
        h = np.float32(abs(x[i]) * 2.0 ** -10)
        xp[i] += h
        xm[i] -= h
        pp, _ = o.penalty_grad(xp, beta, alpha, lam, want_grad=False)
        pm, _ = o.penalty_grad(xm, beta, alpha, lam, want_grad=False)
        fd = (pp - pm) / (float(xp[i]) - float(xm[i]))
        assert g[i] == pytest.approx(fd, rel=1e-5)


@pytest.mark.parametrize("beta", [0.5, 0.8, 1.3, 2.0])
def test_penalty_statistical_identity(beta):
    """(|x|/alpha)^beta of a GG variate is Gamma(1/beta, 1): its mean is 1/beta."""
    rng = np.random.default_rng(8)
    alpha, lam, n = 0.05, 2.0, 1_000_000
    x = gg_synth.gg_host(rng, beta, alpha, n).numpy()
    pen, _ = o.penalty_grad(x, beta, alpha, lam, want_grad=False)
    se = math.sqrt(1 / beta / n)            # variance of Gamma(1/beta,1) is 1/beta
    assert abs(pen / (lam * n) - 1 / beta) < 5 * se


def test_degenerate_parameters_give_zeros():
    x = np.array([1.0, -2.0], dtype=np.float32)
    pen, g = o.penalty_grad(x, 0.0, 0.0, 1.0)
    assert pen == 0.0 and not g.any()
