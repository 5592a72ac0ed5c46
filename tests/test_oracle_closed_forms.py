"""Pins for the oracle's closed forms (Eq. 1-5) against multi-precision integration of the
density itself, library distributions, and the special cases the paper names."""
import math
import os

import mpmath as mp
import numpy as np
import pytest
import scipy.stats

from oracle import gg_oracle as o

mp.mp.dps = 40
BETAS = [0.1, 0.25, 0.5, 0.8, 1.0, 1.3, 2.0, 3.5, 8.0]


def pdf(x, alpha, beta):
    """Eq. 1 typed out in multi-precision (location 0)."""
    return beta / (2 * alpha * mp.gamma(1 / mp.mpf(beta))) * mp.e ** (-(abs(x) / alpha) ** beta)


def integrate(fn, alpha, beta):
    """Integral of fn(|x|) f(x) dx over the real line, f typed out above."""
    a, b = mp.mpf(alpha), mp.mpf(beta)
    if beta >= 1:
        return 2 * mp.quad(lambda x: fn(x) * pdf(x, a, b), [0, a / 2, a, 2 * a, 6 * a, 40 * a])
    # heavy tails: substitute x = alpha * y**(1/beta); f(x) dx becomes e^-y y^(1/beta-1) dy / Gamma(1/beta)

    def g(y):
        return fn(a * y ** (1 / b)) * mp.e ** (-y) * y ** (1 / b - 1)

    return mp.quad(g, [0, 1, 10, 50, 200, mp.inf]) / mp.gamma(1 / b)


def test_special_cases_gaussian_laplace_uniform():
    assert o.rho(2.0) == pytest.approx(2 / math.pi, rel=1e-14)      # Gaussian
    assert o.rho(1.0) == pytest.approx(0.5, rel=1e-14)              # Laplace
    assert o.rho(1e5) == pytest.approx(0.75, rel=1e-6)              # uniform limit
    # beta=2 is N(0, alpha^2/2); beta=1 is Laplace of scale alpha (variance 2 alpha^2)
    assert o.alpha_from_std(3.0, 2.0) == pytest.approx(3.0 * math.sqrt(2), rel=1e-14)
    assert o.alpha_from_std(3.0, 1.0) == pytest.approx(3.0 / math.sqrt(2), rel=1e-14)
    assert o.variance(0.7, 2.0) == pytest.approx(0.7 ** 2 / 2, rel=1e-14)
    assert o.variance(0.7, 1.0) == pytest.approx(2 * 0.7 ** 2, rel=1e-14)
    assert o.mean_abs(0.7, 1.0) == pytest.approx(0.7, rel=1e-14)
    assert o.mean_abs(0.7, 2.0) == pytest.approx(0.7 / math.sqrt(math.pi), rel=1e-14)
    # differential entropies of the two named special cases
    s = 1.9
    assert o.diff_entropy_nats(s * math.sqrt(2), 2.0) == pytest.approx(
        0.5 * math.log(2 * math.pi * math.e * s * s), rel=1e-13)
    assert o.diff_entropy_nats(0.3, 1.0) == pytest.approx(1 + math.log(2 * 0.3), rel=1e-13)


def test_rho_is_strictly_increasing():
    grid = np.exp(np.linspace(math.log(0.05), math.log(20.0), 2000))
    vals = np.array([o.log_rho(b) for b in grid])
    assert np.all(np.diff(vals) > 0)
    assert vals[-1] < math.log(0.75)


@pytest.mark.parametrize("beta", BETAS)
def test_moments_of_the_density_by_quadrature(beta):
    alpha = 0.37
    total = integrate(lambda x: 1, alpha, beta)
    m1 = integrate(lambda x: x, alpha, beta)           # E|x| (x >= 0 on the substituted axis)
    m2 = integrate(lambda x: x * x, alpha, beta)
    assert float(total) == pytest.approx(1.0, rel=1e-12)
    assert o.mean_abs(alpha, beta) == pytest.approx(float(m1), rel=1e-11)
    assert o.variance(alpha, beta) == pytest.approx(float(m2), rel=1e-11)
    assert o.rho(beta) == pytest.approx(float(m1 * m1 / m2), rel=1e-11)
    assert o.alpha_from_std(float(mp.sqrt(m2)), beta) == pytest.approx(alpha, rel=1e-11)


@pytest.mark.parametrize("beta", [0.25, 0.5, 1.0, 1.3, 2.0, 3.5])
def test_entropy_of_the_density_by_quadrature(beta):
    alpha = 0.37
    h = integrate(lambda x: -mp.log(pdf(x, alpha, beta)), alpha, beta)
    assert o.diff_entropy_nats(alpha, beta) == pytest.approx(float(h), rel=1e-11)


@pytest.mark.parametrize("beta", [0.3, 0.7, 1.0, 1.6, 2.0, 5.0])
def test_against_scipy_gennorm(beta):
    """scipy's generalized normal has the same density with scale = alpha."""
    alpha = 0.011
    d = scipy.stats.gennorm(beta, scale=alpha)
    assert o.variance(alpha, beta) == pytest.approx(d.var(), rel=1e-10)
    assert o.diff_entropy_nats(alpha, beta) == pytest.approx(float(d.entropy()), rel=1e-10)
    x = 0.004
    assert float(pdf(x, alpha, beta)) == pytest.approx(d.pdf(x), rel=1e-10)


def test_init_rule_reduces_to_he():
    """Shape 2 with the ReLU correction 2 gives variance 2/d_in (Eq. 4-5 and the remark after)."""
    for d_in in (64, 896, 4096, 11008):
        a = o.init_alpha(d_in, 2.0, 2.0)
        assert o.variance(a, 2.0) == pytest.approx(2.0 / d_in, rel=1e-13)
        for beta in (0.1, 0.5, 1.0, 1.3):
            a = o.init_alpha(d_in, 1.0, beta)
            assert o.variance(a, beta) == pytest.approx(1.0 / d_in, rel=1e-12)
            k = 0.2
            a = o.init_alpha(d_in, 2 / (1 + k * k), beta)
            assert o.variance(a, beta) == pytest.approx(2 / (1 + k * k) / d_in, rel=1e-12)


def test_table1_ordering():
    """Table 1: entropy grows with the shape parameter (only the order is checkable)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_gg_entropy.txt")
    rows = [tuple(map(float, l.split())) for l in open(path) if l.strip() and l[0] != "#"]
    shapes = [r[0] for r in rows]
    assert shapes == sorted(shapes)
    assert [r[1] for r in rows] == sorted(r[1] for r in rows)
    assert [r[2] for r in rows] == sorted(r[2] for r in rows)
    ours = [o.diff_entropy_nats(o.alpha_from_std(0.02, b), b) for b in shapes]
    assert ours == sorted(ours)
