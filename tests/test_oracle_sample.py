"""Pins for the oracle's Philox stream and GG sampler."""
import math
import os
import shutil
import subprocess

import numpy as np
import pytest
import scipy.stats

from oracle import gg_oracle as o

HERE = os.path.dirname(os.path.abspath(__file__))


def test_philox_known_answers():
    path = os.path.join(HERE, "golden", "philox4x32_10_kat.txt")
    rows = [l.split() for l in open(path) if l.strip() and l[0] != "#"]
    assert len(rows) >= 3
    for r in rows:
        v = [int(h, 16) for h in r]
        np.testing.assert_array_equal(o.philox4x32_10(v[0:4], v[4:6]), v[6:10])


@pytest.mark.skipif(shutil.which("nvcc") is None, reason="needs nvcc for the toolkit header")
def test_philox_against_the_toolkit_generator(tmp_path):
    exe = tmp_path / "philox_crosscheck"
    subprocess.run(["nvcc", "-O1", "-o", str(exe), os.path.join(HERE, "philox_crosscheck.cu")],
                   check=True, capture_output=True)
    rng = np.random.default_rng(0)
    cases = rng.integers(0, 2 ** 32, size=(200, 6), dtype=np.uint64)
    cases[0] = 0
    cases[1] = 0xFFFFFFFF
    cases[2] = [5, 0, 0, 0, 0, 0]
    cases[3] = [0, 0, 0xFFFFFFFF, 7, 1, 0]
    text = "\n".join(" ".join(f"{int(v):x}" for v in row) for row in cases) + "\n"
    out = subprocess.run([str(exe)], input=text, capture_output=True, text=True, check=True).stdout
    got = [[int(h, 16) for h in l.split()] for l in out.strip().splitlines()]
    assert len(got) == len(cases)
    for row, ref in zip(cases, got):
        np.testing.assert_array_equal(o.philox4x32_10(row[0:4], row[4:6]), ref)


def test_philox_words_are_uniform_and_counter_sensitive():
    words = np.array([o.philox4x32_10([i, 0, 0, 0], [1, 2]) for i in range(20000)], dtype=np.uint64)
    u = (words + 0.5) / 2.0 ** 32
    for k in range(4):
        assert scipy.stats.kstest(u[:, k], "uniform").pvalue > 1e-4
    bits = ((words[:, :, None] >> np.arange(32, dtype=np.uint64)) & 1).mean(axis=(0, 1))
    assert np.all(np.abs(bits - 0.5) < 0.01)
    base = o.philox4x32_10([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        c = [1, 2, 3, 4]; c[pos] ^= 1
        assert not np.array_equal(o.philox4x32_10(c, [5, 6]), base)
    assert not np.array_equal(o.philox4x32_10([1, 2, 3, 4], [5, 7]), base)
    assert not np.array_equal(o.philox4x32_10([1, 2, 3, 4], [4, 6]), base)


def test_box_muller_normals():
    z = np.array([o.sample_debug(1.0, 9, 3, i)[0] for i in range(50000)])
    assert scipy.stats.kstest(z, "norm").pvalue > 1e-4


@pytest.mark.parametrize("beta", [0.1, 0.5, 0.8, 1.0, 1.3, 2.0, 3.0])
def test_sample_distribution_and_moments(beta):
    alpha, n = 0.37, 400_000
    x, att = o.sample(beta, alpha, seed=1234, tensor_id=3, n=n, want_attempts=True)
    assert att.max() <= o.SAMPLE_MAX_ATTEMPTS and att.min() >= 1
    # (|x|/alpha)^beta ~ Gamma(1/beta, 1)
    y = (np.abs(x) / alpha) ** beta
    assert scipy.stats.kstest(y, scipy.stats.gamma(1.0 / beta).cdf).pvalue > 1e-4
    # moments of the density (Eq. 3 and its first-moment analogue), 5 standard errors
    m1, m2 = o.mean_abs(alpha, beta), o.variance(alpha, beta)
    g = lambda k: math.lgamma(k / beta)
    m4 = alpha ** 4 * math.exp(g(5) - g(1))
    assert abs(np.abs(x).mean() - m1) < 5 * math.sqrt((m2 - m1 * m1) / n)
    if beta >= 0.5:    # below that the fourth moment makes the bound useless at this n
        assert abs((x * x).mean() - m2) < 5 * math.sqrt((m4 - m2 * m2) / n)
    # sign balance
    assert abs((x > 0).mean() - 0.5) < 5 * 0.5 / math.sqrt(n)


def test_sample_special_cases_are_gaussian_and_laplace():
    n, alpha = 200_000, 1.5
    x = o.sample(2.0, alpha, 7, 0, n)
    assert scipy.stats.kstest(x, scipy.stats.norm(scale=alpha / math.sqrt(2)).cdf).pvalue > 1e-4
    x = o.sample(1.0, alpha, 7, 1, n)
    assert scipy.stats.kstest(x, scipy.stats.laplace(scale=alpha).cdf).pvalue > 1e-4
    x = o.sample(0.5, alpha, 7, 2, n)
    assert scipy.stats.kstest(x, scipy.stats.gennorm(0.5, scale=alpha).cdf).pvalue > 1e-4


def test_sample_is_counter_based():
    """Any sub-range regenerates alone; tensor id and seed select independent streams."""
    full = o.sample(1.3, 0.02, 42, 5, 1000)
    part = o.sample(1.3, 0.02, 42, 5, 100, index0=300)
    np.testing.assert_array_equal(full[300:400], part)
    far = o.sample(1.3, 0.02, 42, 5, 4, index0=2 ** 33 + 1)
    assert all(o.lib().ggo_sample_one(1.3, 0.02, 42, 5, 2 ** 33 + 1 + i, None) == far[i] for i in range(4))
    assert not np.array_equal(full[:100], o.sample(1.3, 0.02, 42, 6, 100))
    assert not np.array_equal(full[:100], o.sample(1.3, 0.02, 43, 5, 100))
    # scale is a pure multiplier
    np.testing.assert_allclose(o.sample(1.3, 0.04, 42, 5, 1000), 2 * full, rtol=1e-15)


def test_acceptance_rule_by_brute_force():
    """Replay attempt by attempt from the exposed intermediates."""
    beta, seed, tid = 0.7, 99, 2
    x, att = o.sample(beta, 1.0, seed, tid, 2000, want_attempts=True)
    assert (att > 1).any()                   # some rejections occur in 2000 draws
    for i in range(2000):
        t = 0
        while True:
            z, lhs, rhs = o.sample_debug(beta, seed, tid, i, t)
            if lhs < rhs:
                break
            t += 1
        assert att[i] == t + 1
    a = 1 / beta
    d = a - 1 / 3
    accept_rate = 1.0 / att.mean()
    assert accept_rate > 0.9                 # Marsaglia-Tsang accepts > 95 % for shape >= 1


def test_bf16_rounding_helper():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 0.0,
                  1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 2.0 ** -8 - 2.0 ** -40])
    np.testing.assert_array_equal(o.round_to_bf16_bits(x),
                                  [0x3F80, 0x3F80, 0x3F82, 0xBF80, 0, 0x3F81, 0x3F80])
    np.testing.assert_array_equal(o.bf16_bits_to_f32([0x3F80, 0xBF80, 0x3F81]),
                                  np.array([1.0, -1.0, 1.0078125], np.float32))
