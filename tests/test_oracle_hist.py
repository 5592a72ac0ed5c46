"""Pins for the oracle's quantiser, histogram and empirical entropy."""
import math
from fractions import Fraction

import numpy as np
import pytest

import gg_synth
from oracle import gg_oracle as o


def _brute_symbol(x, step, qmin, qmax):
    """The quantiser's definition in numpy scalar fp32 arithmetic."""
    inv = np.float32(1.0 / float(np.float32(step)))
    t = np.float32(np.float32(x) * inv)
    return int(min(max(math.floor(float(t)), qmin), qmax))


@pytest.mark.parametrize("step", [1e-3, 0.01, 2.0 ** -10, 3.7e-6])
def test_histogram_brute_force(step):
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(64) * 40 * step).astype(np.float32)
    x[:4] = [0.0, -0.0, step, -step]
    hist, cl = o.quantise_hist(x, step)
    ref = np.zeros(65536, dtype=np.uint64)
    for v in x:
        ref[_brute_symbol(v, step, -32768, 32767) + 32768] += 1
    np.testing.assert_array_equal(hist, ref)
    assert hist.sum() == 64 and cl.sum() == 0
    np.testing.assert_array_equal(o.quantise(x, step) + 32768,
                                  [_brute_symbol(v, step, -32768, 32767) + 32768 for v in x])


def test_power_of_two_step_is_the_exact_floor():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(64) * 0.05).astype(np.float32)
    for n_bits in (4, 10, 13):
        q = o.quantise(x, 2.0 ** -n_bits)
        ref = [math.floor(Fraction(float(v)) * 2 ** n_bits) for v in x]
        np.testing.assert_array_equal(q, ref)


def test_floor_is_asymmetric_about_zero():
    """x in [-step, 0) is symbol -1; mirroring the input maps symbol q to -q-1 off the grid."""
    step = 2.0 ** -6
    x = np.array([0.3 * step, 1.7 * step, 5.2 * step, 100.9 * step], dtype=np.float32)
    qp, qm = o.quantise(x, step), o.quantise(-x, step)
    np.testing.assert_array_equal(qp, [0, 1, 5, 100])
    np.testing.assert_array_equal(qm, -qp - 1)
    on_grid = np.array([step, 2 * step], dtype=np.float32)
    np.testing.assert_array_equal(o.quantise(-on_grid, step), [-1, -2])


def test_clamp_and_counters():
    step = 1.0
    x = np.array([-5.5, -3.0, -2.2, 0.5, 2.9, 3.0, 7.0, np.inf, -np.inf, np.nan], dtype=np.float32)
    hist, cl = o.quantise_hist(x, step, qmin=-3, qmax=2)
    # floor: -6,-3,-3,0,2,3,7,+inf,-inf ; nan skipped
    np.testing.assert_array_equal(hist, [4, 0, 0, 1, 0, 4])
    np.testing.assert_array_equal(cl, [2, 3])
    # accumulation into an existing table
    hist2, cl2 = o.quantise_hist(x, step, -3, 2, hist=hist.copy(), clamped=cl.copy())
    np.testing.assert_array_equal(hist2, 2 * hist)
    np.testing.assert_array_equal(cl2, 2 * cl)


def test_entropy_closed_forms():
    assert o.entropy_bits(np.zeros(16, np.uint64)) == 0.0
    h = np.zeros(16, np.uint64); h[5] = 12345
    assert o.entropy_bits(h) == 0.0
    for m in (2, 8, 1024, 65536):
        assert o.entropy_bits(np.full(m, 7, np.uint64)) == pytest.approx(math.log2(m), abs=1e-12)
    # a dyadic distribution: probabilities 1/2, 1/4, 1/8, 1/8 -> 1.75 bits
    assert o.entropy_bits(np.array([8, 4, 2, 2], np.uint64)) == pytest.approx(1.75, abs=1e-14)
    # against the plain -sum p log2 p
    rng = np.random.default_rng(0)
    c = rng.integers(0, 1000, 500).astype(np.uint64)
    p = c[c > 0] / c.sum()
    assert o.entropy_bits(c) == pytest.approx(float(-(p * np.log2(p)).sum()), abs=1e-12)


@pytest.mark.parametrize("beta", [0.8, 1.0, 2.0])
def test_fine_step_entropy_approaches_differential_entropy(beta):
    """H(quantised) + log2(step) -> h(GG)/ln 2 as the step shrinks (large sample)."""
    rng = np.random.default_rng(6)
    alpha = gg_synth.alpha_for_std(1.0, beta)
    x = gg_synth.gg_host(rng, beta, alpha, 4_000_000).numpy()
    step = 2.0 ** -5
    hist, cl = o.quantise_hist(x, step)
    assert cl.sum() == 0
    h = o.entropy_bits(hist) + math.log2(step)
    assert h == pytest.approx(o.diff_entropy_nats(alpha, beta) / math.log(2), abs=0.01)
