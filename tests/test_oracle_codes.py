"""Pins for the oracle's code-length functions (Eq. 6-7, Huffman, fixed length) and the GCT step."""
import heapq
import math
import os

import numpy as np
import pytest

import gg_synth
from oracle import gg_oracle as o

HERE = os.path.dirname(os.path.abspath(__file__))


def test_map_is_the_bijection_of_eq_6():
    # negative -> even, positive -> odd, zero -> zero; onto 0..2N without gaps
    qs = list(range(-500, 501))
    ms = [o.map_unsigned(q) for q in qs]
    assert sorted(ms) == list(range(0, 1001))
    assert all(o.map_unsigned(q) == -2 * q for q in range(-500, 0))
    assert all(o.map_unsigned(q) == 2 * q - 1 for q in range(1, 501))
    assert o.map_unsigned(0) == 0


@pytest.mark.parametrize("k", [0, 1, 2, 3, 5])
def test_eg_lengths_form_a_complete_prefix_code(k):
    # order-k code: 2^k words of length k+1, then 2^(k+1) of length k+3, ...; Kraft sum exactly 1
    lens = [o.eg_length(m, k) for m in range((1 << (k + 12)) - (1 << k))]
    if k == 0:
        assert lens[:7] == [1, 3, 3, 5, 5, 5, 5]
    assert lens == sorted(lens)
    group, start, L = 1 << k, 0, k + 1
    while start + group <= len(lens):
        assert set(lens[start:start + group]) == {L}
        start, group, L = start + group, group * 2, L + 2
    kraft = sum(2.0 ** -l for l in lens)
    assert kraft == pytest.approx(1.0 - 2.0 ** -12, abs=1e-12)      # the first 12 groups of the infinite code
    # the definition with the logarithm written out
    for m in (0, 1, 2, 3, 100, 12345, 2 ** 31):
        assert o.eg_length(m, k) == 2 * int(math.floor(math.log2(m + 2 ** k))) - k + 1


@pytest.mark.parametrize("k", [0, 2])
def test_eg_rate_from_histogram_equals_the_elementwise_mean(k):
    rng = np.random.default_rng(8)
    x = gg_synth.gg_host(rng, 0.8, 0.05, 50_000).numpy()
    step = 2.0 ** -8
    hist, _ = o.quantise_hist(x, step)
    assert o.eg_rate(x, step, k) == pytest.approx(o.eg_rate_hist(hist, k), rel=1e-15)
    # brute force in Python on a few elements
    q = o.quantise(x[:200], step)
    brute = np.mean([o.eg_length(o.map_unsigned(int(v)), k) for v in q])
    assert o.eg_rate(x[:200], step, k) == pytest.approx(brute, rel=1e-15)
    # a narrow clamp moves symbols to the edge bins before they are coded
    q = np.clip(o.quantise(x[:500], step, -3, 4), -3, 4)
    assert o.eg_rate(x[:500], step, k, -3, 4) == pytest.approx(
        np.mean([o.eg_length(o.map_unsigned(int(v)), k) for v in q]), rel=1e-15)


def test_eg_rate_gradient_is_the_derivative_of_the_relaxed_rate():
    """With floor and Map read as straight-through (slope 1/step and 2), R = (1/N) sum 2 log2(m + 2^k) + const;
    its derivative at the quantised point is 4 / (step N ln 2 (m + 2^k)) with the sign of x."""
    rng = np.random.default_rng(9)
    x = gg_synth.gg_host(rng, 1.0, 0.1, 64).numpy()
    x[:3] = [0.0, -0.0, 1e-9]
    step, k, lam = 2.0 ** -6, 1, 0.37
    g = o.eg_rate_grad(x, step, lam, k)
    q = o.quantise(x, step)
    for xi, qi, gi in zip(x, q, g):
        m = o.map_unsigned(int(qi))
        want = 0.0 if xi == 0 else math.copysign(lam * 4.0 / (step * 64 * math.log(2.0) * (m + 2 ** k)), xi)
        assert gi == pytest.approx(want, rel=1e-14, abs=0.0)
    assert g[0] == 0.0 and g[1] == 0.0 and g[2] > 0          # sign(0) = 0; a tiny positive value has m = 0
    # finite difference of the relaxed rate in the unsigned symbol: d/dm [2 log2(m + 2^k)] = 2 / ((m + 2^k) ln 2)
    m, h = 7.0, 1e-6
    fd = (2 * math.log2(m + h + 2 ** k) - 2 * math.log2(m - h + 2 ** k)) / (2 * h)
    assert fd == pytest.approx(2 / ((m + 2 ** k) * math.log(2.0)), rel=1e-8)


@pytest.mark.parametrize("k, qmin, qmax", [(0, -32768, 32767), (3, -32768, 32767), (1, -5, 4)])
def test_eg_rate_gradient_against_a_numerical_derivative_in_mpmath(k, qmin, qmax):
    """The relaxed rate (Eq. 6-7 with floor and Map taken as straight-through: slopes 1/step and 2) is
    R(d) = (1/N) sum_j 2 log2(M_j + 2 (|x_j + d_j| - |x_j|) / step + 2^k) with M_j the mapped symbol of the
    quantised x_j.  Its partial derivatives at d = 0, taken numerically in 40-digit arithmetic, are what
    the dR/dG line of the GCT section states.  Symbols are computed here in numpy fp32, not by the oracle."""
    mpmath = pytest.importorskip("mpmath")
    mp = mpmath.mp
    rng = np.random.default_rng(19)
    n = 72
    x = gg_synth.gg_host(rng, 0.9, 0.2, n).numpy().astype(np.float32)
    x[:4] = [0.0, -0.0, 3e-7, -3e-7]                    # zeros: no gradient; a tiny negative value falls in symbol -1
    x[4:6] = [7.5, -7.5]                                # clamped under the narrow range
    step, lam = np.float32(2.0 ** -5), 0.81
    inv = np.float32(1.0 / np.float64(step))
    q = np.clip(np.floor((x * inv).astype(np.float32)).astype(np.int64), qmin, qmax)
    M = [(-2 * int(v)) if v < 0 else (0 if v == 0 else 2 * int(v) - 1) for v in q]
    assert any(v in (qmin, qmax) for v in q) == (qmax < 100)
    got = o.eg_rate_grad(x, float(step), lam, k, qmin, qmax)
    old = mp.dps
    mp.dps = 40
    try:
        xs = [mpmath.mpf(float(v)) for v in x]
        for i in range(n):
            if x[i] == 0:
                assert got[i] == 0.0
                continue

            def rate(d, i=i):
                tot = mpmath.mpf(0)
                for j in range(n):
                    dj = d if j == i else 0
                    tot += 2 * mpmath.log(M[j] + 2 * (abs(xs[j] + dj) - abs(xs[j])) / mpmath.mpf(float(step)) + 2 ** k, 2)
                return lam * tot / n

            want = mpmath.diff(rate, 0, h=mpmath.mpf(10) ** -12)
            assert float(abs(got[i] - want) / abs(want)) < 1e-13, (i, got[i], want)
    finally:
        mp.dps = old


def _huffman_heap(counts):
    h = [int(c) for c in counts if c]
    if len(h) <= 1:
        return 0.0
    heapq.heapify(h)
    tot, s = sum(h), 0
    while len(h) > 1:
        a, b = heapq.heappop(h), heapq.heappop(h)
        s += a + b
        heapq.heappush(h, a + b)
    return s / tot


def test_huffman_bits_textbook_cases_and_entropy_bounds():
    assert o.huffman_bits(np.array([1, 1, 2, 4], dtype=np.uint64)) == 1.75          # lengths 3, 3, 2, 1
    assert o.huffman_bits(np.array([5, 0, 0], dtype=np.uint64)) == 0.0
    assert o.huffman_bits(np.array([3, 3], dtype=np.uint64)) == 1.0
    # a dyadic distribution is coded at its entropy
    d = np.array([8, 4, 2, 1, 1], dtype=np.uint64)
    assert o.huffman_bits(d) == pytest.approx(o.entropy_bits(d), rel=1e-15)
    rng = np.random.default_rng(10)
    for _ in range(20):
        c = rng.integers(0, 1000, rng.integers(2, 400)).astype(np.uint64)
        if np.count_nonzero(c) < 2:
            continue
        hm, H = o.huffman_bits(c), o.entropy_bits(c)
        assert H - 1e-12 <= hm < H + 1
        assert hm == pytest.approx(_huffman_heap(c), rel=1e-14)                      # heap construction, same optimum


def test_fixed_length_bits():
    z = np.zeros(64, dtype=np.uint64)
    assert o.fixed_length_bits(z) == 0
    z[10] = 1
    assert o.fixed_length_bits(z) == 0
    z[13] = 5
    assert o.fixed_length_bits(z) == 2          # symbols 10..13: four values
    z[14] = 1
    assert o.fixed_length_bits(z) == 3          # five values
    z[0] = 1
    z[63] = 1
    assert o.fixed_length_bits(z) == 6


def test_compression_ratio_reproduces_table_4():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "table4_code_lengths.txt")) if l[0] != "#"]
    assert len(rows) == 10
    for eg, hm, fl, ceg, chm in rows:
        assert 100 * o.compression_ratio(float(eg), float(fl)) == pytest.approx(float(ceg), abs=0.006)
        assert 100 * o.compression_ratio(float(hm), float(fl)) == pytest.approx(float(chm), abs=0.006)


def test_gct_step_follows_algorithm_2():
    rng = np.random.default_rng(12)
    n = 40
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    gp = rng.standard_normal(n) * 1e-3
    w = rng.standard_normal(n)
    eta, lam, eps, step = 1e-3, 0.2, 1e-8, 2.0 ** -12
    # first step: no second-order term, plain gradient descent
    gh, wn = o.gct_step(g, gp, w, step, eta, lam, eps, t=1)
    np.testing.assert_array_equal(gh, g.astype(np.float64))
    np.testing.assert_allclose(wn, w - eta * g.astype(np.float64), rtol=0, atol=0)
    # later steps, written out in Python
    gh, wn = o.gct_step(g, gp, w, step, eta, lam, eps, t=2)
    dr = o.eg_rate_grad(g, step, 1.0)
    h = -(1 / eta) * g.astype(np.float64) / (gp + eps) + 1 / eta
    np.testing.assert_allclose(gh, g + lam * dr * h, rtol=1e-15)
    np.testing.assert_allclose(wn, w - eta * (g + lam * dr * h), rtol=1e-15)
    # a gradient equal to the stored one (and eps = 0) has zero curvature estimate: nothing is added
    gh, _ = o.gct_step(g, g.astype(np.float64), w, step, eta, lam, 0.0, t=5)
    np.testing.assert_allclose(gh, g.astype(np.float64), rtol=0, atol=1e-18)


def test_gct_step_hand_computed_case():
    """Algorithm 2 on three elements, every intermediate written down.
    step 1/4, k = 0: g = (1/2, -1/4, 1/8) scales to (2, -1, 1/2), symbols (2, -1, 0), Eq. 6 maps them to (3, 2, 0).
    dR/dg = 4 * 4 / (3 ln 2) * sign / (m + 1) = 7.694373551407805 * (1/4, -1/3, 1).
    eta = 1/2, eps = 1/4, stored gradients (3/4, -3/4, 1): h = 2 - 2 g / (stored + eps) = (1, 1, 9/5).
    lambda = 1/8: ghat = g + lambda * dR/dg * h;  w = (1, 2, 3) - eta * ghat."""
    g = np.array([0.5, -0.25, 0.125], dtype=np.float32)
    stored = np.array([0.75, -0.75, 1.0])
    w = np.array([1.0, 2.0, 3.0])
    dr = o.eg_rate_grad(g, 0.25, 1.0, 0)
    np.testing.assert_allclose(dr, [1.9235933878519512, -2.5647911838026016, 7.694373551407805], rtol=4e-16)
    gh, wn = o.gct_step(g, stored, w, 0.25, 0.5, 0.125, 0.25, t=2)
    np.testing.assert_allclose(gh, [0.7404491734814939, -0.5705988979753252, 1.856234049066756], rtol=4e-16)
    np.testing.assert_allclose(wn, [0.6297754132592530, 2.2852994489876626, 2.0718829754666220], rtol=4e-16)
    # the first step of training has no stored gradient: plain descent
    gh, wn = o.gct_step(g, stored, w, 0.25, 0.5, 0.125, 0.25, t=1)
    np.testing.assert_array_equal(gh, [0.5, -0.25, 0.125])
    np.testing.assert_array_equal(wn, [0.75, 2.125, 2.9375])
