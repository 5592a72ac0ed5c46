"""GPU parity: every step of the CUDA pass against the fp64 CPU oracle, element by element, on
seeded inputs that span several tiles and ragged tails, plus the degenerate cases.

All calls go through the C interface (ctypes binding).  Gradient, penalty and histogram parity
is always evaluated with the parameter bits the GPU used (its own fit, read back)."""
import math

import numpy as np
import pytest
import torch

import gg_synth
from oracle import gg_oracle as o
from parity_util import (ABS_ENTROPY, REL_FIT, REL_PENALTY, assert_grad_close, assert_rel)

pytestmark = pytest.mark.gpu

TILE = 16384


@pytest.fixture(scope="module")
def ctx():
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import Context
    c = Context(0, guard=True)        # fill patterns around every output the binding allocates
    yield c
    c.close()


@pytest.fixture(autouse=True)
def outputs_stay_inside_their_buffers(ctx):
    """After every test: no kernel wrote before or after a fit result, penalty, histogram, entropy or counter."""
    yield
    ctx.check_guards()


def dev(t):
    return t.to("cuda:0")


def make_segments(dtype, seed=0):
    """Ragged segment set: sub-tile, exact tile, multi-tile with tail, tiny, misaligned views."""
    rng = np.random.default_rng(seed)
    spec = [(0.5, 3e-4, 3 * TILE + 1234), (0.8, 1.0, TILE), (1.0, 0.02, 1), (1.3, 0.014, 7),
            (2.0, 0.03, 2 * TILE + 5), (1.6, 0.02, 4096), (0.6, 0.004, 70001), (1.0, 0.5, 33)]
    return [gg_synth.gg_host(rng, b, a, n, dtype) for b, a, n in spec]


def misaligned_views(tensors, offsets=(1, 3, 5, 2, 7, 0, 9, 6)):
    """Device copies whose first element sits `off` elements past a 256-byte boundary."""
    out = []
    for t, off in zip(tensors, offsets):
        buf = torch.zeros(t.numel() + 16, dtype=t.dtype, device="cuda:0")
        buf[off:off + t.numel()].copy_(t)
        out.append(buf[off:off + t.numel()])
    return out


# --------------------------------------------------------------------------------------- gg_fit
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("misalign", [False, True])
def test_fit_parity(ctx, dtype, misalign):
    xs = make_segments(dtype)
    xd = misaligned_views(xs) if misalign else [dev(x) for x in xs]
    out = ctx.gg_fit(xd)
    torch.cuda.synchronize()
    for s, x in enumerate(xs):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(x))
        assert out["count"][s].item() == n
        assert out["flags"][s].item() == fl
        assert_rel(out["sum_abs"][s].item(), s1, 1e-7, "sum_abs")
        assert_rel(out["sum_sq"][s].item(), s2, 1e-7, "sum_sq")
        if fl & (o.FLAG_BETA_CLAMPED_HI | o.FLAG_BETA_CLAMPED_LO):
            assert out["beta"][s].item() == b
        else:
            assert_rel(out["beta"][s].item(), b, REL_FIT, "beta")
        assert_rel(out["alpha"][s].item(), a, REL_FIT, "alpha")


def test_fit_degenerate_and_flags(ctx):
    xs = [torch.zeros(0), torch.zeros(100), torch.tensor([1.0, -1.0]), torch.tensor([1.0, 2.0, 3.0]),
          torch.tensor([1.0, float("inf"), -2.0, float("nan"), 3.0] * 50),
          torch.cat([torch.ones(1), torch.zeros(10 ** 6)])]
    out = ctx.gg_fit([dev(x) for x in xs])
    torch.cuda.synchronize()
    for s, x in enumerate(xs):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(x))
        assert out["flags"][s].item() == fl, s
        assert out["count"][s].item() == n
        assert out["beta"][s].item() == pytest.approx(b, rel=REL_FIT)
        assert out["alpha"][s].item() == pytest.approx(a, rel=REL_FIT)
        assert out["sum_abs"][s].item() == pytest.approx(s1, rel=1e-7)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_fit_with_magnitudes_whose_squares_leave_the_fp32_range(ctx, dtype):
    """|x| above 1.8e19 squares to more than fp32 holds; the moments must still be those of the oracle."""
    rng = np.random.default_rng(17)
    x = gg_synth.gg_host(rng, 0.7, 1e22, 3 * TILE + 50, torch.float32)
    x[::97] = 3.0e38
    x[5::89] = -2.5e38
    x = x.to(dtype)
    out = ctx.gg_fit([dev(x), dev(x[:1000])])
    torch.cuda.synchronize()
    for s, xs in enumerate((x, x[:1000])):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(xs))
        assert out["flags"][s].item() == fl
        assert_rel(out["sum_abs"][s].item(), s1, 1e-7, "sum_abs")
        assert_rel(out["sum_sq"][s].item(), s2, 1e-7, "sum_sq")
        assert_rel(out["beta"][s].item(), b, REL_FIT, "beta")
        assert_rel(out["alpha"][s].item(), a, REL_FIT, "alpha")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_fit_with_magnitudes_whose_squares_fall_below_the_fp32_range(ctx, dtype):
    """|x| below 1e-19 squares into the fp32 subnormals or to zero; the moments must still be those of the
    oracle, through the long-segment kernels and through the one-warp-per-segment kernel."""
    from paper_2506_00486_b200 import Segments
    rng = np.random.default_rng(18)
    x = gg_synth.gg_host(rng, 0.9, 1e-26, 3 * TILE + 50, torch.float32).to(dtype)
    x[::101] = 0
    out = ctx.gg_fit([dev(x), dev(x[:1000])])
    torch.cuda.synchronize()
    for s, xs in enumerate((x, x[:1000])):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(xs))
        assert out["flags"][s].item() == fl
        assert_rel(out["sum_abs"][s].item(), s1, 1e-7, "sum_abs")
        assert_rel(out["sum_sq"][s].item(), s2, 1e-7, "sum_sq")
        assert_rel(out["beta"][s].item(), b, REL_FIT, "beta")
        assert_rel(out["alpha"][s].item(), a, REL_FIT, "alpha")
    if dtype == torch.bfloat16:
        xs = [x[i * 500:(i + 1) * 500] for i in range(70)]
        out = ctx.gg_fused(Segments([dev(t) for t in xs]), want_penalty=False, want_hist=False)
        torch.cuda.synchronize()
        for s, t in enumerate(xs):
            b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(t))
            assert out["flags"][s].item() == fl
            assert_rel(out["sum_sq"][s].item(), s2, 1e-7, "sum_sq")
            assert_rel(out["beta"][s].item(), b, REL_FIT, "beta")
            assert_rel(out["alpha"][s].item(), a, REL_FIT, "alpha")


def test_fit_over_the_whole_shape_range(ctx):
    """beta from 0.1 to 8 on large samples: the fitted pair matches the oracle's."""
    rng = np.random.default_rng(21)
    betas = [0.1, 0.2, 0.35, 0.5, 0.7, 1.0, 1.4, 2.0, 3.0, 5.0, 8.0]
    xs = [gg_synth.gg_host(rng, b, 0.05, 200_000, torch.float32) for b in betas]
    out = ctx.gg_fit([dev(x) for x in xs])
    torch.cuda.synchronize()
    for s, x in enumerate(xs):
        b, a, *_ = o.fit(gg_synth.to_oracle(x))
        assert_rel(out["beta"][s].item(), b, REL_FIT, f"beta (true {betas[s]})")
        assert_rel(out["alpha"][s].item(), a, REL_FIT, f"alpha (true {betas[s]})")


def test_fit_is_deterministic(ctx):
    xs = [dev(x) for x in make_segments(torch.bfloat16, seed=3)]
    a = ctx.gg_fit(xs)
    b = ctx.gg_fit(xs)
    torch.cuda.synchronize()
    for k in ("beta", "alpha", "sum_abs", "sum_sq"):
        assert torch.equal(a[k].view(torch.int64), b[k].view(torch.int64))


# ------------------------------------------------------------------------------ gg_penalty_grad
SPECIALS = [0.0, -0.0, 1e-45, -1e-45, 1e-40, 1.17549435e-38, -1.17549435e-38, 3.0e38, -3.0e38, 1.0, -1.0,
            2.0, 0.5, 1.4142135, 0.70710678, 1.9999999, 1.0000001]


def penalty_case(ctx, x_host, beta, alpha, lam, misalign=False, grad_dtype=torch.float32, reduction=0):
    from paper_2506_00486_b200 import Segments
    xd = misaligned_views([x_host], offsets=(3,))[0] if misalign else dev(x_host)
    gbuf = torch.full((x_host.numel() + 16,), 7.0, dtype=grad_dtype, device="cuda:0")
    off = 5 if misalign else 0
    gd = gbuf[off:off + x_host.numel()]
    bt = torch.tensor([beta], dtype=torch.float64, device="cuda:0")
    at = torch.tensor([alpha], dtype=torch.float64, device="cuda:0")
    pen = ctx.gg_penalty_grad(Segments([xd]), bt, at, lam, grad=Segments([gd]), reduction=reduction)
    torch.cuda.synchronize()
    # nothing outside the segment was touched
    assert (gbuf[:off] == 7.0).all() and (gbuf[off + x_host.numel():] == 7.0).all()
    return pen[0].item(), gd.float().cpu().numpy()


@pytest.mark.parametrize("beta,alpha", [(0.5, 3e-4), (0.8, 1.1), (1.0, 0.02), (1.3, 0.014), (1.6, 0.02),
                                        (2.0, 0.03), (3.0, 0.5), (0.05, 1e-3), (0.1, 0.01),
                                        (3.7, 0.5), (8.0, 1.0), (20.0, 2.0)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_penalty_grad_parity(ctx, beta, alpha, dtype):
    rng = np.random.default_rng(int(beta * 1000))
    n = 2 * TILE + 777
    x = gg_synth.gg_host(rng, min(beta, 4.0), alpha, n, torch.float32)
    x[:len(SPECIALS)] = torch.tensor(SPECIALS)
    # a wide sweep of magnitudes: every binade from 2^-40 to 2^40 around alpha
    sweep = alpha * np.exp2(rng.uniform(-40, 40, 4000)) * rng.choice([-1.0, 1.0], 4000)
    x[100:4100] = torch.from_numpy(sweep.astype(np.float32))
    x = x.to(dtype)
    lam = 1e-4
    pen, g = penalty_case(ctx, x, beta, alpha, lam)
    xo = gg_synth.to_oracle(x)
    ref_pen, ref_g = o.penalty_grad(xo, beta, alpha, lam)
    worst = assert_grad_close(g, ref_g)
    assert worst <= 4
    if math.isfinite(ref_pen) and ref_pen < 1e300:
        assert_rel(pen, ref_pen, REL_PENALTY, "penalty")


def test_penalty_grad_misaligned_bf16_out_mean_and_accumulate(ctx):
    from paper_2506_00486_b200 import Segments, GG_MEAN
    rng = np.random.default_rng(9)
    n = TILE + 301
    x = gg_synth.gg_host(rng, 1.3, 0.02, n, torch.bfloat16)
    xo = gg_synth.to_oracle(x)
    # misaligned input and output, fp32 gradient
    pen, g = penalty_case(ctx, x, 1.3, 0.0141, 1e-4, misalign=True)
    ref_pen, ref_g = o.penalty_grad(xo, 1.3, 0.0141, 1e-4)
    assert_grad_close(g, ref_g)
    assert_rel(pen, ref_pen, REL_PENALTY, "penalty")
    # mean reduction = lambda / len
    pen, g = penalty_case(ctx, x, 1.3, 0.0141, 1e-4, reduction=GG_MEAN)
    ref_pen, ref_g = o.penalty_grad(xo, 1.3, 0.0141, 1e-4 / n)
    assert_grad_close(g, ref_g)
    assert_rel(pen, ref_pen, REL_PENALTY, "penalty(mean)")
    # bf16 gradient output: the fp32 result rounded once more (within one bf16 ulp of the oracle)
    pen, g = penalty_case(ctx, x, 1.3, 0.0141, 1e-4, grad_dtype=torch.bfloat16)
    ref_pen, ref_g = o.penalty_grad(xo, 1.3, 0.0141, 1e-4)
    ref_bits = o.round_to_bf16_bits(ref_g).astype(np.int64)
    got_bits = torch.from_numpy(g).to(torch.bfloat16).view(torch.int16).numpy().astype(np.int64) & 0xFFFF
    assert np.abs((ref_bits & 0x7FFF) - (got_bits & 0x7FFF)).max() <= 1
    assert ((ref_bits >> 15) == (got_bits >> 15)).all()
    # accumulate: grad += g
    xd = dev(x)
    gd = torch.full((n,), 0.25, dtype=torch.float32, device="cuda:0")
    bt = torch.tensor([1.3], dtype=torch.float64, device="cuda:0")
    at = torch.tensor([0.0141], dtype=torch.float64, device="cuda:0")
    ctx.gg_penalty_grad(Segments([xd]), bt, at, 1e-4, grad=Segments([gd]), accumulate=True)
    torch.cuda.synchronize()
    expect = (np.float32(0.25) + ref_g.astype(np.float32)).astype(np.float32)
    assert np.abs(gd.cpu().numpy() - expect).max() <= 4 * np.spacing(np.float32(0.25))


def test_penalty_grad_degenerate_parameters_and_zero_lambda(ctx):
    x = torch.tensor([1.0, -2.0, 0.0, 3.0])
    for beta, alpha, lam in ((0.0, 0.0, 1e-4), (1.0, 0.02, 0.0)):
        pen, g = penalty_case(ctx, x, beta, alpha, lam)
        assert pen == 0.0 and not g.any()
    # negative lambda flips the sign
    pen, g = penalty_case(ctx, x, 1.5, 0.5, -1e-3)
    ref_pen, ref_g = o.penalty_grad(x.numpy(), 1.5, 0.5, -1e-3)
    assert_grad_close(g, ref_g)
    assert_rel(pen, ref_pen, REL_PENALTY, "penalty")


# --------------------------------------------------------------------------------- gg_rate_hist
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("step", [1e-3, 0.01, 2.0 ** -10])
def test_rate_hist_parity(ctx, dtype, step):
    xs = make_segments(dtype, seed=5)
    xd = [dev(x) for x in xs]
    steps = torch.tensor([step * (1 + 0.37 * s) for s in range(len(xs))], dtype=torch.float32, device="cuda:0")
    out = ctx.gg_rate_hist(xd, steps)
    torch.cuda.synchronize()
    hist = out["hist"].cpu().numpy()
    for s, x in enumerate(xs):
        ref, cl = o.quantise_hist(gg_synth.to_oracle(x), steps[s].item())
        np.testing.assert_array_equal(hist[s], ref.astype(np.int64))
        np.testing.assert_array_equal(out["clamped"][s].cpu().numpy(), cl.astype(np.int64))
        assert abs(out["entropy_bits"][s].item() - o.entropy_bits(ref)) <= ABS_ENTROPY


def test_rate_hist_shared_histogram_clamp_window_and_specials(ctx):
    """Several segments into one table; narrow clamp; symbols outside the on-chip window;
    inf / nan entries; accumulation across calls."""
    rng = np.random.default_rng(6)
    xs = [gg_synth.gg_host(rng, 0.8, 1.0, 40000, torch.bfloat16) for _ in range(3)]
    xs[1][:6] = torch.tensor([float("inf"), float("-inf"), float("nan"), 1e30, -1e30, 0.0]).to(torch.bfloat16)
    xs[2] = gg_synth.add_outliers_host(rng, xs[2], 0.01, 25.0)      # symbols +-2500: outside the window
    xd = [dev(x) for x in xs]
    steps = torch.tensor([0.01, 0.01, 0.01], dtype=torch.float32, device="cuda:0")
    for qmin, qmax in ((-32768, 32767), (-100, 50), (3, 9), (-4000, -2100)):
        out = ctx.gg_rate_hist(xd, steps, hist_id=[0, 1, 0], n_hist=2, qmin=qmin, qmax=qmax)
        torch.cuda.synchronize()
        nb = qmax - qmin + 1
        ref = np.zeros((2, nb), dtype=np.uint64)
        cl = np.zeros((2, 2), dtype=np.uint64)
        for s, h in enumerate([0, 1, 0]):
            o.quantise_hist(gg_synth.to_oracle(xs[s]), 0.01, qmin, qmax, hist=ref[h], clamped=cl[h])
        np.testing.assert_array_equal(out["hist"].cpu().numpy(), ref.astype(np.int64))
        np.testing.assert_array_equal(out["clamped"].cpu().numpy(), cl.astype(np.int64))
        for h in range(2):
            assert abs(out["entropy_bits"][h].item() - o.entropy_bits(ref[h])) <= ABS_ENTROPY
    # accumulate on top of an existing table
    out2 = ctx.gg_rate_hist(xd, steps, hist_id=[0, 1, 0], n_hist=2, qmin=qmin, qmax=qmax,
                            hist=out["hist"].clone(), accumulate=True)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out2["hist"].cpu().numpy(), 2 * ref.astype(np.int64))


def test_rate_hist_all_equal_input(ctx):
    """Worst case for the shared-memory atomics: every element lands in one bin."""
    x = torch.full((3 * TILE + 17,), 0.0123, dtype=torch.float32)
    out = ctx.gg_rate_hist([dev(x)], torch.tensor([1e-3], dtype=torch.float32, device="cuda:0"))
    torch.cuda.synchronize()
    ref, _ = o.quantise_hist(x.numpy(), 1e-3)
    np.testing.assert_array_equal(out["hist"][0].cpu().numpy(), ref.astype(np.int64))
    assert out["entropy_bits"][0].item() == 0.0


# ------------------------------------------------------------------------------------ gg_sample
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_sample_parity(ctx, dtype):
    betas = [0.1, 0.5, 0.8, 1.0, 1.3, 2.0, 3.0]
    lens = [5000, TILE + 3, 1, 40000, 2 * TILE, 777, 12345]
    alphas = [gg_synth.alpha_for_std(0.02, b) for b in betas]
    outs = [torch.empty(n, dtype=dtype, device="cuda:0") for n in lens]
    att = ctx.gg_sample(outs, betas, alphas, seed=0x1234567887654321, tensor_id0=40)
    torch.cuda.synchronize()
    total = mism = 0
    for s, (b, a, n) in enumerate(zip(betas, alphas, lens)):
        ref, ratt = o.sample(b, a, 0x1234567887654321, 40 + s, n, want_attempts=True)
        assert att[s].item() == int(ratt.max())
        got = outs[s].cpu()
        if dtype == torch.float32:
            refr = ref.astype(np.float32)
            gotn = got.numpy()
            diff = np.abs(refr.view(np.int32).astype(np.int64) - gotn.view(np.int32).astype(np.int64))
        else:
            refr = o.round_to_bf16_bits(ref).astype(np.int64)
            gotn = got.view(torch.int16).numpy().astype(np.int64) & 0xFFFF
            diff = np.abs(refr - gotn)
        assert diff.max() <= 1          # never more than one unit of the storage type
        np.testing.assert_array_equal(np.signbit(ref), np.signbit(got.float().numpy()))
        total += n
        mism += int((diff != 0).sum())
    # libm and device math differ in the last bits of the fp64 value (about 1e-15 relative): a value that sits that
    # close to a rounding boundary of the storage type can land on either side.  Per element that has probability
    # about 1e-7 in fp32 and 1e-12 in bf16, so at most one element in a million may differ, none in bf16.
    print(f"sampled values that differ from the oracle by one storage ulp: {mism} of {total} ({dtype})")
    assert mism <= (0 if dtype == torch.bfloat16 else -(-total // 1_000_000))


def test_sample_then_fit_recovers_parameters(ctx):
    """GG initialisation of scaled Qwen-shaped matrices, then the fit: the recovered shape and
    scale agree with the nominal ones statistically and with the oracle's fit of the same data."""
    shapes = gg_synth.scaled_shapes(gg_synth.qwen05b_shapes(), 4)[:9]
    beta = 1.3
    alpha = gg_synth.alpha_for_std(0.02, beta)
    outs = [torch.empty(r * c, dtype=torch.bfloat16, device="cuda:0") for _, r, c in shapes]
    ctx.gg_sample(outs, [beta] * len(outs), [alpha] * len(outs), seed=1, tensor_id0=0)
    fit = ctx.gg_fit(outs)
    torch.cuda.synchronize()
    for s, t in enumerate(outs):
        n = t.numel()
        bh, ah = fit["beta"][s].item(), fit["alpha"][s].item()
        assert abs(bh - beta) < 5 * 2.5 / math.sqrt(n) + 0.01
        assert abs(ah / alpha - 1) < 5 * 2.5 / math.sqrt(n) + 0.01
        b, a, *_ = o.fit(gg_synth.to_oracle(t))
        assert_rel(bh, b, REL_FIT, "beta")
        assert_rel(ah, a, REL_FIT, "alpha")


def test_fused_pass_is_deterministic(ctx):
    """Every output of the fused pass repeats bit for bit from call to call: partial sums are added in a fixed
    order and counts are integers.  Long bf16 and fp32 segments (the two-sweep kernels), many short bf16
    segments (the one-warp-per-segment kernel), and the single-step calls."""
    from paper_2506_00486_b200 import Segments
    rng = np.random.default_rng(53)
    sets = {
        "long_bf16": [gg_synth.gg_host(rng, 0.9, 0.02, n, torch.bfloat16) for n in (5 * TILE + 77, 3 * TILE, 40001)],
        "long_f32": [gg_synth.gg_host(rng, 0.6, 1e-3, n, torch.float32) for n in (4 * TILE + 5, 2 * TILE + 1)],
        "short_bf16": [gg_synth.gg_host(rng, 1.2, 0.3, int(rng.integers(1, 5000)), torch.bfloat16) for _ in range(100)],
    }
    for name, xs in sets.items():
        xd = [dev(x) for x in xs]
        gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
        n = len(xs)
        steps = torch.full((n,), 2.0 ** -9, dtype=torch.float32, device="cuda:0")
        hid = [s % 3 for s in range(n)]
        run = ctx.make_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps, hist_id=hid, n_hist=3)
        snaps = []
        for _ in range(3):
            for g in gd:
                g.fill_(float("nan"))
            out = run()
            torch.cuda.synchronize()
            snaps.append(([g.clone() for g in gd], {k: v.clone() for k, v in out.items() if isinstance(v, torch.Tensor)}))
        for grads, outs in snaps[1:]:
            for a, b in zip(grads, snaps[0][0]):
                assert torch.equal(a.view(torch.int32), b.view(torch.int32)), name
            for k, v in outs.items():
                assert torch.equal(v.view(torch.uint8), snaps[0][1][k].view(torch.uint8)), (name, k)
        # the single-step calls on the same data
        beta, alpha = snaps[0][1]["beta"], snaps[0][1]["alpha"]
        pens, hists = [], []
        for _ in range(2):
            pens.append(ctx.gg_penalty_grad(xd, beta, alpha, 1e-4, grad=gd).clone())
            h = ctx.gg_rate_hist(xd, steps, hist_id=hid, n_hist=3)
            hists.append((h["hist"].clone(), h["entropy_bits"].clone()))
        torch.cuda.synchronize()
        assert torch.equal(pens[0].view(torch.int64), pens[1].view(torch.int64)), name
        assert torch.equal(hists[0][0], hists[1][0]) and torch.equal(hists[0][1].view(torch.int64), hists[1][1].view(torch.int64)), name


# ------------------------------------------------------------------------------------- gg_fused
def check_fused(out, xs, grads, lam, hist_ids, n_hist, steps=None, step_scale=None, given=None,
                qmin=-32768, qmax=32767, mean=False):
    nb = qmax - qmin + 1
    ref_hist = np.zeros((n_hist, nb), dtype=np.uint64)
    ref_cl = np.zeros((n_hist, 2), dtype=np.uint64)
    used_steps = out["step"].cpu().numpy()
    for s, x in enumerate(xs):
        xo = gg_synth.to_oracle(x)
        b, a, s1, s2, n, fl = o.fit(xo)
        bg, ag = out["beta"][s].item(), out["alpha"][s].item()
        assert (out["flags"][s].item() & 15) == fl
        if fl & o.FLAG_DEGENERATE:
            assert bg == 0.0 and ag == 0.0
        else:
            assert_rel(bg, b, REL_FIT, f"beta[{s}]")
            assert_rel(ag, a, REL_FIT, f"alpha[{s}]")
        # parameters the gradient used: the GPU's own fit, or the given ones
        bu, au = (bg, ag) if given is None else given[s]
        lam_s = lam / max(n, 1) if mean else lam
        pen, g = o.penalty_grad(xo, bu, au, lam_s)
        if grads is not None:
            assert_grad_close(grads[s].float().cpu().numpy(), g)
        if pen > 0:
            assert_rel(out["penalty"][s].item(), pen, REL_PENALTY, f"penalty[{s}]")
        else:
            assert out["penalty"][s].item() == 0.0
        if step_scale is not None:
            assert used_steps[s] == np.float32(ag * step_scale)
        o.quantise_hist(xo, used_steps[s], qmin, qmax, hist=ref_hist[hist_ids[s]], clamped=ref_cl[hist_ids[s]])
    np.testing.assert_array_equal(out["hist"].cpu().numpy(), ref_hist.astype(np.int64))
    np.testing.assert_array_equal(out["clamped"].cpu().numpy(), ref_cl.astype(np.int64))
    for h in range(n_hist):
        assert abs(out["entropy_bits"][h].item() - o.entropy_bits(ref_hist[h])) <= ABS_ENTROPY


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_fused_fitted_parity(ctx, dtype):
    from paper_2506_00486_b200 import Segments
    xs = make_segments(dtype, seed=7) + [torch.zeros(50, dtype=dtype), torch.zeros(0, dtype=dtype)]
    xd = [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    n = len(xs)
    steps = torch.full((n,), 2.0 ** -10, dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
    torch.cuda.synchronize()
    check_fused(out, xs, gd, 1e-4, list(range(n)), n)


def test_fused_step_from_alpha_and_shared_histograms(ctx):
    from paper_2506_00486_b200 import Segments, GG_MEAN
    xs = make_segments(torch.float32, seed=8)
    xd = [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    hid = [0, 1, 1, 2, 0, 2, 1, 0]
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=3e-3, step_scale=1 / 16, hist_id=hid, n_hist=3,
                       reduction=GG_MEAN)
    torch.cuda.synchronize()
    check_fused(out, xs, gd, 3e-3, hid, 3, step_scale=1 / 16, mean=True)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_fused_given_parameters_single_sweep(ctx, dtype):
    """Lagged mode: the gradient uses caller parameters while the same sweep produces the new fit."""
    from paper_2506_00486_b200 import Segments, GG_PARAMS_GIVEN
    xs = make_segments(dtype, seed=10)
    xd = misaligned_views(xs) if dtype == torch.float32 else [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    n = len(xs)
    given = [(0.5 + 0.2 * s, 0.01 * (s + 1)) for s in range(n)]
    bi = torch.tensor([g[0] for g in given], dtype=torch.float64, device="cuda:0")
    ai = torch.tensor([g[1] for g in given], dtype=torch.float64, device="cuda:0")
    steps = torch.full((n,), 0.01, dtype=torch.float32, device="cuda:0")
    launches0 = ctx.launch_count
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps, param_mode=GG_PARAMS_GIVEN,
                       beta_in=bi, alpha_in=ai, qmin=-64, qmax=63)
    torch.cuda.synchronize()
    check_fused(out, xs, gd, 1e-4, list(range(n)), n, given=given, qmin=-64, qmax=63)
    assert (out["flags"].cpu().numpy() & 16).any()       # the narrow clamp was reported
    assert ctx.launch_count - launches0 == 3             # ONE sweep, then the fit, then the penalty sums and the entropy together


def test_fused_given_parameters_fp32_moments_of_special_values(ctx):
    """The one-read fp32 sweep takes its moments in fp32 runs of eight and falls back to fp64 where a square leaves
    the fp32 range or an entry is not finite: the sums, the counts of left-out entries and the extremes (through
    the clamp flag) must be those of the oracle."""
    from paper_2506_00486_b200 import Segments, GG_PARAMS_GIVEN
    rng = np.random.default_rng(12)
    big = gg_synth.gg_host(rng, 1.0, 1e25, 3 * TILE + 11, torch.float32)            # squares overflow fp32
    tiny = gg_synth.gg_host(rng, 1.2, 1e-28, 2 * TILE + 3, torch.float32)           # squares underflow
    mixed = gg_synth.gg_host(rng, 0.8, 0.05, 5 * TILE + 1, torch.float32)
    mixed[::997] = float("inf")
    mixed[5::1013] = float("nan")
    mixed[7::991] = -float("inf")
    mixed[3] = 3e38
    mixed[4] = 1e-44                                                                  # subnormal
    xs = [big, tiny, mixed]
    xd = [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    bi = torch.tensor([1.0, 1.2, 0.8], dtype=torch.float64, device="cuda:0")
    ai = torch.tensor([1e25, 1e-28, 0.05], dtype=torch.float64, device="cuda:0")
    steps = torch.tensor([1e23, 1e-30, 0.01], dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps, param_mode=GG_PARAMS_GIVEN, beta_in=bi, alpha_in=ai)
    torch.cuda.synchronize()
    for s, x in enumerate(xs):
        xo = gg_synth.to_oracle(x)
        b, a, s1, s2, n, fl = o.fit(xo)
        assert (out["flags"][s].item() & 15) == fl
        assert_rel(out["sum_abs"][s].item(), s1, 1e-6, "sum_abs")
        assert_rel(out["sum_sq"][s].item(), s2, 1e-6, "sum_sq")
        assert_rel(out["beta"][s].item(), b, REL_FIT, "beta")
        assert_rel(out["alpha"][s].item(), a, REL_FIT, "alpha")
        hist, cl = o.quantise_hist(xo, steps[s].item())
        np.testing.assert_array_equal(out["hist"][s].cpu().numpy(), hist.astype(np.int64))
        assert bool(out["flags"][s].item() & 16) == bool(cl.sum() > 0)


def test_config1_single_fp32_tensor(ctx):
    """1024x1024 fp32 from GG(beta=1, alpha=0.02): fit, penalty gradient (lambda 1e-4) and
    histogram at step 1e-3 with symbols clamped to int16, as separate calls and fused."""
    from paper_2506_00486_b200 import Segments
    w = gg_synth.workload_c1()
    x = w["tensors"][0]
    xo = gg_synth.to_oracle(x)
    xd = dev(x)
    fit = ctx.gg_fit([xd])
    g = torch.empty_like(xd)
    pen = ctx.gg_penalty_grad(Segments([xd]), fit["beta"], fit["alpha"], w["lam"], grad=Segments([g]))
    steps = torch.tensor(w["steps"], dtype=torch.float32, device="cuda:0")
    rh = ctx.gg_rate_hist([xd], steps)
    torch.cuda.synchronize()
    b, a, *_ = o.fit(xo)
    bg, ag = fit["beta"][0].item(), fit["alpha"][0].item()
    assert_rel(bg, b, REL_FIT, "beta")
    assert_rel(ag, a, REL_FIT, "alpha")
    assert abs(bg - 1.0) < 0.01 and abs(ag / 0.02 - 1) < 0.01      # the generating parameters
    rp, rg = o.penalty_grad(xo, bg, ag, w["lam"])
    assert_grad_close(g.cpu().numpy(), rg)
    assert_rel(pen[0].item(), rp, REL_PENALTY, "penalty")
    ref, cl = o.quantise_hist(xo, np.float32(1e-3))
    np.testing.assert_array_equal(rh["hist"][0].cpu().numpy(), ref.astype(np.int64))
    assert abs(rh["entropy_bits"][0].item() - o.entropy_bits(ref)) <= ABS_ENTROPY
    g2 = torch.empty_like(xd)
    out = ctx.gg_fused(Segments([xd]), grad=Segments([g2]), lam=w["lam"], step=steps)
    torch.cuda.synchronize()
    check_fused(out, [x], [g2], w["lam"], [0], 1)
    assert torch.equal(g, g2)


def test_config3_activation_rows_scaled(ctx):
    """Per-token segments of a bf16 activation tensor with outliers, one shared histogram
    (a [2, 96, 4096] slice of the [8, 2048, 4096] workload shape)."""
    from paper_2506_00486_b200 import Segments
    w = gg_synth.workload_c3(batch=2, seq=96)
    x = w["tensor"]
    xd = dev(x)
    gd = torch.empty(x.shape, dtype=torch.float32, device="cuda:0")
    steps = torch.full((w["n_seg"],), w["step"], dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused(Segments.rows(xd), grad=Segments.rows(gd), lam=w["lam"], step=steps,
                       hist_id=w["hist_id"], n_hist=1)
    torch.cuda.synchronize()
    check_fused(out, list(x), list(gd), w["lam"], w["hist_id"], 1)


# Which kernel a list of short segments takes: bf16, one warp per segment; fp32, one team of four warps per
# segment, which holds up to 4096 elements in registers and reads longer segments twice.
SHORT_KINDS = {"warp_bf16": (torch.bfloat16, 9000), "team_f32": (torch.float32, 4000), "team_f32_reread": (torch.float32, 12000)}


def short_segments(seed, n_seg=150, kind="warp_bf16"):
    """Many short segments of ragged lengths, a few of them empty, zero or tiny."""
    dtype, max_len = SHORT_KINDS[kind]
    rng = np.random.default_rng(seed)
    xs = []
    for s in range(n_seg):
        n = int(rng.integers(1, max_len))
        beta = float(rng.uniform(0.5, 2.5))
        xs.append(gg_synth.gg_host(rng, beta, 10.0 ** rng.uniform(-3, 0.5), n, dtype))
    xs[3] = torch.zeros(0, dtype=dtype)
    xs[4] = torch.zeros(77, dtype=dtype)
    xs[5] = torch.tensor([1.0, -1.0], dtype=dtype)
    xs[6] = torch.cat([xs[6], xs[6][:8]])
    xs[6][:8] = torch.tensor([0.0, -0.0, 1e-40, -1e-39, 3e38, -3e38, 1e-30, 1e20]).to(dtype)
    xs[8] = gg_synth.gg_host(rng, 3.4, 0.2, max_len, dtype)            # shape - 1 beyond the fp32 series: the fp64 path
    xs[9] = gg_synth.gg_host(rng, 1.0, 1e-30, max_len // 2, dtype)     # far from every other scale
    return xs


@pytest.mark.parametrize("kind", list(SHORT_KINDS))
def test_fused_many_short_segments_fit_only_with_nonfinite_entries(ctx, kind):
    from paper_2506_00486_b200 import Segments
    xs = short_segments(32, n_seg=80, kind=kind)
    xs[7] = torch.cat([xs[7], xs[7][:3]])
    xs[7][:3] = torch.tensor([float("inf"), float("nan"), float("-inf")]).to(xs[7].dtype)
    out = ctx.gg_fused(Segments([dev(x) for x in xs]), want_penalty=False, want_hist=False)
    torch.cuda.synchronize()
    for s, x in enumerate(xs):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(x))
        assert out["flags"][s].item() == fl and out["count"][s].item() == n
        if fl & o.FLAG_DEGENERATE:
            assert out["beta"][s].item() == 0.0 and out["alpha"][s].item() == 0.0
            continue
        assert_rel(out["sum_abs"][s].item(), s1, 1e-7, "sum_abs")
        assert_rel(out["sum_sq"][s].item(), s2, 1e-7, "sum_sq")
        assert_rel(out["beta"][s].item(), b, REL_FIT, f"beta[{s}]")
        assert_rel(out["alpha"][s].item(), a, REL_FIT, f"alpha[{s}]")


@pytest.mark.parametrize("kind", list(SHORT_KINDS))
@pytest.mark.parametrize("variant", ["shared_hist", "own_hist_step_from_alpha", "misaligned_bf16_grad_mean"])
def test_fused_many_short_segments(ctx, variant, kind):
    """The one-warp-per-segment and one-team-per-segment paths: shared histogram (CTA count table), per-segment
    histograms with steps taken from the fit (element-wise global counts), misaligned data with bf16 gradients."""
    from paper_2506_00486_b200 import Segments, GG_MEAN
    xs = short_segments(31, kind=kind)
    n = len(xs)
    if variant == "misaligned_bf16_grad_mean":
        xd = misaligned_views(xs, offsets=[(3 * s) % 8 for s in range(n)])
        gd = [torch.empty(x.numel(), dtype=torch.bfloat16, device="cuda:0") for x in xs]
        steps = torch.full((n,), 0.01, dtype=torch.float32, device="cuda:0")
        hid = [s % 3 for s in range(n)]
        out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=2e-3, step=steps, hist_id=hid, n_hist=3,
                           reduction=GG_MEAN, qmin=-300, qmax=200)
        torch.cuda.synchronize()
        # bf16 gradients: compare after rounding the oracle's values to bf16 (one bf16 ulp)
        check_fused(out, xs, None, 2e-3, hid, 3, qmin=-300, qmax=200, mean=True)
        for s, x in enumerate(xs):
            if x.numel() == 0:
                continue
            xo = gg_synth.to_oracle(x)
            _, g = o.penalty_grad(xo, out["beta"][s].item(), out["alpha"][s].item(), 2e-3 / x.numel())
            ref = o.round_to_bf16_bits(g).astype(np.int64)
            got = gd[s].cpu().view(torch.int16).numpy().astype(np.int64) & 0xFFFF
            fin = np.isfinite(g)
            assert np.abs((ref & 0x7FFF) - (got & 0x7FFF))[fin].max(initial=0) <= 1
        return
    xd = [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    if variant == "shared_hist":
        steps = torch.full((n,), 2.0 ** -7, dtype=torch.float32, device="cuda:0")
        out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps, hist_id=[0] * n, n_hist=1)
        torch.cuda.synchronize()
        check_fused(out, xs, gd, 1e-4, [0] * n, 1)
    else:
        out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step_scale=1 / 8, qmin=-2000, qmax=1999)
        torch.cuda.synchronize()
        check_fused(out, xs, gd, 1e-4, list(range(n)), n, step_scale=1 / 8, qmin=-2000, qmax=1999)


def test_config4_gradient_buckets_scaled(ctx):
    """fp32 buckets from GG(beta=0.5), per-bucket alpha log-uniform in [1e-6, 1e-3], step alpha/16
    (8 buckets of 250 000 instead of 25 000 000 elements)."""
    from paper_2506_00486_b200 import Segments
    w = gg_synth.workload_c4(bucket=250_000)
    xs = w["tensors"]
    xd = [dev(x) for x in xs]
    gd = [torch.empty_like(x) for x in xd]
    steps = torch.tensor(w["steps"], dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=w["lam"], step=steps)
    torch.cuda.synchronize()
    check_fused(out, xs, gd, w["lam"], w["hist_id"], w["n_hist"])
    for s in range(len(xs)):
        assert abs(out["beta"][s].item() - 0.5) < 0.02


def test_config5_weight_sweep_scaled(ctx):
    """The Llama-7B-shaped bf16 sweep with every matrix dimension divided by 16: 226 segments in one
    segmented launch, one histogram per tensor, step 2^-10."""
    from paper_2506_00486_b200 import Segments
    w = gg_synth.workload_c5_host(divisor=16)
    xs = w["tensors"]
    xd = [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    steps = torch.tensor(w["steps"], dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=w["lam"], step=steps)
    torch.cuda.synchronize()
    check_fused(out, xs, gd, w["lam"], w["hist_id"], w["n_hist"])


def test_fused_replays_from_a_cuda_graph(ctx):
    """After one eager call (plans and scratch exist) the fused pass only enqueues work on the caller's
    stream, so it can be captured in a CUDA graph; a replay on new data in the same buffers gives the
    results of a fresh call.  Long segments, many short segments and the channel-wise pass."""
    from paper_2506_00486_b200 import Segments
    rng = np.random.default_rng(23)
    long_x = [gg_synth.gg_host(rng, 0.9, 0.02, 2 * TILE + 77, torch.bfloat16), gg_synth.gg_host(rng, 1.4, 0.5, 5000, torch.bfloat16)]
    short_x = [gg_synth.gg_host(rng, 1.1, 0.1, 600, torch.bfloat16) for _ in range(70)]
    mat = torch.stack([gg_synth.gg_host(rng, 0.8, 0.3, 96, torch.bfloat16) for _ in range(300)])      # [300, 96]

    def fresh(xs):
        return [gg_synth.gg_host(rng, 1.2, 0.05, x.numel(), torch.bfloat16).view(x.shape) for x in xs]

    cases = []
    for xs in (long_x, short_x):
        xd = [dev(x) for x in xs]
        gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
        steps = torch.full((len(xs),), 2.0 ** -8, dtype=torch.float32, device="cuda:0")
        run = ctx.make_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
        cases.append((run, xd, gd, xs))
    md = dev(mat)
    mg = torch.empty(mat.shape, dtype=torch.float32, device="cuda:0")
    run_c = ctx.make_fused_channels(md, grad=mg, lam=1e-4, step=2.0 ** -8)

    for run, *_ in cases:
        run()
    run_c()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for run, *_ in cases:
            run()
        run_c()
    # new data in the captured buffers, then replay
    new_sets = []
    for run, xd, gd, xs in cases:
        xn = fresh(xs)
        for d, x in zip(xd, xn):
            d.copy_(x)
        for g in gd:
            g.fill_(float("nan"))
        new_sets.append(xn)
    mat_n = fresh([mat])[0]
    md.copy_(mat_n)
    graph.replay()
    torch.cuda.synchronize()
    for (run, xd, gd, xs), xn in zip(cases, new_sets):
        check_fused(run.outputs, xn, gd, 1e-4, list(range(len(xn))), len(xn))
    oc = {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in run_c.outputs.items()}
    for c in (0, 31, 64, 95):
        xo = gg_synth.to_oracle(mat_n[:, c].contiguous())
        b, a, *_ = o.fit(xo)
        assert_rel(oc["beta"][c].item(), b, REL_FIT, "beta")
        _, g = o.penalty_grad(xo, oc["beta"][c].item(), oc["alpha"][c].item(), 1e-4)
        assert_grad_close(mg[:, c].cpu().numpy(), g)
    assert oc["hist"].sum().item() == mat.numel()


def test_more_layouts_than_cached_plans(ctx):
    """The context keeps the plans of the 64 most recently used layouts; more layouts than that evict the
    oldest ones, which are rebuilt when they come back.  Results do not depend on any of it."""
    rng = np.random.default_rng(29)
    xs = [gg_synth.gg_host(rng, 1.0 + 0.01 * i, 0.05, 3000 + 17 * i, torch.bfloat16) for i in range(70)]
    xd = [dev(x) for x in xs]
    refs = [o.fit(gg_synth.to_oracle(x)) for x in xs]
    for rnd in range(2):                               # the second round finds the first layouts evicted
        for i, t in enumerate(xd):
            out = ctx.gg_fit([t])
            assert_rel(out["beta"][0].item(), refs[i][0], REL_FIT, f"beta[{i}] round {rnd}")
            assert_rel(out["alpha"][0].item(), refs[i][1], REL_FIT, f"alpha[{i}] round {rnd}")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_fused_random_layouts(ctx, dtype):
    """Random segment lists: any number of segments of any length from 0 to a few tiles at any element offset,
    grouped at random into shared histograms, sum or mean reduction.  Short and long bf16 lists take different
    kernels; every list must give the oracle's results."""
    from paper_2506_00486_b200 import Segments, GG_MEAN, GG_SUM
    rng = np.random.default_rng(47)
    for case in range(8):
        n_seg = int(rng.integers(1, 90)) if case % 2 else int(rng.integers(64, 130))
        cap = 9000 if case % 2 else 3 * TILE
        lens = [int(np.exp(rng.uniform(0, np.log(cap)))) - 1 for _ in range(n_seg)]
        xs = [gg_synth.gg_host(rng, float(rng.uniform(0.5, 2.2)), 10.0 ** rng.uniform(-3, 0), n, dtype) for n in lens]
        xd = misaligned_views(xs, offsets=[int(rng.integers(0, 8)) for _ in xs])
        gd = [torch.empty(n, dtype=torch.float32, device="cuda:0") for n in lens]
        n_hist = int(rng.integers(1, 4))
        hid = [int(rng.integers(0, n_hist)) for _ in xs]
        steps = torch.full((n_seg,), float(2.0 ** rng.integers(-9, -4)), dtype=torch.float32, device="cuda:0")
        mean = bool(case & 4)
        out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=2e-4, step=steps, hist_id=hid, n_hist=n_hist,
                           reduction=GG_MEAN if mean else GG_SUM, qmin=-3000, qmax=2500)
        torch.cuda.synchronize()
        check_fused(out, xs, gd, 2e-4, hid, n_hist, qmin=-3000, qmax=2500, mean=mean)


def test_one_layout_at_many_addresses_reuses_its_plans(ctx):
    """The same segment lengths at addresses that keep changing (buffers an allocator moves, the same shapes in
    another layer): after the layout's 16 plans exist, a call with new addresses points the least recently used
    of them at the new buffers instead of building a plan.  Every call must still read and write the buffers it
    was given: checked against the oracle at several of the 100 positions, the misaligned ones among them."""
    from paper_2506_00486_b200 import Context, Segments
    c = Context(0)
    rng = np.random.default_rng(31)
    lens = [40000, 7, 20000]
    stride, n_pos = 1000, 100
    pool = gg_synth.gg_host(rng, 0.9, 0.03, sum(lens) + stride * n_pos + 8, torch.bfloat16)
    pool_d = dev(pool)
    gpool = torch.full((pool.numel(),), 7.0, dtype=torch.float32, device="cuda:0")
    steps = torch.full((3,), 2.0 ** -9, dtype=torch.float32, device="cuda:0")

    def windows(k, buf):
        o0 = k * stride + (k % 3)                 # (every third position starts on a 16-byte boundary)
        return [buf[o0:o0 + lens[0]], buf[o0 + lens[0]:o0 + lens[0] + lens[1]],
                buf[o0 + lens[0] + lens[1]:o0 + sum(lens)]]

    other = [dev(gg_synth.gg_host(rng, 1.2, 0.1, 5000, torch.bfloat16))]
    for rnd in range(2):
        for k in range(n_pos):
            xd, gd = windows(k, pool_d), windows(k, gpool)
            out = c.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
            if k % 10 == 3:
                c.gg_fit(other)                   # (another layout in between changes nothing)
            if k in (0, 1, 17, 50, 64, 65, 99):
                torch.cuda.synchronize()
                check_fused(out, windows(k, pool), gd, 1e-4, [0, 1, 2], 3)
                gpool[k * stride:(k + 1) * stride + sum(lens) + 8] = 7.0
    torch.cuda.synchronize()
    built, repointed = c.plan_stats
    assert built == 16 + 1                        # the layout's plans and the other layout's one
    assert repointed == 2 * n_pos - 16            # every other call found its layout but not its addresses
    c.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("path", ["sweeps", "short"])
def test_fit_of_short_flat_topped_segments(ctx, dtype, path):
    """Few elements of similar magnitude: the moment ratio lies just below 3/4, where beta is 10 .. 20 and moves by
    up to 150 times the relative change of the ratio, so the sums have to be right to the last bits of fp64, not of
    the fp32 run sums that suffice elsewhere.  Thousands of such segments, so that the unlucky roundings occur; with
    one long segment in the list they take the sweeps and the fit kernel, without it the short-segment kernels."""
    rng = np.random.default_rng(61 + (path == "short"))
    n_seg = 3000
    lens = [int(rng.integers(6, 48)) for _ in range(n_seg)]
    if path == "sweeps":
        lens[7] = 20000
    xs = [gg_synth.gg_host(rng, float(rng.uniform(9.0, 19.0)), 10.0 ** rng.uniform(-3, 2), n, dtype) for n in lens]
    flat = torch.cat(xs).to("cuda:0")
    offs = np.concatenate([[0], np.cumsum(lens)])
    xd = [flat[offs[s]:offs[s + 1]] for s in range(n_seg)]
    fit = ctx.gg_fit(xd)
    out = ctx.gg_fused(xd, lam=1e-4, step=torch.full((n_seg,), 2.0 ** -6, dtype=torch.float32, device="cuda:0"),
                       hist_id=[0] * n_seg, n_hist=1)
    torch.cuda.synchronize()
    res = {k: (fit[k].cpu().numpy(), out[k].cpu().numpy()) for k in ("beta", "alpha", "flags")}
    large = 0
    for s, x in enumerate(xs):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(x))
        large += 8.0 < b < 20.0
        for which in (0, 1):
            assert (int(res["flags"][which][s]) & 15) == fl, (s, which)
            assert_rel(float(res["beta"][which][s]), b, REL_FIT, f"beta[{s}] of call {which}")
            assert_rel(float(res["alpha"][which][s]), a, REL_FIT, f"alpha[{s}] of call {which}")
    assert large >= 150                 # (the case is what it says; most of the others clamp at 20)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_fused_segments_that_start_off_the_block_boundaries(ctx, dtype):
    """The vector body of a run starts where the gradient (else the input) begins a 512-byte or 1 KB block, so the
    scalar head before it is up to a few hundred elements long, depending on both addresses.  Input and gradient at
    matching and at unrelated offsets from a 1 KB boundary, with and without a gradient; all against the oracle."""
    from paper_2506_00486_b200 import Segments
    rng = np.random.default_rng(83)
    n = 3 * 16384 + 77
    esz = 2 if dtype == torch.bfloat16 else 4
    for xo_bytes, go_bytes in ((16, 32), (128, 256), (0, 256), (16, 0), (48, 480), (1008, 992), (0, 0)):
        xs = [gg_synth.gg_host(rng, 0.9, 0.02, n, dtype), gg_synth.gg_host(rng, 1.7, 0.3, 300, dtype)]
        xd, gd = [], []
        for x in xs:
            xb = torch.zeros(x.numel() + 1024, dtype=dtype, device="cuda:0")
            gb = torch.full((x.numel() + 1024,), 9.0, dtype=torch.float32, device="cuda:0")
            assert xb.data_ptr() % 512 == 0 and gb.data_ptr() % 512 == 0
            xo = (-xb.data_ptr() % 1024 + xo_bytes) // esz
            go = (-gb.data_ptr() % 1024 + go_bytes) // 4
            xb[xo:xo + x.numel()].copy_(x)
            xd.append(xb[xo:xo + x.numel()])
            gd.append(gb[go:go + x.numel()])
        steps = torch.full((2,), 2.0 ** -9, dtype=torch.float32, device="cuda:0")
        out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
        torch.cuda.synchronize()
        check_fused(out, xs, gd, 1e-4, [0, 1], 2, steps=steps)
        hist_only = ctx.gg_rate_hist(xd, steps)
        fit_only = ctx.gg_fit(xd)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(hist_only["hist"].cpu().numpy(), out["hist"].cpu().numpy())
        assert torch.equal(fit_only["beta"], out["beta"]) and torch.equal(fit_only["sum_sq"], out["sum_sq"])
