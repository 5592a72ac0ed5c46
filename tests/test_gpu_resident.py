"""GPU parity of the one-launch form of the fitted pass of gg_fused (bf16 input): moments, fit and gradient +
histogram of every group of tensors in one cooperative launch whose CTAs hand tensors over through L2.

The form is switched on through gg_test_hook (it is off by default), on small ragged layouts and on tensors of
tens of megabytes; every output is compared with the fp64 oracle element by element.  Its bounded waits are made
to run out by asking the fitting CTA to wait for an arrival that never comes: the segments are then flagged and
the context stays usable."""
import numpy as np
import pytest
import torch

import gg_synth
from oracle import gg_oracle as o
from test_gpu_parity import TILE, check_fused, dev, make_segments, misaligned_views

pytestmark = pytest.mark.gpu


@pytest.fixture()
def forced():
    """A context that takes the one-launch pass whenever it can run."""
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import Context
    from paper_2506_00486_b200.binding import HOOK_RESIDENT_MODE
    c = Context(0)
    c.gg_test_hook(HOOK_RESIDENT_MODE, 1)
    yield c
    c.close()


def launches_of(ctx, run):
    before = ctx.launch_count
    out = run()
    torch.cuda.synchronize()
    return out, ctx.launch_count - before


@pytest.mark.parametrize("misalign", [False, True])
def test_forced_on_ragged_segments(forced, misalign):
    from paper_2506_00486_b200 import Segments
    xs = make_segments(torch.bfloat16, seed=31) + [torch.zeros(50, dtype=torch.bfloat16), torch.zeros(0, dtype=torch.bfloat16)]
    xd = misaligned_views(xs, offsets=(1, 3, 5, 2, 7, 0, 4, 6, 3, 0)) if misalign else [dev(x) for x in xs]
    gd = [torch.full((x.numel(),), float("nan"), dtype=torch.float32, device="cuda:0") for x in xs]
    n = len(xs)
    steps = torch.full((n,), 2.0 ** -10, dtype=torch.float32, device="cuda:0")
    out, launches = launches_of(forced, forced.make_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps))
    assert launches == 2              # the pass; the penalty sums and the entropy together
    check_fused(out, xs, gd, 1e-4, list(range(n)), n)


def test_forced_step_from_alpha_shared_histograms_mean_and_bf16_gradient(forced):
    from paper_2506_00486_b200 import GG_MEAN, Segments
    rng = np.random.default_rng(33)
    lens = [5 * TILE + 17, 3, TILE, 2 * TILE - 1, 40000, 0, 7 * TILE + 5] * 6        # 42 segments: three groups
    xs = [gg_synth.gg_host(rng, float(rng.uniform(0.5, 2.0)), 10.0 ** rng.uniform(-3, 0), n, torch.bfloat16) for n in lens]
    xd = [dev(x) for x in xs]
    gd = [torch.empty(n, dtype=torch.bfloat16, device="cuda:0") for n in lens]
    hid = [int(v) for v in rng.integers(0, 4, len(xs))]
    out, launches = launches_of(forced, forced.make_fused(Segments(xd), grad=Segments(gd), lam=3e-3, step_scale=1 / 16, hist_id=hid,
                                                          n_hist=4, reduction=GG_MEAN))
    assert launches == 2
    # (the gradient is compared in bf16: rounding the oracle's value the same way)
    steps_used = out["step"].cpu().numpy()
    ref_hist = np.zeros((4, 65536), dtype=np.uint64)
    for s, x in enumerate(xs):
        xo = gg_synth.to_oracle(x)
        b, a, _, _, n, fl = o.fit(xo)
        assert (out["flags"][s].item() & 15) == fl
        if fl & o.FLAG_DEGENERATE:
            continue
        bg, ag = out["beta"][s].item(), out["alpha"][s].item()
        assert abs(bg - b) <= 1e-5 * b and abs(ag - a) <= 1e-5 * a
        assert steps_used[s] == np.float32(ag / 16)
        pen, g = o.penalty_grad(xo, bg, ag, 3e-3 / n)
        assert abs(out["penalty"][s].item() - pen) <= 1e-6 * pen
        ref = torch.from_numpy(g.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().astype(np.int64)
        got = gd[s].cpu().view(torch.int16).numpy().astype(np.int64)
        assert np.abs(ref - got).max() <= 1          # one bf16 step: the fp32 value may sit a few ulp from a bf16 tie
        o.quantise_hist(xo, steps_used[s], hist=ref_hist[hid[s]])
    np.testing.assert_array_equal(out["hist"].cpu().numpy(), ref_hist.astype(np.int64))


@pytest.mark.parametrize("what", ["histogram_only", "gradient_only", "accumulate"])
def test_forced_partial_passes(forced, what):
    from paper_2506_00486_b200 import Segments
    xs = make_segments(torch.bfloat16, seed=35)
    xd = [dev(x) for x in xs]
    n = len(xs)
    steps = torch.full((n,), 0.01, dtype=torch.float32, device="cuda:0")
    if what == "histogram_only":
        out = forced.gg_fused(Segments(xd), want_penalty=False, step=steps, qmin=-100, qmax=90)
        torch.cuda.synchronize()
        ref = np.zeros((n, 191), dtype=np.uint64)
        cl = np.zeros((n, 2), dtype=np.uint64)
        for s, x in enumerate(xs):
            o.quantise_hist(gg_synth.to_oracle(x), 0.01, -100, 90, hist=ref[s], clamped=cl[s])
        np.testing.assert_array_equal(out["hist"].cpu().numpy(), ref.astype(np.int64))
        np.testing.assert_array_equal(out["clamped"].cpu().numpy(), cl.astype(np.int64))
        return
    base = [torch.full((x.numel(),), 0.25, dtype=torch.float32, device="cuda:0") for x in xs]
    out = forced.gg_fused(Segments(xd), grad=Segments(base), lam=-2e-4, want_hist=False, accumulate_grad=(what == "accumulate"))
    torch.cuda.synchronize()
    from parity_util import assert_grad_close
    for s, x in enumerate(xs):
        xo = gg_synth.to_oracle(x)
        pen, g = o.penalty_grad(xo, out["beta"][s].item(), out["alpha"][s].item(), -2e-4)
        if what == "accumulate":
            got = base[s].cpu().numpy().astype(np.float64) - 0.25
            assert np.abs(got - g).max() <= 2.0 ** -24 * 0.25 + 4 * np.spacing(np.abs(g).max().astype(np.float32))
        else:
            assert_grad_close(base[s].cpu().numpy(), g)
        assert abs(out["penalty"][s].item() - pen) <= 1e-6 * abs(pen)


def test_forced_random_layouts(forced):
    from paper_2506_00486_b200 import GG_MEAN, GG_SUM, Segments
    rng = np.random.default_rng(37)
    for case in range(6):
        n_seg = int(rng.integers(1, 70))
        lens = [int(np.exp(rng.uniform(0, np.log(6 * TILE)))) - 1 for _ in range(n_seg)]
        xs = [gg_synth.gg_host(rng, float(rng.uniform(0.5, 2.2)), 10.0 ** rng.uniform(-3, 0), n, torch.bfloat16) for n in lens]
        xd = misaligned_views(xs, offsets=[int(rng.integers(0, 8)) for _ in xs])
        gd = [torch.empty(n, dtype=torch.float32, device="cuda:0") for n in lens]
        n_hist = int(rng.integers(1, 4))
        hid = [int(rng.integers(0, n_hist)) for _ in xs]
        steps = torch.full((n_seg,), float(2.0 ** rng.integers(-9, -4)), dtype=torch.float32, device="cuda:0")
        mean = bool(case & 1)
        out = forced.gg_fused(Segments(xd), grad=Segments(gd), lam=2e-4, step=steps, hist_id=hid, n_hist=n_hist,
                              reduction=GG_MEAN if mean else GG_SUM, qmin=-3000, qmax=2500)
        torch.cuda.synchronize()
        check_fused(out, xs, gd, 2e-4, hid, n_hist, qmin=-3000, qmax=2500, mean=mean)


def test_large_tensors_and_repeats_bit_for_bit(forced):
    """Three tensors of 18 to 34 MB, one group each (several tiles per streaming CTA); two calls give the same bits
    everywhere."""
    from paper_2506_00486_b200 import Segments
    ctx = forced
    gen = torch.Generator(device="cuda:0")
    gen.manual_seed(39)
    lens = [12_000_003, 17_000_000, 9_000_001]
    xd = [gg_synth.gg_device(gen, b, gg_synth.alpha_for_std(0.02, b), n, torch.bfloat16, torch.device("cuda:0"))
          for b, n in zip((0.7, 1.2, 1.6), lens)]
    gd = [torch.empty(n, dtype=torch.float32, device="cuda:0") for n in lens]
    steps = torch.full((3,), 2.0 ** -10, dtype=torch.float32, device="cuda:0")
    run = ctx.make_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
    out, launches = launches_of(ctx, run)
    assert launches == 2
    first = {k: v.clone() for k, v in out.items() if isinstance(v, torch.Tensor)}
    g_first = [g.clone() for g in gd]
    for g in gd:
        g.fill_(float("nan"))
    out = run()
    torch.cuda.synchronize()
    for k, v in first.items():
        assert torch.equal(v.view(torch.uint8), out[k].view(torch.uint8)), k
    for a, b in zip(g_first, gd):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    check_fused(out, [x.cpu() for x in xd], gd, 1e-4, [0, 1, 2], 3)


def test_a_wait_that_cannot_end_is_reported_and_the_context_stays_usable(forced):
    from paper_2506_00486_b200 import Segments
    from paper_2506_00486_b200.binding import FLAG_TIMEOUT, HOOK_EXTRA_ARRIVALS, HOOK_WAIT_CAP
    xs = make_segments(torch.bfloat16, seed=41)
    xd = [dev(x) for x in xs]
    gd = [torch.empty(x.numel(), dtype=torch.float32, device="cuda:0") for x in xs]
    n = len(xs)
    steps = torch.full((n,), 2.0 ** -10, dtype=torch.float32, device="cuda:0")
    run = forced.make_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
    forced.gg_test_hook(HOOK_EXTRA_ARRIVALS, 1)      # the fitting CTA waits for one arrival more than there are CTAs
    forced.gg_test_hook(HOOK_WAIT_CAP, 1 << 12)
    out = run()
    torch.cuda.synchronize()                          # the launch ends by itself: no error, no hang
    assert (out["flags"].cpu().numpy() & FLAG_TIMEOUT).all()
    forced.gg_test_hook(HOOK_EXTRA_ARRIVALS, 0)
    forced.gg_test_hook(HOOK_WAIT_CAP, 1 << 18)
    out = run()
    torch.cuda.synchronize()
    assert not (out["flags"].cpu().numpy() & FLAG_TIMEOUT).any()
    check_fused(out, xs, gd, 1e-4, list(range(n)), n)


def test_forced_pass_replays_from_a_cuda_graph(forced):
    from paper_2506_00486_b200 import Segments
    rng = np.random.default_rng(43)
    lens = [3 * TILE + 77, 5000, 9 * TILE]
    xs = [gg_synth.gg_host(rng, 0.9, 0.02, n, torch.bfloat16) for n in lens]
    xd = [dev(x) for x in xs]
    gd = [torch.empty(n, dtype=torch.float32, device="cuda:0") for n in lens]
    steps = torch.full((3,), 2.0 ** -8, dtype=torch.float32, device="cuda:0")
    run = forced.make_fused(Segments(xd), grad=Segments(gd), lam=1e-4, step=steps)
    run()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run()
    xn = [gg_synth.gg_host(rng, 1.3, 0.05, n, torch.bfloat16) for n in lens]
    for d, x in zip(xd, xn):
        d.copy_(x)
    for g in gd:
        g.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    check_fused(run.outputs, xn, gd, 1e-4, [0, 1, 2], 3)
