"""Parity at the full sizes of the five workloads, in the launch configuration the benchmark times.
What the oracle can do in seconds is compared element by element on sampled tensors / rows; the
rest is checked through properties that hold at any size (histogram totals, counts, the generating
parameters)."""
import numpy as np
import pytest
import torch

import gg_synth
from oracle import gg_oracle as o
from parity_util import ABS_ENTROPY, REL_FIT, REL_PENALTY, assert_grad_close, assert_rel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import Context
    c = Context(0)
    yield c
    c.close()


def check_segment(x_host, g_dev, out, s, lam, step, hist_row=None):
    xo = gg_synth.to_oracle(x_host)
    b, a, s1, s2, n, fl = o.fit(xo)
    bg, ag = out["beta"][s].item(), out["alpha"][s].item()
    assert (out["flags"][s].item() & 15) == fl and out["count"][s].item() == n
    assert_rel(bg, b, REL_FIT, f"beta[{s}]")
    assert_rel(ag, a, REL_FIT, f"alpha[{s}]")
    pen, g = o.penalty_grad(xo, bg, ag, lam)
    assert_grad_close(g_dev.float().cpu().numpy().reshape(-1), g)
    assert_rel(out["penalty"][s].item(), pen, REL_PENALTY, f"penalty[{s}]")
    if hist_row is not None:
        ref, _ = o.quantise_hist(xo, step)
        np.testing.assert_array_equal(hist_row.cpu().numpy(), ref.astype(np.int64))
        return ref
    return None


def test_config5_llama7b_sweep_full_size(ctx):
    """The whole 6.74e9-element sweep as bench.py runs it; three tensors (an attention matrix, an MLP
    matrix, the output head) against the oracle in full, every tensor through its invariants."""
    from paper_2506_00486_b200 import Segments
    dev = torch.device("cuda", 0)
    w = gg_synth.workload_c5_device(dev, torch.bfloat16, seed=4)
    flat, offs, lens = w["flat"], w["offsets"], w["lens"]
    n_seg = len(lens)
    gflat = torch.empty(flat.numel(), dtype=torch.float32, device=dev)
    steps = torch.full((n_seg,), 2.0 ** -10, dtype=torch.float32, device=dev)
    run = ctx.make_fused(Segments.slices(flat, offs, lens), grad=Segments.slices(gflat, offs, lens), lam=1e-4, step=steps)
    out = run()
    out = run()             # a second call over the cached plan must give the same tables
    torch.cuda.synchronize()
    totals = out["hist"].sum(dim=1).cpu().numpy()
    np.testing.assert_array_equal(totals, np.asarray(lens))
    np.testing.assert_array_equal(out["count"].cpu().numpy(), np.asarray(lens))
    beta = out["beta"].cpu().numpy()
    assert np.abs(beta - np.asarray(w["beta_true"])).max() < 0.01          # the generating shapes, statistically
    assert (out["flags"].cpu().numpy() == 0).all()
    for s in (1, 5, n_seg - 1):
        sl = slice(offs[s], offs[s] + lens[s])
        ref = check_segment(flat[sl].cpu(), gflat[sl], out, s, 1e-4, 2.0 ** -10, out["hist"][s])
        assert abs(out["entropy_bits"][s].item() - o.entropy_bits(ref)) <= ABS_ENTROPY
    del flat, gflat, run, out
    torch.cuda.empty_cache()


def test_config3_activations_full_size(ctx):
    """bf16 [8, 2048, 4096] with outliers, per-token segments, one shared histogram: the histogram in
    full, 48 sampled rows element by element."""
    from paper_2506_00486_b200 import Segments
    w = gg_synth.workload_c3()
    x = w["tensor"]
    xd = x.to("cuda:0")
    gd = torch.empty(x.shape, dtype=torch.float32, device="cuda:0")
    steps = torch.full((w["n_seg"],), w["step"], dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused(Segments.rows(xd), grad=Segments.rows(gd), lam=w["lam"], step=steps,
                       hist_id=w["hist_id"], n_hist=1)
    torch.cuda.synchronize()
    ref, cl = o.quantise_hist(gg_synth.to_oracle(x), w["step"])
    np.testing.assert_array_equal(out["hist"][0].cpu().numpy(), ref.astype(np.int64))
    np.testing.assert_array_equal(out["clamped"][0].cpu().numpy(), cl.astype(np.int64))
    assert abs(out["entropy_bits"][0].item() - o.entropy_bits(ref)) <= ABS_ENTROPY
    rows = np.random.default_rng(0).choice(w["n_seg"], 48, replace=False)
    for s in rows:
        check_segment(x[s], gd[s], out, int(s), w["lam"], w["step"])
    b = out["beta"].cpu().numpy()
    assert np.isfinite(b).all() and (b > 0.3).all() and (b < 1.5).all()     # outliers pull the fitted shape below 0.8


def test_config4_gradient_buckets_full_size(ctx):
    """8 fp32 buckets of 25 M elements, step = alpha / 16 from each bucket's own fit: two buckets against
    the oracle in full, all through their invariants."""
    from paper_2506_00486_b200 import Segments
    w = gg_synth.workload_c4()
    xs = w["tensors"]
    xd = [x.to("cuda:0") for x in xs]
    gd = [torch.empty_like(x) for x in xd]
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=w["lam"], step_scale=1 / 16)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out["hist"].sum(dim=1).cpu().numpy(), [x.numel() for x in xs])
    for s in range(len(xs)):
        assert abs(out["beta"][s].item() - 0.5) < 0.01
        assert out["step"][s].item() == np.float32(out["alpha"][s].item() / 16)
    for s in (0, 5):
        ref = check_segment(xs[s], gd[s], out, s, w["lam"], out["step"][s].item(), out["hist"][s])
        H = o.entropy_bits(ref)
        assert abs(out["entropy_bits"][s].item() - H) <= ABS_ENTROPY
        # bits per element near the fine-step formula h(alpha, beta) - log2(step) (loose: beta = 0.5 is sharply peaked)
        assert abs(H - (o.diff_entropy_nats(out["alpha"][s].item(), out["beta"][s].item()) / np.log(2)
                        - np.log2(out["step"][s].item()))) < 0.5


def test_config2_qwen_initialisation_full_size(ctx):
    """gg_sample of the 169 Qwen-0.5B-shaped bf16 matrices (beta 1.3, std 0.02, seed 1), then gg_fit:
    three matrices against the oracle's sampler in full, the recovered parameters of all of them."""
    shapes = gg_synth.qwen05b_shapes()
    beta, alpha = 1.3, gg_synth.alpha_for_std(0.02, 1.3)
    outs = [torch.empty(r * c, dtype=torch.bfloat16, device="cuda:0") for _, r, c in shapes]
    att = ctx.gg_sample(outs, [beta] * len(outs), [alpha] * len(outs), seed=1, tensor_id0=0)
    fit = ctx.gg_fit(outs)
    torch.cuda.synchronize()
    assert att.max().item() <= 64
    n = np.array([t.numel() for t in outs], dtype=np.float64)
    assert (np.abs(fit["beta"].cpu().numpy() - beta) < 5 * 2.5 / np.sqrt(n) + 0.01).all()
    assert (np.abs(fit["alpha"].cpu().numpy() / alpha - 1) < 5 * 2.5 / np.sqrt(n) + 0.01).all()
    for s in (2, 5, 168):          # a key projection, a gate projection, the last down projection
        ref = o.sample(beta, alpha, 1, s, outs[s].numel())
        refb = o.round_to_bf16_bits(ref).astype(np.int64)
        got = outs[s].cpu().view(torch.int16).numpy().astype(np.int64) & 0xFFFF
        diff = np.abs(refb - got)
        assert diff.max() <= 1 and int((diff != 0).sum()) == 0          # (bf16 storage: see test_sample_parity)
        b, a, *_ = o.fit(gg_synth.to_oracle(outs[s].cpu()))
        assert_rel(fit["beta"][s].item(), b, REL_FIT, "beta")
        assert_rel(fit["alpha"][s].item(), a, REL_FIT, "alpha")


def test_sampled_bf16_values_equal_the_oracle_over_millions_of_elements(ctx):
    """bf16 output takes attempt 0 in fp32 with error bounds and hands every doubtful element to the fp64 path, so
    its values must be the oracle's bit for bit: four shapes (gamma shape above and below 1), 3 M elements each."""
    n = 3_000_000
    betas = [0.3, 0.8, 1.0, 2.5]
    alphas = [gg_synth.alpha_for_std(0.02, b) for b in betas]
    outs = [torch.empty(n, dtype=torch.bfloat16, device="cuda:0") for _ in betas]
    att = ctx.gg_sample(outs, betas, alphas, seed=0xABCDEF0123, tensor_id0=7)
    torch.cuda.synchronize()
    for s, (b, a) in enumerate(zip(betas, alphas)):
        ref, ratt = o.sample(b, a, 0xABCDEF0123, 7 + s, n, want_attempts=True)
        assert att[s].item() == int(ratt.max())
        refb = o.round_to_bf16_bits(ref).astype(np.int64)
        got = outs[s].cpu().view(torch.int16).numpy().astype(np.int64) & 0xFFFF
        assert np.array_equal(refb, got), (b, int((refb != got).sum()))


def test_one_segment_longer_than_2_to_31_elements(ctx):
    """A single bf16 segment of 2^31 + 12345 elements (64-bit offsets in both sweeps): 2048 copies of a 2^20-element
    block and a ragged rest, so that the exact results follow from the oracle's results on the block and the
    rest: sums and counts add up, the gradient repeats."""
    from paper_2506_00486_b200 import Segments
    blk, n = 1 << 20, (1 << 31) + 12345
    k_full, rest = n // blk, n % blk
    rng = np.random.default_rng(31)
    base = gg_synth.gg_host(rng, 0.9, 0.02, blk, torch.bfloat16)
    base[::1009] = 0
    x = base.to("cuda:0").repeat(k_full + 1)[:n].contiguous()
    g = torch.empty(n, dtype=torch.float32, device="cuda:0")
    step, lam = 2.0 ** -10, 1e-4
    out = ctx.gg_fused(Segments([x]), grad=Segments([g]), lam=lam, step=torch.full((1,), step, dtype=torch.float32, device="cuda:0"))
    torch.cuda.synchronize()
    xb, xr = gg_synth.to_oracle(base), gg_synth.to_oracle(base[:rest])
    s1b, s2b, _, _ = o.moments(xb)
    s1r, s2r, _, _ = o.moments(xr)
    s1, s2 = k_full * s1b + s1r, k_full * s2b + s2r
    assert out["count"][0].item() == n and out["flags"][0].item() == 0
    # (every copy of the block rounds its fp32 runs of eight the same way, so these errors do not average out
    # over the copies: the bound is that of one block, 1e-7)
    assert_rel(out["sum_abs"][0].item(), s1, 1e-7, "sum_abs")
    assert_rel(out["sum_sq"][0].item(), s2, 1e-7, "sum_sq")
    b, a, _ = o.fit_from_moments(s1, s2, n)
    bg, ag = out["beta"][0].item(), out["alpha"][0].item()
    assert_rel(bg, b, REL_FIT, "beta")
    assert_rel(ag, a, REL_FIT, "alpha")
    # histogram and penalty: 2048 blocks and the rest
    hb, _ = o.quantise_hist(xb, np.float32(step))
    hr, _ = o.quantise_hist(xr, np.float32(step))
    np.testing.assert_array_equal(out["hist"][0].cpu().numpy(), (k_full * hb.astype(np.int64) + hr.astype(np.int64)))
    pb, gb = o.penalty_grad(xb, bg, ag, lam)
    pr, _ = o.penalty_grad(xr, bg, ag, lam)
    assert_rel(out["penalty"][0].item(), k_full * pb + pr, REL_PENALTY, "penalty")
    # the gradient of the first block, of the block that straddles element 2^31, and of the ragged rest
    for k in (0, 1023, 2047):
        assert_grad_close(g[k * blk:(k + 1) * blk].cpu().numpy(), gb)
    assert_grad_close(g[k_full * blk:].cpu().numpy(), gb[:rest])
    # every other block repeats the first one bit for bit
    g2 = g[:k_full * blk].view(k_full, blk)
    assert bool((g2 == g2[0]).all())


def test_sample_elements_past_index_2_to_32(ctx):
    """gg_sample of one bf16 segment of 2^32 + 4096 elements: the element index is a 64-bit counter (its high
    word enters the Philox counter).  The oracle regenerates windows of elements around 2^32 and at the end."""
    n = (1 << 32) + 4096
    x = torch.empty(n, dtype=torch.bfloat16, device="cuda:0")
    beta, alpha, seed = 1.3, gg_synth.alpha_for_std(0.02, 1.3), 77
    att = ctx.gg_sample([x], [beta], [alpha], seed=seed, tensor_id0=5)
    torch.cuda.synchronize()
    for i0 in (0, (1 << 32) - 2048, (1 << 32), n - 1000):
        m = min(3000, n - i0)
        ref = o.sample(beta, alpha, seed, 5, m, index0=i0)
        got = x[i0:i0 + m].cpu()
        refb = o.round_to_bf16_bits(ref).astype(np.int64)
        gotb = got.view(torch.int16).numpy().astype(np.int64) & 0xFFFF
        assert np.array_equal(refb >> 15, gotb >> 15)                       # signs
        assert np.array_equal(refb, gotb)                                   # bf16 storage: the same patterns
    assert 1 <= att[0].item() <= 64
    del x
