"""GPU parity of the code-length entry points and the GCT step against the CPU oracle."""
import numpy as np
import pytest
import torch

import gg_synth
from oracle import gg_oracle as o
from parity_util import assert_grad_close, ulp_distance

pytestmark = pytest.mark.gpu

TILE = 16384


@pytest.fixture(scope="module")
def ctx():
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import Context
    c = Context(0)
    yield c
    c.close()


def segs(dtype, seed):
    rng = np.random.default_rng(seed)
    spec = [(0.5, 3e-4, 2 * TILE + 77), (1.0, 0.02, TILE), (1.5, 0.5, 5), (0.8, 1.0, 40001)]
    xs = [gg_synth.gg_host(rng, b, a, n, dtype) for b, a, n in spec]
    xs[0][:4] = torch.tensor([0.0, -0.0, float("nan"), 1e-30]).to(dtype)
    return xs


@pytest.mark.parametrize("k", [0, 3])
def test_eg_rate_and_code_stats_from_histograms(ctx, k):
    xs = segs(torch.bfloat16, 41)
    xd = [x.to("cuda:0") for x in xs]
    steps = torch.tensor([2e-5, 1e-3, 0.05, 0.01], dtype=torch.float32, device="cuda:0")
    for qmin, qmax in ((-32768, 32767), (-40, 25)):
        rh = ctx.gg_rate_hist(xd, steps, qmin=qmin, qmax=qmax)
        eg = ctx.gg_eg_rate(rh["hist"], k=k, qmin=qmin, qmax=qmax)
        stats = ctx.gg_code_stats(rh["hist"], k=k, qmin=qmin, qmax=qmax)
        torch.cuda.synchronize()
        for s, x in enumerate(xs):
            xo = gg_synth.to_oracle(x)
            ref_hist, _ = o.quantise_hist(xo, steps[s].item(), qmin, qmax)
            ref = o.eg_rate(xo, steps[s].item(), k, qmin, qmax)
            assert abs(eg[s].item() - ref) <= 1e-12 * max(1.0, ref)
            assert abs(stats["eg_bits"][s] - ref) <= 1e-12 * max(1.0, ref)
            assert abs(stats["hm_bits"][s] - o.huffman_bits(ref_hist)) <= 1e-12
            assert stats["fl_bits"][s] == o.fixed_length_bits(ref_hist)
            H = o.entropy_bits(ref_hist)
            if np.count_nonzero(ref_hist) > 1:
                assert H - 1e-9 <= stats["hm_bits"][s] < H + 1


def test_compression_ratio_helper():
    from paper_2506_00486_b200 import gg_compression_ratio
    assert gg_compression_ratio(1.59, 12.0) == pytest.approx(0.8675, abs=5e-5)        # a row of the paper's Table 4
    assert gg_compression_ratio(14.99, 13.0) == pytest.approx(-0.1531, abs=5e-5)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_eg_rate_grad_parity(ctx, dtype):
    from paper_2506_00486_b200 import Segments
    xs = segs(dtype, 42)
    xd = [x.to("cuda:0") for x in xs]
    gd = [torch.full((x.numel(),), 0.5, dtype=torch.float32, device="cuda:0") for x in xs]
    steps = torch.tensor([2e-5, 1e-3, 0.05, 0.01], dtype=torch.float32, device="cuda:0")
    ctx.gg_eg_rate_grad(Segments(xd), steps, 0.3, Segments(gd), k=1, qmin=-1000, qmax=900)
    torch.cuda.synchronize()
    for s, x in enumerate(xs):
        ref = o.eg_rate_grad(gg_synth.to_oracle(x), steps[s].item(), 0.3, 1, -1000, 900)
        assert_grad_close(gd[s].cpu().numpy(), ref, max_ulp=2)
    # accumulate on top
    ctx.gg_eg_rate_grad(Segments(xd), steps, 0.3, Segments(gd), k=1, qmin=-1000, qmax=900, accumulate=True)
    torch.cuda.synchronize()
    ref = o.eg_rate_grad(gg_synth.to_oracle(xs[1]), steps[1].item(), 0.3, 1, -1000, 900)
    np.testing.assert_allclose(gd[1].cpu().numpy(), 2 * ref.astype(np.float32), rtol=3e-7)


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16])
def test_gct_step_parity_over_three_steps(ctx, g_dtype):
    """Algorithm 2 for three steps: t = 1 is plain gradient descent, later steps use the stored gradient."""
    from paper_2506_00486_b200 import Segments
    rng = np.random.default_rng(43)
    lens = [TILE + 333, 7, 3 * TILE]
    w = [rng.standard_normal(n).astype(np.float32) for n in lens]
    wd = [torch.from_numpy(a.copy()).to("cuda:0") for a in w]
    hd = [torch.zeros(n, dtype=torch.float32, device="cuda:0") for n in lens]
    w64 = [a.astype(np.float64) for a in w]
    h64 = [np.zeros(n) for n in lens]
    step_vals = [2.0 ** -14, 1e-4, 3e-5]
    steps = torch.tensor(step_vals, dtype=torch.float32, device="cuda:0")
    eta, lam, eps = 1e-2, 0.05, 1e-8
    for t in (1, 2, 3):
        g = [gg_synth.gg_host(rng, 0.7, 1e-3, n, g_dtype) for n in lens]
        ctx.gg_gct_step(Segments([x.to("cuda:0") for x in g]), Segments(hd), Segments(wd), steps, eta, lam, eps, t)
        torch.cuda.synchronize()
        for s in range(len(lens)):
            # the oracle continues from the fp32 values the GPU stored, as the next GPU step does
            gh, wn = o.gct_step(gg_synth.to_oracle(g[s]), h64[s], w64[s], step_vals[s], eta, lam, eps, t)
            got_h, got_w = hd[s].cpu().numpy(), wd[s].cpu().numpy()
            assert ulp_distance(got_h, gh).max() <= 1
            assert ulp_distance(got_w, wn).max() <= 1
            h64[s], w64[s] = got_h.astype(np.float64), got_w.astype(np.float64)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("variant", ["coarse", "fine", "clamped"])
def test_fused_pass_with_the_code_length_rate(ctx, dtype, variant):
    """GG_RATE_EG: moments and fit, the gradient of lambda * R (Eq. 6-7), the histogram, its entropy and its mean code
    length from ONE read of x.  Every output against the oracle's separate functions.  coarse: 192 (bf16) or 128
    (fp32) steps reach 6.5 standard deviations, so the kernels count by symbol in lane-private rows; fine: they do
    not; clamped: the symbols are cut to a narrow range inside the count window."""
    from paper_2506_00486_b200 import GG_RATE_EG, Segments
    rng = np.random.default_rng({"coarse": 51, "fine": 52, "clamped": 53}[variant])
    spec = [(0.7, 0.02, 3 * TILE + 77), (1.0, 0.02, 5), (2.0, 0.02, 0), (1.3, 0.02, 2 * TILE), (0.9, 0.02, 40000)]
    xs = [gg_synth.gg_host(rng, b, gg_synth_alpha(0.02, b), n, dtype) for b, a, n in spec]
    xs[0][:6] = torch.tensor([0.0, -0.0, float("nan"), 1e-30, float("inf"), -7.5]).to(dtype)     # specials and a far outlier
    xs[3][100] = float("-inf")
    # the first segment starts two elements into its buffer (not on a 16-byte boundary)
    buf = torch.zeros(xs[0].numel() + 8, dtype=dtype, device="cuda:0")
    buf[2:2 + xs[0].numel()].copy_(xs[0])
    xd = [buf[2:2 + xs[0].numel()]] + [x.to("cuda:0") for x in xs[1:]]
    gd = [torch.full((x.numel() + 4,), 3.0, dtype=torch.float32, device="cuda:0")[2:2 + x.numel()] for x in xs]
    step_val = {"coarse": 0.02 / 16, "fine": 0.02 / 3000, "clamped": 0.02 / 16}[variant]
    qmin, qmax = (-50, 40) if variant == "clamped" else (-32768, 32767)
    k, lam = (2, -0.3) if variant == "fine" else (0, 0.3)
    steps = torch.full((len(xs),), step_val, dtype=torch.float32, device="cuda:0")
    hid = [0, 1, 1, 2, 0]
    out = ctx.gg_fused(Segments(xd), grad=Segments(gd), lam=lam, step=steps, hist_id=hid, n_hist=3, qmin=qmin, qmax=qmax,
                       param_mode=GG_RATE_EG, eg_k=k)
    torch.cuda.synchronize()
    nb = qmax - qmin + 1
    ref_hist = np.zeros((3, nb), dtype=np.uint64)
    ref_cl = np.zeros((3, 2), dtype=np.uint64)
    step32 = steps[0].item()
    for s, x in enumerate(xs):
        xo = gg_synth.to_oracle(x)
        b, a, s1, s2, n, fl = o.fit(xo)
        assert (out["flags"][s].item() & 15) == fl
        if not (fl & o.FLAG_DEGENERATE):
            assert abs(out["beta"][s].item() / b - 1) <= 1e-5 and abs(out["alpha"][s].item() / a - 1) <= 1e-5
        if x.numel():
            ref = o.eg_rate_grad(xo, step32, lam, k, qmin, qmax)
            assert_grad_close(gd[s].cpu().numpy(), ref, max_ulp=2)
        o.quantise_hist(xo, step32, qmin, qmax, hist=ref_hist[hid[s]], clamped=ref_cl[hid[s]])
    np.testing.assert_array_equal(out["hist"].cpu().numpy(), ref_hist.astype(np.int64))
    np.testing.assert_array_equal(out["clamped"].cpu().numpy(), ref_cl.astype(np.int64))
    for h in range(3):
        assert abs(out["entropy_bits"][h].item() - o.entropy_bits(ref_hist[h])) <= 1e-9
        bits = o.eg_rate_hist(ref_hist[h], k, qmin)
        assert abs(out["eg_bits"][h].item() - bits) <= 1e-12 * max(1.0, bits)
    for s in range(len(xs)):
        want = lam * out["eg_bits"][hid[s]].item()
        assert out["penalty"][s].item() == pytest.approx(want, rel=1e-15, abs=0.0)


def gg_synth_alpha(sigma, beta):
    from paper_2506_00486_b200 import gg_alpha_from_std
    return gg_alpha_from_std(sigma, beta)


def test_code_length_rate_mode_needs_a_histogram_with_a_given_step(ctx):
    from paper_2506_00486_b200 import GG_RATE_EG, GGError
    x = [torch.ones(4096, dtype=torch.bfloat16, device="cuda:0")]
    before = ctx.launch_count
    with pytest.raises(GGError) as e:
        ctx.gg_fused(x, lam=0.1, want_hist=False, param_mode=GG_RATE_EG)
    assert e.value.status == 1
    with pytest.raises(GGError) as e:
        ctx.gg_fused(x, lam=0.1, step_scale=0.1, param_mode=GG_RATE_EG)
    assert e.value.status == 1
    with pytest.raises(GGError) as e:
        ctx.gg_fused(x, lam=0.1, step=torch.ones(1, device="cuda:0"), param_mode=GG_RATE_EG, eg_k=31)
    assert e.value.status == 1
    assert ctx.launch_count == before
