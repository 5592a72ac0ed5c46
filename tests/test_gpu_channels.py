"""GPU parity of the channel-wise pass: every column of a row-major matrix is one segment.  The oracle
has no notion of strides: each column is gathered on the host and goes through the same oracle calls
as a contiguous segment."""
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


def channel_matrix(rows, cols, seed, wide_scales=True, dtype=torch.bfloat16):
    """[rows, cols]: column c is GG(beta_c, alpha_c) with its own shape and scale."""
    rng = np.random.default_rng(seed)
    x = torch.empty((rows, cols), dtype=dtype)
    for c in range(cols):
        beta = float(rng.uniform(0.4, 2.5))
        alpha = 10.0 ** rng.uniform(-4, 1) if wide_scales else 0.05 * (1 + c % 7)
        x[:, c] = gg_synth.gg_host(rng, beta, alpha, rows, dtype)
    return x


def check_channels(out, x, grad, lam, step=None, qmin=-32768, qmax=32767, mean=False, grad_before=None,
                   hist_before=None, cols=None):
    rows, ncol = x.shape
    nb = qmax - qmin + 1
    ref_hist = np.zeros(nb, dtype=np.uint64) if hist_before is None else hist_before.astype(np.uint64).copy()
    ref_cl = np.zeros(2, dtype=np.uint64)
    for c in (range(ncol) if cols is None else cols):
        xo = gg_synth.to_oracle(x[:, c].contiguous())
        b, a, s1, s2, n, fl = o.fit(xo)
        bg, ag = out["beta"][c].item(), out["alpha"][c].item()
        assert (out["flags"][c].item() & 15) == fl, f"flags[{c}]"
        assert out["count"][c].item() == n
        if fl & o.FLAG_DEGENERATE:
            assert bg == 0.0 and ag == 0.0
        else:
            assert_rel(out["sum_abs"][c].item(), s1, 1e-7, f"sum_abs[{c}]")
            assert_rel(out["sum_sq"][c].item(), s2, 1e-7, f"sum_sq[{c}]")
            assert_rel(bg, b, REL_FIT, f"beta[{c}]")
            assert_rel(ag, a, REL_FIT, f"alpha[{c}]")
        lam_c = lam / max(n, 1) if mean else lam
        pen, g = o.penalty_grad(xo, bg, ag, lam_c)
        if grad is not None:
            got = grad[:, c]
            if grad.dtype == torch.bfloat16:
                if grad_before is not None:
                    with np.errstate(invalid="ignore", over="ignore"):
                        g = (g.astype(np.float32) + grad_before[:, c].float().numpy()).astype(np.float64)
                ref = o.round_to_bf16_bits(g).astype(np.int64)
                gb = got.view(torch.int16).numpy().astype(np.int64) & 0xFFFF
                fin = np.isfinite(g)
                assert np.abs((ref & 0x7FFF) - (gb & 0x7FFF))[fin].max(initial=0) <= 1, f"grad[:, {c}]"
            else:
                assert grad_before is None
                nan = np.isnan(g)                      # a nan entry gives a nan gradient: any nan will do
                assert np.isnan(got.numpy()[nan]).all()
                assert_grad_close(got.numpy()[~nan], g[~nan])
        if out["penalty"] is not None:
            if not np.isfinite(pen):                   # inf or nan entries: the sum is not a number either
                assert not np.isfinite(out["penalty"][c].item())
            elif pen != 0:
                assert_rel(out["penalty"][c].item(), pen, REL_PENALTY, f"penalty[{c}]")
            else:
                assert out["penalty"][c].item() == 0.0
        if step is not None and cols is None:
            cl = np.zeros(2, dtype=np.uint64)
            o.quantise_hist(xo, np.float32(step), qmin, qmax, hist=ref_hist, clamped=cl)
            ref_cl += cl
            assert bool(out["flags"][c].item() & 16) == bool(cl.sum() > 0), f"clamp flag[{c}]"
    if step is not None and cols is None:
        np.testing.assert_array_equal(out["hist"].cpu().numpy(), ref_hist.astype(np.int64))
        np.testing.assert_array_equal(out["clamped"].cpu().numpy(), ref_cl.astype(np.int64))
        assert abs(out["entropy_bits"][0].item() - o.entropy_bits(ref_hist)) <= ABS_ENTROPY


def cpu(out):
    return {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in out.items()}


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_channels_ragged_padded_with_special_columns(ctx, dtype):
    """Full strips and a ragged one, rows that fill no whole block, padded rows (ld > cols),
    scales 1e-4 .. 10 inside one strip, and columns of zeros, specials, tiny and huge values."""
    rows, cols, ld = 1500, 200, 208
    x = channel_matrix(rows, cols, seed=41, dtype=dtype)
    x[:, 5] = 0
    x[:, 6] = torch.where(torch.arange(rows) % 2 == 0, x[:, 6], torch.zeros(()).to(dtype))   # half exact zeros
    x[:9, 7] = torch.tensor([0.0, -0.0, 1e-40, -1e-39, 3e38, -3e38, 1e-30, 1e20, -1e-20]).to(dtype)
    x[:3, 8] = torch.tensor([float("inf"), float("nan"), float("-inf")]).to(dtype)
    x[:, 70] = (x[:, 70].float() * 1e-25).to(dtype)       # far below the strip's exponent window
    x[:, 130] = (x[:, 130].float() * 1e20).to(dtype)      # pushes the window up for its strip
    buf = torch.full((rows, ld), 7.0, dtype=dtype, device="cuda:0")
    buf[:, :cols].copy_(x)
    gbuf = torch.full((rows, ld), -1.0, dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused_channels(buf[:, :cols], grad=gbuf[:, :cols], lam=1e-4, step=2.0 ** -7)
    torch.cuda.synchronize()
    assert torch.all(gbuf[:, cols:] == -1.0)                      # the padding is not written
    check_channels(cpu(out), x, gbuf[:, :cols].cpu(), 1e-4, step=2.0 ** -7)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_channels_odd_width_bf16_grad_mean_accumulate_and_clamp(ctx, dtype):
    """Odd column count and odd leading dimension (scalar loads and stores), bf16 gradient added to
    what is there, mean reduction, negative lambda, a clamp narrower than the count window, counts
    added to an existing histogram."""
    from paper_2506_00486_b200 import GG_MEAN
    rows, cols, ld = 777, 131, 133
    x = channel_matrix(rows, cols, seed=42, wide_scales=False, dtype=dtype)
    buf = torch.zeros((rows, ld), dtype=dtype, device="cuda:0")
    buf[:, :cols].copy_(x)
    g0 = (torch.randn((rows, cols), generator=torch.Generator().manual_seed(1)) * 1e-4).to(torch.bfloat16)
    gbuf = torch.zeros((rows, ld), dtype=torch.bfloat16, device="cuda:0")
    gbuf[:, :cols].copy_(g0)
    qmin, qmax = -300, 200
    h0 = torch.arange(qmax - qmin + 1, dtype=torch.int64)
    hist = h0.to("cuda:0")
    out = ctx.gg_fused_channels(buf[:, :cols], grad=gbuf[:, :cols], lam=-2e-3, reduction=GG_MEAN, accumulate_grad=True,
                                step=0.01, qmin=qmin, qmax=qmax, accumulate_hist=True, hist=hist)
    torch.cuda.synchronize()
    check_channels(cpu(out), x, gbuf[:, :cols].cpu(), -2e-3, step=0.01, qmin=qmin, qmax=qmax, mean=True,
                   grad_before=g0, hist_before=h0.numpy())


def test_channels_fit_only_and_empty_shapes(ctx):
    x = channel_matrix(300, 70, seed=43)
    out = ctx.gg_fused_channels(x.to("cuda:0"), want_penalty=False)
    torch.cuda.synchronize()
    check_channels(cpu(out), x, None, 0.0)
    # no rows: every column degenerate; no columns: nothing to do
    out = ctx.gg_fused_channels(torch.empty((0, 5), dtype=torch.bfloat16, device="cuda:0"), step=0.5)
    torch.cuda.synchronize()
    assert torch.all(out["beta"] == 0) and torch.all(out["flags"] == 1) and torch.all(out["penalty"] == 0)
    assert out["hist"].sum().item() == 0 and out["entropy_bits"][0].item() == 0.0
    out = ctx.gg_fused_channels(torch.empty((4, 0), dtype=torch.bfloat16, device="cuda:0"), step=0.5)
    torch.cuda.synchronize()
    assert out["beta"].numel() == 0
    # one row: |x| is the whole sample, the ratio is 1 and beta clamps high
    one = torch.tensor([[0.5, -2.0, 0.0]], dtype=torch.bfloat16)
    g = torch.empty((1, 3), dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused_channels(one.to("cuda:0"), grad=g, step=0.25)
    torch.cuda.synchronize()
    check_channels(cpu(out), one, g.cpu(), 1e-4, step=0.25)


def test_channels_rejects_what_it_does_not_take(ctx):
    from paper_2506_00486_b200 import GGError
    with pytest.raises(GGError):
        ctx.gg_fused_channels(torch.zeros((4, 4), dtype=torch.bfloat16, device="cuda:0"), step=0.0)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_channels_activation_shaped_matrix_sampled_columns(ctx, dtype):
    """[8192 tokens, 4096 channels] bf16 with channel-dependent scale and 0.1 % outliers: several row
    slices per strip.  Sampled columns against the oracle element by element; for the whole matrix the
    histogram against torch's own floor and bincount, and column sums against torch reductions."""
    rows, cols = 8192, 4096
    gen = torch.Generator(device="cuda:0").manual_seed(44)
    a = gg_synth.alpha_for_std(1.0, 0.8)
    x = gg_synth.gg_device(gen, 0.8, a, rows * cols, dtype, torch.device("cuda:0")).view(rows, cols)
    scale = torch.exp2(torch.arange(cols, device="cuda:0") % 9 - 4.0).to(dtype)
    x = (x * scale).contiguous()
    gg_synth.add_outliers_device(gen, x, 1e-3, 20.0)
    g = torch.empty((rows, cols), dtype=torch.float32, device="cuda:0")
    step = 0.01
    out = ctx.gg_fused_channels(x, grad=g, lam=1e-4, step=step)
    torch.cuda.synchronize()
    xf = x.float()
    inv = torch.tensor(1.0 / step, dtype=torch.float64).float().item()
    q = torch.floor(xf * inv).clamp_(-32768, 32767).to(torch.int64) + 32768
    ref = torch.bincount(q.view(-1), minlength=65536)
    assert torch.equal(out["hist"], ref)
    assert out["hist"].sum().item() == rows * cols
    torch.testing.assert_close(out["sum_abs"], xf.double().abs().sum(0), rtol=1e-7, atol=0)
    torch.testing.assert_close(out["sum_sq"], (xf.double() ** 2).sum(0), rtol=1e-7, atol=0)
    sample = [0, 1, 63, 64, 2047, 2048, 4031, 4095] + list(np.random.default_rng(5).integers(0, cols, 8))
    oc = cpu(out)
    check_channels(oc, x.cpu(), g.cpu(), 1e-4, cols=sample)


def test_channels_matrix_with_more_than_2_to_31_elements(ctx):
    """[2^19, 4100] bf16 (2.15e9 elements: element offsets need 64 bits; the last strip is ragged): sampled columns
    against the oracle, column sums and the histogram total for the whole matrix."""
    rows, cols = 1 << 19, 4100
    gen = torch.Generator(device="cuda:0").manual_seed(45)
    x = gg_synth.gg_device(gen, 1.1, gg_synth.alpha_for_std(0.5, 1.1), rows * cols, torch.bfloat16, torch.device("cuda:0")).view(rows, cols)
    g = torch.empty((rows, cols), dtype=torch.float32, device="cuda:0")
    out = ctx.gg_fused_channels(x, grad=g, lam=1e-4, step=2.0 ** -6)
    torch.cuda.synchronize()
    assert out["hist"].sum().item() == rows * cols
    assert torch.all(out["count"] == rows)
    s1 = torch.zeros(cols, dtype=torch.float64, device="cuda:0")
    for r0 in range(0, rows, 1 << 16):                       # (in slabs: a float64 copy of the matrix would not fit)
        s1 += x[r0:r0 + (1 << 16)].double().abs().sum(0)
    torch.testing.assert_close(out["sum_abs"], s1, rtol=1e-7, atol=0)
    sample = [0, 63, 2050, 4095, 4096, 4099]
    oc = cpu(out)
    xs = torch.stack([x[:, c] for c in sample], dim=1).cpu()
    gs = torch.stack([g[:, c] for c in sample], dim=1).cpu()
    sub = {k: (v[sample] if isinstance(v, torch.Tensor) and v.numel() == cols else v) for k, v in oc.items()}
    check_channels(sub, xs, gs, 1e-4, cols=list(range(len(sample))))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_channels_random_shapes_and_alignments(ctx, dtype):
    """Random small matrices: any row and column count, padded or not, first element at any element offset from a
    256-byte boundary (aligned and unaligned rows for the vector paths), fp32 and bf16 gradients."""
    rng = np.random.default_rng(46)
    for case in range(10):
        rows, cols = int(rng.integers(1, 700)), int(rng.integers(1, 150))
        ld = cols + int(rng.integers(0, 4))
        off = int(rng.integers(0, 8))
        gdt = torch.bfloat16 if case % 3 == 2 else torch.float32
        x = channel_matrix(rows, cols, seed=100 + case, wide_scales=(case % 2 == 0), dtype=dtype)
        flat = torch.zeros(rows * ld + 16, dtype=dtype, device="cuda:0")
        xd = flat[off:off + rows * ld].view(rows, ld)[:, :cols]
        xd.copy_(x)
        gflat = torch.zeros(rows * ld + 16, dtype=gdt, device="cuda:0")
        gd = gflat[off:off + rows * ld].view(rows, ld)[:, :cols]
        step = float(2.0 ** rng.integers(-9, -3))
        out = ctx.gg_fused_channels(xd, grad=gd, lam=3e-4, step=step, qmin=-5000, qmax=4000)
        torch.cuda.synchronize()
        check_channels(cpu(out), x, gd.cpu(), 3e-4, step=step, qmin=-5000, qmax=4000)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_channels_short_flat_topped_columns(ctx, dtype):
    """Columns of a few dozen rows with flat-topped data: beta between 10 and 20, where it moves by up to 150 times the
    relative change of the moment ratio.  The fit then needs the column sums to the last bits of fp64 (the fit kernel
    takes them again from the elements); checked on 3000 columns, so that the unlucky roundings occur."""
    rng = np.random.default_rng(71)
    rows, cols = 40, 3000
    x = torch.empty((rows, cols), dtype=dtype)
    for c in range(cols):
        x[:, c] = gg_synth.gg_host(rng, float(rng.uniform(9.0, 19.0)), 10.0 ** rng.uniform(-3, 2), rows, dtype)
    out = cpu(ctx.gg_fused_channels(x.to("cuda:0"), lam=1e-4, step=2.0 ** -6))
    torch.cuda.synchronize()
    large = 0
    for c in range(cols):
        b, a, s1, s2, n, fl = o.fit(gg_synth.to_oracle(x[:, c].contiguous()))
        large += 8.0 < b < 20.0
        assert (out["flags"][c].item() & 15) == fl, f"flags[{c}]"
        assert_rel(out["beta"][c].item(), b, REL_FIT, f"beta[{c}]")
        assert_rel(out["alpha"][c].item(), a, REL_FIT, f"alpha[{c}]")
    assert large >= 150
