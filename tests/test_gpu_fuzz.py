"""Randomised parity of gg_fused over everything that decides which kernels run: element type, segment lengths from
empty to 70 tiles (short-segment kernels, the two sweeps, the optional one-launch and cluster forms), alignment,
gradient type, shared histograms, sum or mean, fitted or given parameters, steps given or taken from the fit, the sign
of lambda, the clamp range, the GG penalty or the code-length rate of Eq. 6-7.  Every case is compared with the fp64
oracle: fit, flags, gradient element by element, penalty, histogram, clamp counters, entropy (and code length); and no
output may be written outside its buffer."""
import numpy as np
import pytest
import torch

import gg_synth
from oracle import gg_oracle as o
from parity_util import ulp_distance

pytestmark = pytest.mark.gpu

TILE = 16384


@pytest.mark.parametrize("seed0", [11, 12])
def test_fused_random_cases_over_every_option(seed0):
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import GG_MEAN, GG_PARAMS_GIVEN, GG_RATE_EG, GG_SUM, Context, Segments
    ctx = Context(0, guard=True)
    n_cases = 40
    failures = []
    for case in range(n_cases):
        rng = np.random.default_rng(seed0 * 100000 + case)
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        kind = rng.choice(["short", "medium", "long", "mixed"])
        if kind == "short":
            n_seg, cap = int(rng.integers(64, 200)), int(rng.choice([600, 5000, 16000]))
        elif kind == "medium":
            n_seg, cap = int(rng.integers(2, 40)), int(rng.choice([3 * TILE, 20 * TILE]))
        elif kind == "long":
            n_seg, cap = int(rng.integers(1, 5)), 70 * TILE
        else:
            n_seg, cap = int(rng.integers(1, 100)), 10 * TILE
        lens = [max(0, int(np.exp(rng.uniform(0, np.log(cap)))) - 1) for _ in range(n_seg)]
        xs = [gg_synth.gg_host(rng, float(rng.uniform(0.3, 2.6)), 10.0 ** rng.uniform(-4, 1), n, dtype) for n in lens]
        if rng.random() < 0.3 and lens[0] > 10:
            xs[0][:4] = torch.tensor([0.0, -0.0, 3e38, 1e-39]).to(dtype)
        misalign = rng.random() < 0.4
        offs = [int(rng.integers(0, 8)) if misalign else 0 for _ in xs]
        xd = []
        for t, off in zip(xs, offs):
            buf = torch.zeros(t.numel() + 16, dtype=t.dtype, device="cuda:0"); buf[off:off + t.numel()].copy_(t); xd.append(buf[off:off + t.numel()])
        gdt = torch.float32 if rng.random() < 0.7 else torch.bfloat16
        gd = [torch.full((n,), 0.5, dtype=gdt, device="cuda:0") for n in lens]
        n_hist = int(rng.integers(1, 4)); hid = [int(rng.integers(0, n_hist)) for _ in xs]
        mean = rng.random() < 0.3
        given = rng.random() < 0.3
        step_alpha = (not given) and rng.random() < 0.3
        lam = float(rng.choice([1e-4, -3e-3, 2.0]))
        resident = int(rng.random() < 0.3 and dtype == torch.bfloat16); cluster = int(rng.choice([0, 0, 1, 2]))
        ctx.gg_test_hook(0, resident)      # the one-launch form on or off
        ctx.gg_test_hook(3, cluster)       # the cluster form: never / when the layout suits / whenever it can run
        qmin, qmax = (-32768, 32767) if rng.random() < 0.5 else (-300, 250)
        kw = dict(grad=Segments(gd), lam=lam, hist_id=hid, n_hist=n_hist, reduction=GG_MEAN if mean else GG_SUM, qmin=qmin, qmax=qmax)
        step_val = float(2.0 ** rng.integers(-10, -3))
        if step_alpha: kw["step_scale"] = 1 / 8
        else: kw["step"] = torch.full((n_seg,), step_val, dtype=torch.float32, device="cuda:0")
        giv = None
        if given:
            giv = [(float(rng.uniform(0.4, 2.4)), 10.0 ** rng.uniform(-3, 0)) for _ in xs]
            kw.update(param_mode=GG_PARAMS_GIVEN, beta_in=torch.tensor([g[0] for g in giv], dtype=torch.float64, device="cuda:0"),
                      alpha_in=torch.tensor([g[1] for g in giv], dtype=torch.float64, device="cuda:0"))
        # (drawn from a generator of its own, so that the cases of the other options stay what they were)
        rng_eg = np.random.default_rng(seed0 * 100000 + 50000 + case)
        eg = (not given) and (not step_alpha) and rng_eg.random() < 0.3
        eg_k = int(rng_eg.choice([0, 1, 4]))
        if eg: kw.update(param_mode=GG_RATE_EG, eg_k=eg_k)
        desc = f"case {case} eg={eg} dtype={dtype} kind={kind} n_seg={n_seg} cap={cap} mis={misalign} gdt={gdt} given={given} step_alpha={step_alpha} lam={lam} res={resident} clu={cluster} q=({qmin},{qmax}) mean={mean}"
        try:
            out = ctx.gg_fused(Segments(xd), **kw)
            torch.cuda.synchronize(); ctx.check_guards()
            nb = qmax - qmin + 1
            ref_hist = np.zeros((n_hist, nb), dtype=np.uint64); ref_cl = np.zeros((n_hist, 2), dtype=np.uint64)
            steps_used = out["step"].cpu().numpy()
            for s, x in enumerate(xs):
                xo = gg_synth.to_oracle(x)
                b, a, s1, s2, n, fl = o.fit(xo)
                assert (out["flags"][s].item() & 15) == fl, ("flags", s)
                bg, ag = out["beta"][s].item(), out["alpha"][s].item()
                if fl & 1: assert bg == 0 and ag == 0
                else: assert abs(bg - b) <= 1e-5 * b and abs(ag - a) <= 1e-5 * a, ("fit", s, bg, b)
                bu, au = (bg, ag) if giv is None else giv[s]
                lam_s = lam / max(n, 1) if mean else lam
                pen, g = o.penalty_grad(xo, bu, au, lam_s)
                if eg:
                    g = o.eg_rate_grad(xo, steps_used[s], lam, eg_k, qmin, qmax) if n else g
                    pen = float("nan")       # (checked against the histogram's code length below)
                got = gd[s].float().cpu().numpy().astype(np.float64) - 0.5 if False else None
                # gradient written (not accumulated): compare
                gg = gd[s].cpu()
                if gdt == torch.float32:
                    fin = np.isfinite(g.astype(np.float32))
                    d = ulp_distance(gg.numpy()[fin], g[fin]); assert d.size == 0 or d.max() <= (2 if eg else 4), ("grad", s, int(d.max()))
                else:
                    ref = o.round_to_bf16_bits(g).astype(np.int64); gb = gg.view(torch.int16).numpy().astype(np.int64) & 0xFFFF
                    fin = np.isfinite(g) & (np.abs(g) < 3e38)
                    assert np.abs((ref & 0x7FFF) - (gb & 0x7FFF))[fin].max(initial=0) <= 1, ("grad16", s)
                if np.isfinite(pen) and abs(pen) > 0: assert abs(out["penalty"][s].item() - pen) <= 1e-6 * abs(pen), ("pen", s, out["penalty"][s].item(), pen)
                if step_alpha: assert steps_used[s] == np.float32(ag / 8), ("step", s)
                if steps_used[s] > 0 and np.isfinite(steps_used[s]):
                    o.quantise_hist(xo, steps_used[s], qmin, qmax, hist=ref_hist[hid[s]], clamped=ref_cl[hid[s]])
            if not (step_alpha and any((out["flags"][s].item() & 1) for s in range(n_seg))):
                assert np.array_equal(out["hist"].cpu().numpy(), ref_hist.astype(np.int64)), "hist"
                assert np.array_equal(out["clamped"].cpu().numpy(), ref_cl.astype(np.int64)), "clamped"
                for h in range(n_hist): assert abs(out["entropy_bits"][h].item() - o.entropy_bits(ref_hist[h])) <= 1e-9, "entropy"
                if eg:
                    for h in range(n_hist):
                        bits = o.eg_rate_hist(ref_hist[h], eg_k, qmin)
                        assert abs(out["eg_bits"][h].item() - bits) <= 1e-12 * max(1.0, bits), "eg_bits"
                    for s in range(n_seg): assert out["penalty"][s].item() == lam * out["eg_bits"][hid[s]].item(), ("eg penalty", s)
        except AssertionError as e:
            failures.append((desc, str(e)))
    ctx.close()
    assert not failures, failures


@pytest.mark.parametrize("seed0", [1, 2])
def test_single_step_calls_random_cases(seed0):
    """The same for the single-step calls: gg_fit, gg_penalty_grad (random given parameters, written or accumulated,
    fp32 or bf16 gradients), gg_rate_hist (power-of-two and arbitrary steps, shared histograms, two clamp ranges) and
    gg_sample (attempt counts exact, values equal after rounding to the storage type) on random segment lists."""
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import GG_MEAN, GG_SUM, Context, Segments
    ctx = Context(0, guard=True)
    failures = []
    for case in range(25):
        rng = np.random.default_rng(900000 + seed0 * 1000 + case)
        dtype = torch.bfloat16 if rng.random() < 0.5 else torch.float32
        kind = rng.choice(["short", "medium", "long", "mixed"])
        if kind == "short": n_seg, cap = int(rng.integers(64, 200)), int(rng.choice([600, 5000, 16000]))
        elif kind == "medium": n_seg, cap = int(rng.integers(2, 40)), int(rng.choice([3 * TILE, 20 * TILE]))
        elif kind == "long": n_seg, cap = int(rng.integers(1, 5)), 70 * TILE
        else: n_seg, cap = int(rng.integers(1, 100)), 10 * TILE
        lens = [max(0, int(np.exp(rng.uniform(0, np.log(cap)))) - 1) for _ in range(n_seg)]
        xs = [gg_synth.gg_host(rng, float(rng.uniform(0.3, 12.0) if rng.random() < 0.3 else rng.uniform(0.3, 2.6)), 10.0 ** rng.uniform(-4, 1), n, dtype) for n in lens]
        if rng.random() < 0.3 and lens[0] > 10:
            xs[0][:6] = torch.tensor([0.0, -0.0, 3e38, 1e-39, float("inf"), float("nan")]).to(dtype)
        mis = rng.random() < 0.4
        xd = []
        for t in xs:
            off = int(rng.integers(0, 8)) if mis else 0
            buf = torch.zeros(t.numel() + 16, dtype=t.dtype, device="cuda:0"); buf[off:off + t.numel()].copy_(t); xd.append(buf[off:off + t.numel()])
        desc = f"case {case} {dtype} {kind} n_seg={n_seg} cap={cap} mis={mis}"
        try:
            # ---- fit
            fit = ctx.gg_fit(xd); torch.cuda.synchronize(); ctx.check_guards()
            refs = [o.fit(gg_synth.to_oracle(x)) for x in xs]
            for s, (b, a, s1, s2, n, fl) in enumerate(refs):
                assert (fit["flags"][s].item() & 15) == fl, ("fit flags", s)
                if not fl & 1:
                    assert abs(fit["beta"][s].item() - b) <= 1e-5 * b and abs(fit["alpha"][s].item() - a) <= 1e-5 * a, ("fit", s, fit["beta"][s].item(), b)
            # ---- penalty_grad with random parameters
            gdt = torch.float32 if rng.random() < 0.7 else torch.bfloat16
            gd = [torch.full((n,), 0.25, dtype=gdt, device="cuda:0") for n in lens]
            pb = [float(rng.uniform(0.3, 3.2)) for _ in xs]; pa = [10.0 ** rng.uniform(-3, 0.5) for _ in xs]
            lam = float(rng.choice([1e-4, -3e-3, 2.0])); mean = rng.random() < 0.3; acc = rng.random() < 0.25
            pen = ctx.gg_penalty_grad(xd, torch.tensor(pb, dtype=torch.float64, device="cuda:0"), torch.tensor(pa, dtype=torch.float64, device="cuda:0"),
                                      lam, grad=Segments(gd), reduction=GG_MEAN if mean else GG_SUM, accumulate=acc)
            torch.cuda.synchronize(); ctx.check_guards()
            for s, x in enumerate(xs):
                xo = gg_synth.to_oracle(x)
                p, g = o.penalty_grad(xo, pb[s], pa[s], lam / max(len(xo), 1) if mean else lam)
                if acc: g = (g.astype(np.float32).astype(np.float64) + 0.25) if gdt == torch.float32 else g + 0.25
                got = gd[s].cpu()
                if gdt == torch.float32:
                    fin = np.isfinite(g.astype(np.float32))
                    if acc:
                        assert np.allclose(got.numpy()[fin], g[fin], rtol=1e-6, atol=1e-7), ("grad acc", s)
                    else:
                        d = ulp_distance(got.numpy()[fin], g[fin]); assert d.size == 0 or d.max() <= 4, ("grad", s, int(d.max()))
                else:
                    fin = np.isfinite(g) & (np.abs(g) < 3e38)
                    ref = o.round_to_bf16_bits(g).astype(np.int64); gb = got.view(torch.int16).numpy().astype(np.int64) & 0xFFFF
                    if acc:   # (cancellation against the old value: compare absolutely, at the precision of the gradient itself)
                        gf = got.float().numpy().astype(np.float64)
                        assert np.all(np.abs(gf - g)[fin] <= 2.0 ** -8 * np.abs(g)[fin] + 1e-6 * np.abs(g - 0.25)[fin] + 1e-30), ("grad16 acc", s)
                    else:
                        assert np.abs((ref & 0x7FFF) - (gb & 0x7FFF))[fin].max(initial=0) <= 1, ("grad16", s)
                if np.isfinite(p) and abs(p) > 0: assert abs(pen[s].item() - p) <= 1e-6 * abs(p), ("pen", s, pen[s].item(), p)
            # ---- rate_hist
            n_hist = int(rng.integers(1, 4)); hid = [int(rng.integers(0, n_hist)) for _ in xs]
            qmin, qmax = (-32768, 32767) if rng.random() < 0.5 else (-300, 250)
            steps = np.array([2.0 ** rng.integers(-12, -2) if rng.random() < 0.5 else 10.0 ** rng.uniform(-4, -1) for _ in xs], dtype=np.float32)
            rh = ctx.gg_rate_hist(xd, torch.from_numpy(steps).to("cuda:0"), hist_id=hid, n_hist=n_hist, qmin=qmin, qmax=qmax)
            torch.cuda.synchronize(); ctx.check_guards()
            ref_hist = np.zeros((n_hist, qmax - qmin + 1), dtype=np.uint64); ref_cl = np.zeros((n_hist, 2), dtype=np.uint64)
            for s, x in enumerate(xs):
                o.quantise_hist(gg_synth.to_oracle(x), steps[s], qmin, qmax, hist=ref_hist[hid[s]], clamped=ref_cl[hid[s]])
            assert np.array_equal(rh["hist"].cpu().numpy(), ref_hist.astype(np.int64)), "hist"
            assert np.array_equal(rh["clamped"].cpu().numpy(), ref_cl.astype(np.int64)), "clamped"
            for h in range(n_hist): assert abs(rh["entropy_bits"][h].item() - o.entropy_bits(ref_hist[h])) <= 1e-9, "entropy"
            # ---- sample (a few short tensors)
            ns = [int(rng.integers(1, 30000)) for _ in range(3)]
            sb = [float(rng.uniform(0.25, 6.0)) for _ in ns]; sa = [10.0 ** rng.uniform(-3, 1) for _ in ns]
            outs = [torch.empty(n, dtype=dtype, device="cuda:0") for n in ns]
            seed = int(rng.integers(0, 2 ** 62)); tid0 = int(rng.integers(0, 1000))
            att = ctx.gg_sample(outs, sb, sa, seed, tensor_id0=tid0)
            torch.cuda.synchronize(); ctx.check_guards()
            for s, n in enumerate(ns):
                ref, ra = o.sample(sb[s], sa[s], seed, tid0 + s, n, want_attempts=True)
                got = outs[s].cpu()
                assert att[s].item() == int(ra.max()), ("attempts", s)
                if dtype == torch.bfloat16:
                    rb = o.round_to_bf16_bits(ref).astype(np.int64); gb = got.view(torch.int16).numpy().astype(np.int64) & 0xFFFF
                    assert np.array_equal(rb, gb), ("sample16", s, int((rb != gb).sum()))
                else:
                    d = ulp_distance(got.numpy(), ref); assert d.max() <= 1 and (d > 0).sum() <= max(1, n // 100000), ("sample32", s, int(d.max()), int((d > 0).sum()))
        except AssertionError as e:
            failures.append((desc, str(e)[:300]))
    ctx.close()
    assert not failures, failures
