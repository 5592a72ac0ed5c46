#!/usr/bin/env python
"""Timings of the secondary workloads (everything but the weight sweep that bench.py times as its headline).

    python -m paper_2506_00486_b200.bench_configs [c1] [c2] [c3] [c4] [codes] [calls] [channels]

Each record gives the CUDA-event time of one call through the C interface on cuda:0, inputs resident in
device memory, and the algorithmic GB/s (input read once + output written once).  Inputs are the seeded
synthetic tensors of gg_synth drawn on the device.  bench.py puts the same records into its JSON line.
"""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gg_synth  # noqa: E402
from paper_2506_00486_b200 import Context, Segments  # noqa: E402

ALL = ("c1", "c2", "c3", "c4", "medium", "codes", "calls", "channels")


def timeit(fn, n=10, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def rec(name, what, ms, alg_bytes=None, steps=10, **extra):
    r = {"name": name, "what": what, "ms": ms, "steps": steps}
    if alg_bytes is not None:
        r["algorithmic_bytes"] = int(alg_bytes)
        r["gbs"] = alg_bytes / ms / 1e6
    r.update(extra)
    return r


def sweeps(ctx, run, n=5):
    """Time of a fused call and of its two sweeps (the library's own event pairs)."""
    run()                            # (the first launch of a kernel loads it: keep that out of the sweep timers)
    ms = timeit(run, n)              # the call as a user sees it: no event pairs inside
    ctx.timing_enable(True)
    ctx.timing_read()
    for _ in range(n):
        run()
    t = ctx.timing_read()
    ctx.timing_enable(False)
    return ms, (t[0] / t[1] if t[1] else None), (t[2] / t[3] if t[3] else None)


def cases(ctx, dev, which=ALL):
    """Yields one record per secondary measurement."""
    gen = torch.Generator(device=dev)
    gen.manual_seed(2)
    if "c1" in which:
        x = gg_synth.gg_device(gen, 1.0, 0.02, 1024 * 1024, torch.float32, dev)
        g = torch.empty_like(x)
        run = ctx.make_fused(Segments([x]), grad=Segments([g]), lam=1e-4,
                             step=torch.full((1,), 1e-3, dtype=torch.float32, device=dev))
        yield rec("c1_fused", "fused pass, fp32 1024x1024, one segment (fits in L2: launch latency, not bandwidth)",
                  timeit(run), 8 * x.numel())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            run()
        yield rec("c1_fused_graph", "the same call replayed from a CUDA graph", timeit(graph.replay), 8 * x.numel())
        del graph
    if "c2" in which:
        shapes = gg_synth.qwen05b_shapes()
        outs = [torch.empty(r * c, dtype=torch.bfloat16, device=dev) for _, r, c in shapes]
        beta, al = 1.3, gg_synth.alpha_for_std(0.02, 1.3)
        n = sum(o.numel() for o in outs)
        ms = timeit(lambda: ctx.gg_sample(outs, [beta] * len(outs), [al] * len(outs), seed=1), 3, 1)
        yield rec("c2_sample", f"gg_sample, {len(outs)} bf16 matrices of a Qwen-0.5B-shaped decoder, {n:.3e} elements",
                  ms, 2 * n, steps=3, g_elements_per_s=n / ms / 1e6, bound="alu")
        yield rec("c2_fit", "gg_fit of them", timeit(lambda: ctx.gg_fit(outs), 5), 2 * n, steps=5)
        gs = [torch.empty(o_.numel(), dtype=torch.float32, device=dev) for o_ in outs]
        run = ctx.make_fused(Segments(outs), grad=Segments(gs), lam=1e-4,
                             step=torch.full((len(outs),), 2.0 ** -10, dtype=torch.float32, device=dev))
        yield rec("c2_fused", "fused pass over them (fp32 gradients, one histogram per matrix)", timeit(run, 5), 6 * n, steps=5)
        del gs, run, outs
    if "c3" in which:
        a = gg_synth.alpha_for_std(1.0, 0.8)
        x = gg_synth.gg_device(gen, 0.8, a, 8 * 2048 * 4096, torch.bfloat16, dev).view(8 * 2048, 4096)
        gg_synth.add_outliers_device(gen, x, 1e-3, 20.0)
        g = torch.empty(x.shape, dtype=torch.float32, device=dev)
        nseg = x.shape[0]
        run = ctx.make_fused(Segments.rows(x), grad=Segments.rows(g), lam=1e-4,
                             step=torch.full((nseg,), 0.01, dtype=torch.float32, device=dev), hist_id=[0] * nseg, n_hist=1)
        yield rec("c3_fused", "fused pass, bf16 [8, 2048, 4096] activations with outliers, per-token segments, one histogram",
                  timeit(run), 6 * x.numel())
        del g, run
        xf = x.float()
        gf = torch.empty_like(xf)
        run = ctx.make_fused(Segments.rows(xf), grad=Segments.rows(gf), lam=1e-4,
                             step=torch.full((nseg,), 0.01, dtype=torch.float32, device=dev), hist_id=[0] * nseg, n_hist=1)
        yield rec("c3_fused_fp32", "the same activations in fp32", timeit(run), 8 * xf.numel())
        del x, xf, gf, run
    if "c4" in which or "codes" in which:
        n = 25_000_000
        xs = [gg_synth.gg_device(gen, 0.5, 10 ** (-6 + 3 * u), n, torch.float32, dev) for u in np.linspace(0.05, 0.95, 8)]
        gs = [torch.empty_like(t) for t in xs]
        if "c4" in which:
            run = ctx.make_fused(Segments(xs), grad=Segments(gs), lam=1e-4, step_scale=1 / 16)
            ms, first, tail = sweeps(ctx, run)
            yield rec("c4_fused", "fused pass, 8 fp32 gradient buckets of 25 M, step = alpha / 16", ms, 8 * 8 * n, steps=5,
                      first_sweep_ms=first, second_sweep_ms=tail)
            fit = run.outputs
            from paper_2506_00486_b200 import GG_PARAMS_GIVEN
            steps = run.outputs["step"].clone()
            run1 = ctx.make_fused(Segments(xs), grad=Segments(gs), lam=1e-4, step=steps, param_mode=GG_PARAMS_GIVEN,
                                  beta_in=fit["beta"].clone(), alpha_in=fit["alpha"].clone())
            ms, first, tail = sweeps(ctx, run1)
            yield rec("c4_fused_given", "the same with the parameters of the step before (penalty lags one step)", ms, 8 * 8 * n,
                      steps=5, first_sweep_ms=first, second_sweep_ms=tail)
            del run, run1
        if "codes" in which:
            w = [torch.zeros(n, dtype=torch.float32, device=dev) for _ in range(8)]
            steps = torch.tensor([10 ** (-6 + 3 * u) / 16 for u in np.linspace(0.05, 0.95, 8)], dtype=torch.float32, device=dev)
            sx, sg, sw = Segments(xs), Segments(gs), Segments(w)
            for t_ in gs:
                t_.fill_(1e-4)
            yield rec("gct_step", "gg_gct_step (Algorithm 2), 8 x 25 M fp32: 3 reads + 2 writes",
                      timeit(lambda: ctx.gg_gct_step(sx, sg, sw, steps, 1e-3, 0.05, 1e-8, 2)), 20 * 8 * n)
            yield rec("eg_rate_grad", "gg_eg_rate_grad, 8 x 25 M fp32: 1 read + 1 write",
                      timeit(lambda: ctx.gg_eg_rate_grad(sx, steps, 0.3, sg)), 8 * 8 * n)
            rh = ctx.gg_rate_hist(xs, steps)
            yield rec("eg_rate", "gg_eg_rate, 8 histograms of 65536 bins", timeit(lambda: ctx.gg_eg_rate(rh["hist"])), 8 * 8 * 65536)
            del w
        del xs, gs
    if "medium" in which:
        # bf16 segments between the short-segment kernels and the long sweeps: one thread-block cluster per segment
        # (the segment staged in shared memory, one DRAM read) against the two sweeps
        from paper_2506_00486_b200.binding import HOOK_CLUSTER_MODE
        for n_seg, seg_len, label in ((4096, 32768, "64 KB"), (1024, 131072, "256 KB"), (256, 524288, "1 MB")):
            x = gg_synth.gg_device(gen, 1.1, gg_synth.alpha_for_std(0.02, 1.1), n_seg * seg_len, torch.bfloat16, dev)
            g = torch.empty(x.numel(), dtype=torch.float32, device=dev)
            offs, lens = [s * seg_len for s in range(n_seg)], [seg_len] * n_seg
            steps = torch.full((n_seg,), 2.0 ** -10, dtype=torch.float32, device=dev)
            for mode, name in ((2, "cluster"), (0, "sweeps")):
                ctx.gg_test_hook(HOOK_CLUSTER_MODE, mode)
                run = ctx.make_fused(Segments.slices(x, offs, lens), grad=Segments.slices(g, offs, lens), lam=1e-4, step=steps,
                                     hist_id=[0] * n_seg, n_hist=1)
                yield rec(f"medium_{n_seg}x{seg_len}_{name}",
                          f"fused pass, {n_seg} bf16 segments of {label}, one histogram; " +
                          ("one cluster per segment, staged in shared memory" if mode else "moments sweep, then gradient + histogram sweep"),
                          timeit(run, 5), 6 * x.numel(), steps=5)
                del run
            ctx.gg_test_hook(HOOK_CLUSTER_MODE, 0)
            del x, g
    if "calls" in which:
        # the single-step entry points on the Llama-7B-shaped sweep with every dimension halved (1.68e9 elements)
        w = gg_synth.workload_c5_device(dev, torch.bfloat16, shapes=gg_synth.scaled_shapes(gg_synth.llama7b_shapes(), 2), seed=4)
        flat, offs, lens = w["flat"], w["offsets"], w["lens"]
        segs = Segments.slices(flat, offs, lens)
        g = torch.empty(flat.numel(), dtype=torch.float32, device=dev)
        gsegs = Segments.slices(g, offs, lens)
        n = flat.numel()
        steps = torch.full((len(lens),), 2.0 ** -10, dtype=torch.float32, device=dev)
        fit = ctx.gg_fit(segs)
        yield rec("call_fit", f"gg_fit, {len(lens)} bf16 matrices (Llama-7B shapes with halved dimensions), {n:.3e} elements",
                  timeit(lambda: ctx.gg_fit(segs)), 2 * n)
        yield rec("call_penalty_grad", "gg_penalty_grad on them (fp32 gradients)",
                  timeit(lambda: ctx.gg_penalty_grad(segs, fit["beta"], fit["alpha"], 1e-4, grad=gsegs)), 6 * n)
        yield rec("call_rate_hist", "gg_rate_hist on them (one histogram per matrix, entropy)",
                  timeit(lambda: ctx.gg_rate_hist(segs, steps)), 2 * n)
        # the training step of the paper's rate-constrained objective (loss + lambda * R, R the Exponential-Golomb
        # code length of Eq. 6-7): gradient of the rate, histogram and rate of every matrix
        from paper_2506_00486_b200 import GG_RATE_EG
        run = ctx.make_fused(segs, grad=gsegs, lam=1e-4, step=steps, param_mode=GG_RATE_EG, eg_k=0)
        yield rec("rate_step_fused", "gg_fused with GG_RATE_EG on them: fit, gradient of lambda * R, histogram, entropy and code length "
                  "of every matrix from one read (fp32 gradients)", timeit(run), 6 * n)

        hist = run.outputs["hist"]

        def separate():
            ctx.gg_eg_rate_grad(segs, steps, 1e-4, gsegs, k=0)
            ctx.gg_rate_hist(segs, steps, hist=hist)
            ctx.gg_eg_rate(hist, k=0)
        yield rec("rate_step_separate", "the same from the single-step calls (gg_eg_rate_grad, gg_rate_hist, gg_eg_rate: two reads, no fit)",
                  timeit(separate), 6 * n)
        del w, flat, g, segs, gsegs, run
    if "channels" in which:
        for rows, cols, spread, dt in ((16384, 4096, 3, torch.bfloat16), (65536, 4096, 3, torch.bfloat16),
                                       (16384, 11008, 3, torch.bfloat16), (16384, 4096, 9, torch.bfloat16),
                                       (16384, 4096, 3, torch.float32)):
            # column c scaled by 2^(c mod spread - spread // 2): with 9 the widest columns' symbols leave the
            # shared symbol window and their strips are counted by bit pattern
            a = gg_synth.alpha_for_std(1.0, 0.8)
            x = gg_synth.gg_device(gen, 0.8, a, rows * cols, dt, dev).view(rows, cols)
            x.mul_(torch.exp2(torch.arange(cols, device=dev) % spread - float(spread // 2)).to(dt))
            gg_synth.add_outliers_device(gen, x, 1e-3, 20.0)
            g = torch.empty((rows, cols), dtype=torch.float32, device=dev)
            run = ctx.make_fused_channels(x, grad=g, lam=1e-4, step=0.01)
            ms, first, tail = sweeps(ctx, run)
            name = "bf16" if dt == torch.bfloat16 else "fp32"
            yield rec(f"channels_{name}_{rows}x{cols}_spread{spread}",
                      f"gg_fused_channels, {name} [{rows}, {cols}], column scales 2^-{spread // 2}..2^{spread // 2}, one GG per column, one histogram",
                      ms, (x.element_size() + 4) * x.numel(), steps=5, first_sweep_ms=first, second_sweep_ms=tail)
            del x, g, run


def main(which):
    dev = torch.device("cuda", 0)
    ctx = Context(0)
    for r in cases(ctx, dev, which):
        line = f"{r['name']:<36s} {r['ms'] * 1e3:10.1f} us"
        if "gbs" in r:
            line += f"  {r['gbs']:7.0f} GB/s"
        for k in ("first_sweep_ms", "second_sweep_ms", "g_elements_per_s"):
            if r.get(k) is not None:
                line += f"  {k} {r[k]:.3f}"
        print(line + "   " + r["what"], flush=True)
    ctx.close()


if __name__ == "__main__":
    main(set(sys.argv[1:]) or set(ALL))
