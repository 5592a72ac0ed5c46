#!/usr/bin/env python
"""Timings of the secondary workloads (everything but the weight sweep that bench.py reports).

    python -m paper_2506_00486_b200.bench_configs [c1] [c2] [c3] [c4] [codes] [calls] [channels]

Each line gives the CUDA-event time of one call through the C interface on cuda:0, inputs resident
in device memory, and the algorithmic GB/s (input read once + output written once).  Inputs are the
seeded synthetic tensors of gg_synth drawn on the device.
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


def main(which):
    dev = torch.device("cuda", 0)
    ctx = Context(0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(2)
    if "c1" in which:
        x = gg_synth.gg_device(gen, 1.0, 0.02, 1024 * 1024, torch.float32, dev)
        g = torch.empty_like(x)
        run = ctx.make_fused(Segments([x]), grad=Segments([g]), lam=1e-4,
                             step=torch.full((1,), 1e-3, dtype=torch.float32, device=dev))
        ms = timeit(run)
        print(f"c1  fused, fp32 1024x1024, one segment: {ms * 1e3:.1f} us  {8 * x.numel() / ms / 1e6:.0f} GB/s")
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            run()
        ms = timeit(graph.replay)
        print(f"c1  the same call replayed from a CUDA graph: {ms * 1e3:.1f} us")
    if "c2" in which:
        shapes = gg_synth.qwen05b_shapes()
        outs = [torch.empty(r * c, dtype=torch.bfloat16, device=dev) for _, r, c in shapes]
        beta, al = 1.3, gg_synth.alpha_for_std(0.02, 1.3)
        n = sum(o.numel() for o in outs)
        ms = timeit(lambda: ctx.gg_sample(outs, [beta] * len(outs), [al] * len(outs), seed=1), 3, 1)
        print(f"c2  gg_sample, {len(outs)} bf16 matrices, {n:.3e} elements: {ms:.2f} ms  {n / ms / 1e6:.1f} G elements/s")
        ms = timeit(lambda: ctx.gg_fit(outs), 5)
        print(f"c2  gg_fit of them: {ms:.3f} ms  {2 * n / ms / 1e6:.0f} GB/s")
        gs = [torch.empty(o_.numel(), dtype=torch.float32, device=dev) for o_ in outs]
        run = ctx.make_fused(Segments(outs), grad=Segments(gs), lam=1e-4,
                             step=torch.full((len(outs),), 2.0 ** -10, dtype=torch.float32, device=dev))
        ms = timeit(run, 5)
        print(f"c2  fused pass over them (fp32 gradients, one histogram per matrix): {ms:.3f} ms  {6 * n / ms / 1e6:.0f} GB/s")
        del gs, run
        del outs
    if "c3" in which:
        a = gg_synth.alpha_for_std(1.0, 0.8)
        x = gg_synth.gg_device(gen, 0.8, a, 8 * 2048 * 4096, torch.bfloat16, dev).view(8 * 2048, 4096)
        gg_synth.add_outliers_device(gen, x, 1e-3, 20.0)
        g = torch.empty(x.shape, dtype=torch.float32, device=dev)
        nseg = x.shape[0]
        run = ctx.make_fused(Segments.rows(x), grad=Segments.rows(g), lam=1e-4,
                             step=torch.full((nseg,), 0.01, dtype=torch.float32, device=dev), hist_id=[0] * nseg, n_hist=1)
        ms = timeit(run)
        print(f"c3  fused, bf16 [8, 2048, 4096], per-token segments, one histogram: {ms * 1e3:.1f} us  "
              f"{6 * x.numel() / ms / 1e6:.0f} GB/s")
        del x, g, run
    if "c4" in which or "codes" in which:
        n = 25_000_000
        xs = [gg_synth.gg_device(gen, 0.5, 10 ** (-6 + 3 * u), n, torch.float32, dev) for u in np.linspace(0.05, 0.95, 8)]
        gs = [torch.empty_like(t) for t in xs]
        if "c4" in which:
            run = ctx.make_fused(Segments(xs), grad=Segments(gs), lam=1e-4, step_scale=1 / 16)
            run()                    # (the first launch of a kernel loads it: keep that out of the sweep timers)
            ctx.timing_enable(True)
            ctx.timing_read()
            ms = timeit(run, 5)
            t = ctx.timing_read()
            ctx.timing_enable(False)
            print(f"c4  fused, 8 fp32 buckets of 25 M, step = alpha / 16: {ms:.3f} ms  {8 * 8 * n / ms / 1e6:.0f} GB/s  "
                  f"(moments {t[0] / t[1]:.3f} ms, gradient + histogram {t[2] / t[3]:.3f} ms)")
        if "codes" in which:
            w = [torch.zeros(n, dtype=torch.float32, device=dev) for _ in range(8)]
            steps = torch.tensor([10 ** (-6 + 3 * u) / 16 for u in np.linspace(0.05, 0.95, 8)], dtype=torch.float32, device=dev)
            sx, sg, sw = Segments(xs), Segments(gs), Segments(w)
            for t_ in gs:
                t_.fill_(1e-4)
            ms = timeit(lambda: ctx.gg_gct_step(sx, sg, sw, steps, 1e-3, 0.05, 1e-8, 2))
            print(f"codes  gg_gct_step, 8 x 25 M fp32: {ms:.3f} ms  {20 * 8 * n / ms / 1e6:.0f} GB/s (3 reads + 2 writes)")
            ms = timeit(lambda: ctx.gg_eg_rate_grad(sx, steps, 0.3, sg))
            print(f"codes  gg_eg_rate_grad, 8 x 25 M fp32: {ms:.3f} ms  {8 * 8 * n / ms / 1e6:.0f} GB/s (1 read + 1 write)")
            rh = ctx.gg_rate_hist(xs, steps)
            ms = timeit(lambda: ctx.gg_eg_rate(rh["hist"]))
            print(f"codes  gg_eg_rate, 8 histograms of 65536 bins: {ms * 1e3:.1f} us")
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
        ms = timeit(lambda: ctx.gg_fit(segs))
        print(f"calls  gg_fit, {len(lens)} bf16 matrices, {n:.3e} elements: {ms:.3f} ms  {2 * n / ms / 1e6:.0f} GB/s")
        ms = timeit(lambda: ctx.gg_penalty_grad(segs, fit["beta"], fit["alpha"], 1e-4, grad=gsegs))
        print(f"calls  gg_penalty_grad (fp32 gradients): {ms:.3f} ms  {6 * n / ms / 1e6:.0f} GB/s")
        ms = timeit(lambda: ctx.gg_rate_hist(segs, steps))
        print(f"calls  gg_rate_hist (one histogram per matrix, entropy): {ms:.3f} ms  {2 * n / ms / 1e6:.0f} GB/s")
        del w, flat, g, segs, gsegs
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
            run()                    # (the first launch of a kernel loads it: keep that out of the sweep timers)
            ctx.timing_enable(True)
            ctx.timing_read()
            ms = timeit(run, 5)
            t = ctx.timing_read()
            ctx.timing_enable(False)
            name = "bf16" if dt == torch.bfloat16 else "fp32"
            print(f"channels  fused, {name} [{rows}, {cols}], column scales 2^-{spread // 2}..2^{spread // 2}, one GG per column, one histogram: {ms * 1e3:.1f} us  "
                  f"{(x.element_size() + 4) * x.numel() / ms / 1e6:.0f} GB/s  (moments {t[0] / t[1] * 1e3:.1f} us, "
                  f"gradient + histogram {t[2] / t[3] * 1e3:.1f} us)")
            del x, g, run
    ctx.close()


if __name__ == "__main__":
    main(set(sys.argv[1:]) or {"c1", "c2", "c3", "c4", "codes", "calls", "channels"})
