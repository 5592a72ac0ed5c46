#!/usr/bin/env python
"""Benchmark of the fused GG pass (fit + penalty gradient + symbol histogram + entropy).

One step = one gg_fused call (parameters fitted in the same call) over the whole Llama-7B-shaped
bf16 weight sweep: 226 tensors, 6.74e9 elements, each GG with its own shape in [0.6, 1.6] and
standard deviation 0.02; fp32 gradients; one 65536-bin histogram per tensor at step 2^-10.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused GG fit+penalty-grad+histogram pass throughput (algorithmic bytes: input read once + gradient written once)"
UNIT = "GB/s"
LAM = 1e-4
STEP = 2.0 ** -10


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--divisor", type=int, default=1,
                    help="divide every matrix dimension of the sweep (debugging; 1 = the full workload)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--sweep-steps", type=int, default=20,
                    help="steps of the separate loop that times the two sweeps of the pass with the library's event pairs")
    ap.add_argument("--no-secondary", action="store_true", help="skip the other workloads (the `secondary` object)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--single-read-steps", type=int, default=20,
                    help="timed steps of the one-read form of the pass (parameters given), 0 to skip")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--grad-dtype", default="f32", choices=["f32", "bf16"])
    ap.add_argument("--one-launch", action="store_true",
                    help="time the one-launch form of the fitted pass (every tensor handed from its moments to its second "
                         "read through L2; slower on B200, off by default) instead of the two sweeps")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy kernel)"
    except Exception:
        return 6650.0, "fallback (earlier copy measurement on this pool)"


TAIL_KERNEL_SOURCE = os.path.join(ROOT, "paper_2506_00486_b200", "csrc", "gg_tail_bf16.cu")


def whole_call_traffic(n_elem, grad_dtype):
    """DRAM bytes (read, written) of one whole fused call from the committed one-pass ncu capture at full size
    (profiles/traffic_whole_call_llama7b.txt).  None unless this run is that workload and every kernel source named
    in the file is the one the counters were taken on."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic_whole_call_llama7b.txt")
    try:
        kv, digests = {}, {}
        with open(path) as f:
            for line in f:
                if "=" not in line or line.lstrip().startswith("#"):
                    continue
                k, v = (t.strip() for t in line.split("=", 1))
                if k.startswith("sha256 "):
                    digests[k[7:]] = v
                else:
                    kv[k] = v
        if int(kv["elements"]) != n_elem or kv["grad_dtype"] != grad_dtype:
            return None
        for name, want in digests.items():
            with open(os.path.join(ROOT, "paper_2506_00486_b200", "csrc", name), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != want:
                    return None
        return float(kv["dram_bytes_read_per_call"]), float(kv["dram_bytes_written_per_call"])
    except Exception:
        return None


def traffic_per_element(grad_dtype):
    """DRAM bytes per element of the second-sweep kernel from the committed ncu capture
    (profiles/traffic_tail_bf16_kernel.txt: `key = value` lines).  None if there is no capture for this
    gradient type or if the kernel source has changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic_tail_bf16_kernel.txt")
    try:
        kv = {}
        with open(path) as f:
            for line in f:
                if "=" in line and not line.lstrip().startswith("#"):
                    k, v = line.split("=", 1)
                    kv[k.strip()] = v.strip()
        with open(TAIL_KERNEL_SOURCE, "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
        if kv.get("kernel_source_sha256") != digest or kv.get("grad_dtype") != grad_dtype:
            return None
        return float(kv["dram_bytes_per_element"])
    except Exception:
        return None


class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, power, reasons = [], [], [], set()
        for line in self.file:
            p = [v.strip() for v in line.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2])); power.append(float(p[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            # "under load": samples in the upper half of the power range seen
            lim = (max(power) + min(power)) / 2
            load = sorted(s for s, w in zip(sm, power) if w >= lim) or sorted(sm)
            out.update(sm_mhz=load[len(load) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return out


# ------------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(divisor, max_elements=None):
    """A bounded sample of the workload for the CPU oracle: the matrices of layer 0 of the sweep (all seven,
    or as many of them, or as long a piece of the first, as max_elements allows), generated on the host with
    the same recipe."""
    import numpy as np
    import torch
    import gg_synth
    shapes, betas, alphas = gg_synth.workload_c5_params(
        gg_synth.scaled_shapes(gg_synth.llama7b_shapes(), divisor) if divisor > 1 else None)
    rng = np.random.default_rng(4)
    xs, n = [], 0
    for i in range(1, 8):        # layer 0: q, k, v, o, gate, up, down
        _, r, c = shapes[i]
        m = r * c
        if max_elements is not None and n + m > max_elements:
            if not xs:
                m = max(1024, int(max_elements))
                xs.append(gg_synth.to_oracle(gg_synth.gg_host(rng, betas[i], alphas[i], m, torch.bfloat16)))
                n += m
            break
        xs.append(gg_synth.to_oracle(gg_synth.gg_host(rng, betas[i], alphas[i], m, torch.bfloat16)))
        n += m
    return xs, f"{len(xs)} of the 7 bf16 matrices of layer 0 of the sweep ({n:.3e} of 6.74e9 elements)"


def oracle_step(xs):
    """The whole pass, tensor by tensor, with the oracle as it stands."""
    from oracle import gg_oracle as o
    acc = 0.0
    for x in xs:
        b, a, *_ = o.fit(x)
        pen, g = o.penalty_grad(x, b, a, LAM)
        hist, _ = o.quantise_hist(x, STEP)
        acc += o.entropy_bits(hist) + pen
    return acc


def time_oracle(xs, steps, warmup):
    for _ in range(warmup):
        oracle_step(xs)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(xs)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    alg = sum(x.size for x in xs) * (2 + 4)
    return alg / dt / 1e9, dt


def omp_threads():
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v and v.isdigit() else (os.cpu_count() or 1)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import gg_oracle as o
    o.build()
    # exactly the steps asked for, on a sample sized so that all of them take about two minutes (the oracle
    # does about 50 M elements per second on 16 cores)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    x, what = oracle_sample(args.divisor, max_elements=120.0 * 50e6 / (steps + warmup))
    gbs, dt = time_oracle(x, steps, warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama7b_weight_sweep_bf16 (oracle on a bounded sample)", "sample": what},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": omp_threads(), "kind": "oracle", "sample": what},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------- whole-job figures over ranks
def max_over_ranks(value, world, device="cpu"):
    """The largest of the ranks' values (every rank gets it): the job is as slow as its slowest rank."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def whole_job_gbs(world, bytes_per_rank, ms):
    """Replicas are independent (weak scaling): the job moves world * bytes_per_rank in the slowest rank's time."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


# ----------------------------------------------------------------------------------- GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import gg_synth
    from paper_2506_00486_b200 import Context, Segments

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- workload: every rank holds the whole sweep (segments are independent: weak scaling)
    shapes = gg_synth.scaled_shapes(gg_synth.llama7b_shapes(), args.divisor) if args.divisor > 1 else None
    w = gg_synth.workload_c5_device(dev, torch.bfloat16, shapes=shapes, seed=4 + rank)
    flat, offs, lens = w["flat"], w["offsets"], w["lens"]
    n_seg, n_elem = len(lens), int(sum(lens))
    gdtype = torch.float32 if args.grad_dtype == "f32" else torch.bfloat16
    gflat = torch.empty(flat.numel(), dtype=gdtype, device=dev)
    segs = Segments.slices(flat, offs, lens)
    gsegs = Segments.slices(gflat, offs, lens)
    steps_t = torch.full((n_seg,), STEP, dtype=torch.float32, device=dev)
    ctx = Context(local)
    if args.one_launch:
        ctx.gg_test_hook(0, 1)
    run = ctx.make_fused(segs, grad=gsegs, lam=LAM, step=steps_t)
    in_bytes = n_elem * 2
    g_bytes = n_elem * gflat.element_size()
    alg_bytes = in_bytes + g_bytes

    for _ in range(args.warmup):
        run()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = ctx.launch_count
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        run()
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1) / max(args.steps, 1)
    launches = ctx.launch_count - launches0
    # the two sweeps by themselves, in a loop of their own: the library's event pairs stay out of the headline loop
    ctx.timing_enable(True)
    ctx.timing_read()
    for _ in range(args.sweep_steps):
        run()
    ms_first, n_first, ms_tail, n_tail = ctx.timing_read()
    ctx.timing_enable(False)
    clocks = sampler.stop() if sampler else None
    ms = max_over_ranks(ms, world, dev)
    value = whole_job_gbs(world, alg_bytes, ms)

    # ---- a quick self-check of the timed outputs (host logic only: no oracle here)
    out = run.outputs
    torch.cuda.synchronize()
    beta_err = max(abs(out["beta"][s].item() - w["beta_true"][s]) for s in range(n_seg))
    total_counts = int(out["hist"].sum().item())

    # ---- roofline of the dominant kernel (the second sweep: read x, write the gradient, histogram)
    peak, peak_src = measured_peak()
    tail_ms = ms_tail / max(n_tail, 1)
    first_ms = ms_first / max(n_first, 1)
    achieved = alg_bytes / (tail_ms * 1e-3) / 1e9 if tail_ms > 0 else None
    tr = None if args.one_launch else traffic_per_element(args.grad_dtype)
    traffic = tr * n_elem if tr is not None else None
    kernel = ("resident_bf16_kernel<%s grad, grad|hist> (moments, fit and second read in one launch)" if args.one_launch
              else "tail_bf16_kernel<%s grad, grad|hist> (second sweep)") % args.grad_dtype
    roofline = {"bound": "hbm", "kernel": kernel,
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak if achieved else None,
                "frac_of_nominal_8TBs": achieved / 8000.0 if achieved else None,
                "traffic": traffic, "peak_source": peak_src, "ms_per_launch": tail_ms,
                "algorithmic_bytes_per_launch": alg_bytes,
                "first_sweep": {"ms_per_launch": first_ms,
                                "achieved": in_bytes / (first_ms * 1e-3) / 1e9 if first_ms > 0 else None,
                                "frac": in_bytes / (first_ms * 1e-3) / 1e9 / peak if first_ms > 0 else None}}

    # ---- what DRAM moves per call (counters of the committed capture) over this run's time per call: the second
    # read of x is traffic that the algorithmic figure does not count
    dram = None
    wc = None if args.one_launch else whole_call_traffic(n_elem, args.grad_dtype)
    if wc is not None and ms > 0:
        rate = (wc[0] + wc[1]) / (ms * 1e-3) / 1e9
        dram = {"bytes_read_per_step": wc[0], "bytes_written_per_step": wc[1], "achieved": rate, "unit": "GB/s per GPU",
                "of_measured_copy_peak": rate / peak, "of_nominal_8TBs": rate / 8000.0,
                "bytes_per_element": (wc[0] + wc[1]) / n_elem,
                "source": "profiles/traffic_whole_call_llama7b.txt (one-pass ncu capture of the same call at full size)"}

    # ---- the one-read form of the same pass (secondary figure): the parameters of the step before (here:
    # those just fitted) drive penalty and gradient while the new fit is made in the same sweep
    single = None
    if args.single_read_steps > 0:
        from paper_2506_00486_b200 import GG_PARAMS_GIVEN
        run1 = ctx.make_fused(segs, grad=gsegs, lam=LAM, step=steps_t, param_mode=GG_PARAMS_GIVEN,
                              beta_in=out["beta"].clone(), alpha_in=out["alpha"].clone(), hist=out["hist"])
        for _ in range(3):
            run1()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.single_read_steps):
            run1()
        e1.record()
        barrier()
        ms1 = max_over_ranks(e0.elapsed_time(e1) / args.single_read_steps, world, dev)
        v1 = whole_job_gbs(world, alg_bytes, ms1)
        single = {"value": v1, "unit": UNIT, "ms_per_step": ms1, "steps": args.single_read_steps,
                  "params": "given (those of the previous step); moments, fit, gradient and histogram in one sweep",
                  "of_measured_copy_peak": v1 / world / peak}
        del run1

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, ctx, w, world, dev, gdtype, in_bytes, g_bytes, alg_bytes, barrier)

    # ---- the other workloads (rank 0, one GPU): a few timed calls each, as fractions of the same measured peak
    secondary = None
    if rank == 0 and world == 1 and not args.no_secondary and args.divisor == 1:
        from paper_2506_00486_b200 import bench_configs
        secondary = {}
        for r in bench_configs.cases(ctx, dev):
            if "gbs" in r and r.get("bound") != "alu":
                r["of_measured_copy_peak"] = r["gbs"] / peak
            secondary[r.pop("name")] = r

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import gg_oracle as o
        o.build()
        x, what = oracle_sample(args.divisor)
        gbs, dt = time_oracle(x, 3, 0)
        cpu_baseline = {"value": gbs, "unit": UNIT, "cores": omp_threads(), "kind": "oracle",
                        "sample": what + f"; three passes of {dt:.1f} s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "llama7b_weight_sweep_bf16" + ("" if args.divisor == 1 else f"/div{args.divisor}"),
                       "segments": n_seg, "elements": n_elem, "in_dtype": "bf16", "grad_dtype": args.grad_dtype,
                       "histograms": n_seg, "bins": 65536, "step": STEP, "lambda": LAM, "params": "fitted in the same call",
                       "l2": "inputs larger than L2 (no flush needed)", "parallelism": f"replicas x{world} (segments are independent)"},
            "fraction_of_hbm_peak": {"of_measured_copy_peak": value / world / peak, "of_nominal_8TBs": value / world / 8000.0},
            "dram": dram,
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "single_read": single,
            "secondary": secondary,
            "gpu_launches": int(launches),
            "clocks": clocks,
            "check": {"max_abs_beta_error_vs_generating": beta_err, "histogram_total": total_counts,
                      "elements": n_elem},
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, ctx, w, world, dev, gdtype, in_bytes, g_bytes, alg_bytes, barrier):
    import psutil
    import torch
    from paper_2506_00486_b200 import Segments
    local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
    need = in_bytes + g_bytes
    avail = psutil.virtual_memory().available / max(local_world, 1)
    if need * 1.25 > avail:
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": g_bytes,
                "skipped": f"host memory: need {need / 1e9:.0f} GB pinned per rank, {avail / 1e9:.0f} GB available"}
    flat, offs, lens = w["flat"], w["offsets"], w["lens"]
    n_seg = len(lens)
    hx = torch.empty(flat.numel(), dtype=flat.dtype, pin_memory=True)
    hx.copy_(flat)
    hg = torch.empty(flat.numel(), dtype=gdtype, pin_memory=True)
    hstep = torch.full((n_seg,), STEP, dtype=torch.float32)
    runh = ctx.make_fused_host(Segments.slices(hx, offs, lens), grad=Segments.slices(hg, offs, lens),
                               lam=LAM, step=hstep)
    runh()                                      # warm-up: allocates the staging buffers and plans
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        runh()
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / max(args.e2e_steps, 1)
    dt = max_over_ranks(dt, world, dev)
    out = runh.outputs
    d2h = g_bytes + out["hist"].numel() * 8 + n_seg * (8 * 6 + 4 + 8 + 16)
    return {"value": whole_job_gbs(world, alg_bytes, dt * 1e3), "unit": UNIT, "ms_per_step": dt * 1e3, "steps": args.e2e_steps,
            "h2d_bytes_per_step": in_bytes + n_seg * 4, "d2h_bytes_per_step": int(d2h),
            "api": "gg_fused_host (pinned host tensors in, gradients + fit + histograms back on the host)"}


if __name__ == "__main__":
    a = parse()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
