"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

Only input recipes live here: tensor shapes of the workloads and draws from library random
number generators (numpy on the host, torch on the device).  None of the method's own
arithmetic (moments, fit, penalty, quantiser, the Philox/Marsaglia-Tsang sampler) is here,
and neither the CUDA library nor the CPU oracle is imported.

A GG(0, alpha, beta) variate is drawn as alpha * s * G**(1/beta) with G ~ Gamma(1/beta, 1)
from the library generator and s a fair sign; alpha for a wanted standard deviation uses
the standard-deviation/scale relation of the density (Eq. 2), evaluated with math.lgamma.
"""
import math

import numpy as np
import torch


def alpha_for_std(std, beta):
    """Scale that gives the wanted standard deviation (Eq. 2)."""
    return std * math.exp(0.5 * (math.lgamma(1.0 / beta) - math.lgamma(3.0 / beta)))


# ------------------------------------------------------------------ shapes
def llama7b_shapes():
    """The 226 weight matrices of a Llama-7B-shaped decoder (32 layers, hidden 4096,
    MLP 11008, 32 heads, vocabulary 32000); norm vectors are not included."""
    shapes = [("embed", 32000, 4096)]
    for l in range(32):
        for name in ("q", "k", "v", "o"):
            shapes.append((f"l{l}.{name}", 4096, 4096))
        shapes.append((f"l{l}.gate", 11008, 4096))
        shapes.append((f"l{l}.up", 11008, 4096))
        shapes.append((f"l{l}.down", 4096, 11008))
    shapes.append(("lm_head", 32000, 4096))
    return shapes


def qwen05b_shapes():
    """The 169 weight matrices of a Qwen-0.5B-shaped decoder (24 layers, hidden 896, MLP 4864,
    14 query heads and 2 key/value heads of dimension 64, vocabulary 151936, tied output head)."""
    shapes = [("embed", 151936, 896)]
    for l in range(24):
        shapes.append((f"l{l}.q", 896, 896))
        shapes.append((f"l{l}.k", 128, 896))
        shapes.append((f"l{l}.v", 128, 896))
        shapes.append((f"l{l}.o", 896, 896))
        shapes.append((f"l{l}.gate", 4864, 896))
        shapes.append((f"l{l}.up", 4864, 896))
        shapes.append((f"l{l}.down", 896, 4864))
    return shapes


def scaled_shapes(shapes, divisor):
    """The same list with both matrix dimensions divided (for cases a CPU finishes in seconds)."""
    return [(n, max(1, r // divisor), max(1, c // divisor)) for n, r, c in shapes]


# ------------------------------------------------------------ host (numpy)
def gg_host(rng, beta, alpha, n, dtype=torch.float32):
    """n GG variates as a CPU torch tensor of the storage dtype (values rounded to it)."""
    g = rng.gamma(1.0 / beta, 1.0, size=n)
    s = np.where(rng.random(n) < 0.5, -1.0, 1.0)
    x = alpha * s * np.power(g, 1.0 / beta)
    return torch.from_numpy(x.astype(np.float32)).to(dtype)


def add_outliers_host(rng, t, fraction, magnitude):
    """Replace a seeded fraction of the entries by +-magnitude."""
    n = t.numel()
    mask = rng.random(n) < fraction
    sign = np.where(rng.random(n) < 0.5, -1.0, 1.0)
    x = t.float().numpy().copy().reshape(-1)
    x[mask] = (sign * magnitude)[mask]
    return torch.from_numpy(x).to(t.dtype).reshape(t.shape)


def to_oracle(t):
    """Exact widening of a stored tensor to the fp32 numpy array the oracle takes."""
    return t.detach().cpu().float().contiguous().numpy().reshape(-1)


# ---------------------------------------------------------- device (torch)
def gg_device(gen, beta, alpha, n, dtype, device, out=None, chunk=1 << 26):
    """n GG variates on `device` from torch's generator `gen`, written into `out` if given.

    Drawn in chunks so the fp32 temporaries stay small next to multi-GB workloads."""
    if out is None:
        out = torch.empty(n, dtype=dtype, device=device)
    inv_beta = 1.0 / beta
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        conc = torch.full((m,), inv_beta, dtype=torch.float32, device=device)
        g = torch._standard_gamma(conc, generator=gen)
        g.pow_(inv_beta).mul_(alpha)
        sign = torch.randint(0, 2, (m,), generator=gen, device=device, dtype=torch.int8)
        g.mul_(sign.to(torch.float32).mul_(2.0).sub_(1.0))
        out[lo:lo + m].copy_(g)
        del conc, g, sign
    return out


def add_outliers_device(gen, t, fraction, magnitude):
    flat = t.view(-1)
    u = torch.rand(flat.numel(), generator=gen, device=t.device)
    mask = u < fraction
    sign = (torch.rand(flat.numel(), generator=gen, device=t.device) < 0.5)
    vals = torch.where(sign, -magnitude, magnitude).to(t.dtype)
    flat[mask] = vals[mask]
    return t


# ---------------------------------------------------- the named workloads
def workload_c1(device="cpu"):
    """fp32 1024x1024 from GG(beta=1, alpha=0.02), seed 0; one segment; lambda 1e-4; step 1e-3."""
    rng = np.random.default_rng(0)
    x = gg_host(rng, 1.0, 0.02, 1024 * 1024, torch.float32)
    return dict(tensors=[x.to(device)], lam=1e-4, steps=[1e-3], hist_id=[0], n_hist=1,
                beta_true=[1.0], alpha_true=[0.02])


def workload_c3(device="cpu", batch=8, seq=2048, hidden=4096):
    """bf16 activations [batch, seq, hidden] from GG(beta=0.8, std 1) with 0.1 % of the entries
    replaced by +-20 sigma; one segment per token; one shared histogram; step 0.01."""
    rng = np.random.default_rng(2)
    a = alpha_for_std(1.0, 0.8)
    n = batch * seq * hidden
    x = gg_host(rng, 0.8, a, n, torch.bfloat16)
    x = add_outliers_host(rng, x, 1e-3, 20.0)
    x = x.reshape(batch * seq, hidden).to(device)
    n_seg = batch * seq
    return dict(tensor=x, n_seg=n_seg, seg_len=hidden, lam=1e-4, step=0.01,
                hist_id=[0] * n_seg, n_hist=1)


def workload_c4(device="cpu", n_buckets=8, bucket=25_000_000):
    """fp32 gradient buckets from GG(beta=0.5) with per-bucket alpha log-uniform in [1e-6, 1e-3],
    seed 3; step alpha/16 per bucket; one histogram per bucket."""
    rng = np.random.default_rng(3)
    alphas = [10.0 ** (-6.0 + 3.0 * rng.random()) for _ in range(n_buckets)]
    tensors = [gg_host(rng, 0.5, a, bucket, torch.float32).to(device) for a in alphas]
    steps = [float(np.float32(a / 16.0)) for a in alphas]
    return dict(tensors=tensors, lam=1e-4, steps=steps, hist_id=list(range(n_buckets)),
                n_hist=n_buckets, beta_true=[0.5] * n_buckets, alpha_true=alphas)


def workload_c5_params(shapes=None, seed=4):
    """Per-tensor (beta, alpha) of the weight sweep: beta uniform in [0.6, 1.6], std 0.02."""
    shapes = llama7b_shapes() if shapes is None else shapes
    rng = np.random.default_rng(seed)
    betas = [0.6 + rng.random() for _ in shapes]
    alphas = [alpha_for_std(0.02, b) for b in betas]
    return shapes, betas, alphas


def workload_c5_host(divisor=16, dtype=torch.bfloat16):
    """The weight sweep with every matrix dimension divided by `divisor`, on the host."""
    shapes, betas, alphas = workload_c5_params(scaled_shapes(llama7b_shapes(), divisor))
    rng = np.random.default_rng(4)
    tensors = [gg_host(rng, b, a, r * c, dtype) for (_, r, c), b, a in zip(shapes, betas, alphas)]
    return dict(tensors=tensors, lam=1e-4, steps=[2.0 ** -10] * len(shapes),
                hist_id=list(range(len(shapes))), n_hist=len(shapes),
                beta_true=betas, alpha_true=alphas)


def workload_c5_device(device, dtype=torch.bfloat16, shapes=None, seed=4):
    """The full weight sweep as ONE flat device buffer plus per-tensor (offset, length)."""
    shapes, betas, alphas = workload_c5_params(shapes, seed)
    lens = [r * c for _, r, c in shapes]
    # every tensor starts on a 256-byte boundary inside the flat buffer
    align = 256 // torch.empty(0, dtype=dtype).element_size()
    offs, total = [], 0
    for n in lens:
        offs.append(total)
        total += (n + align - 1) // align * align
    flat = torch.zeros(total, dtype=dtype, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    for off, n, b, a in zip(offs, lens, betas, alphas):
        gg_device(gen, b, a, n, dtype, device, out=flat[off:off + n])
    return dict(flat=flat, offsets=offs, lens=lens, lam=1e-4, steps=[2.0 ** -10] * len(lens),
                hist_id=list(range(len(lens))), n_hist=len(lens),
                beta_true=betas, alpha_true=alphas, shapes=shapes)
