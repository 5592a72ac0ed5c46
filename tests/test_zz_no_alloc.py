"""gg_fit_noalloc: the fit for callers that cannot allocate device memory (a frozen or pool-owned
allocator, a plug-in that only receives buffers and a stream).  Its tile tables and partial sums
live in a fixed array inside the library, shared by all calls on a device, instead of a plan
obtained with cudaMalloc.  Checked here through the C interface against gg_fit on the same data,
on two calls in a row whose sizes differ, so that anything the first call left in the array
would show up in the second."""
import ctypes

import pytest
import torch

import gg_synth
from parity_util import REL_FIT, assert_rel

pytestmark = pytest.mark.gpu

TILE = 16384


def call_noalloc(L, x):
    dev = x.device
    o = dict(beta=torch.full((1,), -1.0, dtype=torch.float64, device=dev),
             alpha=torch.full((1,), -1.0, dtype=torch.float64, device=dev),
             sum_abs=torch.full((1,), -1.0, dtype=torch.float64, device=dev),
             sum_sq=torch.full((1,), -1.0, dtype=torch.float64, device=dev),
             count=torch.full((1,), -1, dtype=torch.int64, device=dev),
             flags=torch.full((1,), -1, dtype=torch.int32, device=dev))
    code = 0 if x.dtype == torch.float32 else 1
    st = L.gg_fit_noalloc(dev.index or 0, ctypes.c_void_p(x.data_ptr()), x.numel(), code,
                          *(ctypes.c_void_p(o[k].data_ptr()) for k in ("beta", "alpha", "sum_abs", "sum_sq", "count", "flags")),
                          ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream))
    assert st == 0, L.gg_status_str(st)
    return o


def test_noalloc_fit_matches_gg_fit_on_two_calls_in_a_row():
    import numpy as np
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import Context, binding
    L = binding.lib()
    rng = np.random.default_rng(77)
    # the second call is shorter than the first and of the other dtype: stale tiles must not leak in
    cases = [gg_synth.gg_host(rng, 0.7, 0.02, 9 * TILE + 1234, torch.bfloat16),
             gg_synth.gg_host(rng, 1.4, 0.3, 2 * TILE + 5, torch.float32),
             torch.zeros(100, dtype=torch.float32),
             gg_synth.gg_host(rng, 1.0, 1.0, 7, torch.bfloat16)]
    xs = [x.to("cuda:0") for x in cases]
    got = [call_noalloc(L, x) for x in xs]          # back to back on one stream
    torch.cuda.synchronize()
    ctx = Context(0)
    ref = ctx.gg_fit(xs[0:1]), ctx.gg_fit(xs[1:2]), ctx.gg_fit(xs[2:3]), ctx.gg_fit(xs[3:4])
    torch.cuda.synchronize()
    for g, r, x in zip(got, ref, xs):
        assert g["count"].item() == r["count"].item() == x.numel()
        assert g["flags"].item() == r["flags"].item()
        for k, tol in (("beta", REL_FIT), ("alpha", REL_FIT), ("sum_abs", 1e-7), ("sum_sq", 1e-7)):
            a, b = g[k].item(), r[k][0].item()
            if b == 0.0:
                assert a == 0.0, k
            else:
                assert_rel(a, b, tol, k)
    ctx.close()


def test_noalloc_fit_against_the_oracle_without_touching_device_memory():
    """The same entry point against the fp64 oracle (its fit searches the root with lgamma evaluations: no table,
    because a table would have to be allocated): both element types, a 4-byte aligned fp32 pointer that is not
    16-byte aligned, a shape clamped at either end, an all-zero and an empty segment.  After the first call the
    free device memory must not move: that is what the entry point is for."""
    import numpy as np
    import __graft_entry__ as entry
    entry.build()
    from oracle import gg_oracle as o
    from paper_2506_00486_b200 import binding
    L = binding.lib()
    rng = np.random.default_rng(78)
    spikes = np.zeros(3_000_000, dtype=np.float32)
    spikes[1234567] = 3.0                                 # one non-zero entry: ratio 1/n = 3.3e-7 < rho(0.05) = 4.1e-7, clamped low
    buf = torch.zeros(3 * TILE + 16, dtype=torch.float32, device="cuda:0")
    host_odd = gg_synth.gg_host(rng, 0.8, 0.05, 3 * TILE + 9, torch.float32)
    buf[3:3 + host_odd.numel()].copy_(host_odd)
    cases = [(gg_synth.gg_host(rng, 0.7, 0.02, 9 * TILE + 1234, torch.bfloat16), None),
             (gg_synth.gg_host(rng, 1.9, 0.3, 2 * TILE + 5, torch.float32), None),
             (host_odd, buf[3:3 + host_odd.numel()]),
             (torch.full((4000,), -2.5, dtype=torch.bfloat16), None),          # constant magnitude: ratio 1, clamped high
             (torch.from_numpy(spikes), None),
             (torch.zeros(100, dtype=torch.float32), None),
             (torch.zeros(0, dtype=torch.bfloat16), None)]
    xs = [(h, d if d is not None else h.to("cuda:0")) for h, d in cases]
    call_noalloc(L, xs[0][1])                            # first calls on the device (one per element type): they look the
    call_noalloc(L, xs[1][1])                            # array up and make the runtime load the kernels
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info(0)[0]
    outs = [torch.empty(1, dtype=dt, device="cuda:0") for dt in (torch.float64,) * 4 + (torch.int64, torch.int32)]
    torch.cuda.synchronize()
    free1 = torch.cuda.mem_get_info(0)[0]
    seen = set()
    for h, d in xs:
        p = ctypes.c_void_p
        st = L.gg_fit_noalloc(0, p(d.data_ptr()) if d.numel() else None, d.numel(), 0 if d.dtype == torch.float32 else 1,
                              *(p(t.data_ptr()) for t in outs), p(torch.cuda.current_stream().cuda_stream))
        assert st == 0
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(0)[0] == free1     # nothing was allocated by the call
        beta, alpha, s1, s2 = (t.item() for t in outs[:4])
        b, a, r1, r2, n, fl = o.fit(gg_synth.to_oracle(h))
        assert outs[4].item() == n == h.numel() and outs[5].item() == fl
        seen.add(fl)
        if fl & o.FLAG_DEGENERATE:
            assert beta == 0.0 and alpha == 0.0
            continue
        assert_rel(beta, b, REL_FIT, "beta")
        assert_rel(alpha, a, REL_FIT, "alpha")
        assert_rel(s1, r1, 1e-7, "sum_abs")
        assert_rel(s2, r2, 1e-7, "sum_sq")
    assert free1 <= free0
    assert {0, o.FLAG_DEGENERATE, o.FLAG_BETA_CLAMPED_LO, o.FLAG_BETA_CLAMPED_HI} <= seen


def test_noalloc_fit_refuses_segments_beyond_its_fixed_capacity():
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import binding
    L = binding.lib()
    cap = L.gg_fit_noalloc_max_len()
    assert cap == 16384 * 16384
    out = torch.zeros(2, dtype=torch.float64, device="cuda:0")
    x = torch.zeros(8, dtype=torch.float32, device="cuda:0")
    p = ctypes.c_void_p
    st = L.gg_fit_noalloc(0, p(x.data_ptr()), cap + 1, 0, p(out.data_ptr()), p(out.data_ptr() + 8),
                          None, None, None, None, None)
    assert st == 4 and b"scratch" in L.gg_status_str(st)      # GG_ERR_WORKSPACE, nothing enqueued
    assert L.gg_fit_noalloc(0, p(x.data_ptr()), -1, 0, p(out.data_ptr()), p(out.data_ptr() + 8),
                            None, None, None, None, None) == 1
