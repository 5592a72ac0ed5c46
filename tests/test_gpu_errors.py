"""Status codes of the context entry points: every malformed call is refused on the host, with the status the
interface documents, before anything is enqueued (the launch counter does not move and the outputs keep their
fill values)."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

OK, INVALID, DTYPE, ALIGN, WORKSPACE = 0, 1, 2, 3, 4
P = ctypes.c_void_p


@pytest.fixture(scope="module")
def env():
    import __graft_entry__ as entry
    entry.build()
    from paper_2506_00486_b200 import Context, binding
    c = Context(0)
    yield c, binding.lib()
    c.close()


def seg_array(entries):
    from paper_2506_00486_b200.binding import _SEG_DTYPE
    arr = np.zeros(len(entries), dtype=_SEG_DTYPE)
    for i, (ptr, n) in enumerate(entries):
        arr["ptr"][i], arr["len"][i] = ptr, n
    return arr


def refused(ctx, status, want):
    assert status == want, status


def test_fit_penalty_hist_and_sample_argument_errors(env):
    ctx, L = env
    x = torch.ones(4096, dtype=torch.float32, device="cuda:0")
    g = torch.full((4096,), 7.0, dtype=torch.float32, device="cuda:0")
    out = torch.full((8,), -3.0, dtype=torch.float64, device="cuda:0")
    step = torch.full((2,), 0.01, dtype=torch.float32, device="cuda:0")
    hist = torch.full((2 * 11,), 5, dtype=torch.int64, device="cuda:0")
    b, a = P(out.data_ptr()), P(out.data_ptr() + 16)
    segs = seg_array([(x.data_ptr(), 1000), (x.data_ptr() + 4000, 2000)])
    sp = segs.ctypes.data
    before = ctx.launch_count
    # element type
    refused(ctx, L.gg_fit(ctx._h, sp, 2, 7, b, a, None, None, None, None, None), DTYPE)
    gs = seg_array([(g.data_ptr(), 1000), (g.data_ptr() + 4000, 2000)])
    refused(ctx, L.gg_penalty_grad(ctx._h, sp, 2, 0, b, a, 1e-4, 0, gs.ctypes.data, 5, 0, None, None), DTYPE)
    # pointers that are not aligned to their element
    odd = seg_array([(x.data_ptr() + 2, 100)])
    refused(ctx, L.gg_fit(ctx._h, odd.ctypes.data, 1, 0, b, a, None, None, None, None, None), ALIGN)
    odd16 = seg_array([(x.data_ptr() + 1, 100)])
    refused(ctx, L.gg_fit(ctx._h, odd16.ctypes.data, 1, 1, b, a, None, None, None, None, None), ALIGN)
    godd = seg_array([(g.data_ptr() + 2, 1000), (g.data_ptr() + 4000, 2000)])
    refused(ctx, L.gg_penalty_grad(ctx._h, sp, 2, 0, b, a, 1e-4, 0, godd.ctypes.data, 0, 0, None, None), ALIGN)
    # a gradient segment of another length, a null pointer with a length, a negative length, an unknown reduction
    gbad = seg_array([(g.data_ptr(), 999), (g.data_ptr() + 4000, 2000)])
    refused(ctx, L.gg_penalty_grad(ctx._h, sp, 2, 0, b, a, 1e-4, 0, gbad.ctypes.data, 0, 0, None, None), INVALID)
    refused(ctx, L.gg_fit(ctx._h, seg_array([(0, 5)]).ctypes.data, 1, 0, b, a, None, None, None, None, None), INVALID)
    refused(ctx, L.gg_fit(ctx._h, seg_array([(x.data_ptr(), -1)]).ctypes.data, 1, 0, b, a, None, None, None, None, None), INVALID)
    refused(ctx, L.gg_penalty_grad(ctx._h, sp, 2, 0, b, a, 1e-4, 3, None, 0, 0, None, None), INVALID)
    refused(ctx, L.gg_fit(ctx._h, sp, 2, 0, None, a, None, None, None, None, None), INVALID)
    # histogram ids out of range, an empty symbol range, ids missing when the counts differ
    hp, stp = P(hist.data_ptr()), P(step.data_ptr())
    ids = np.array([0, 2], dtype=np.int32)
    refused(ctx, L.gg_rate_hist(ctx._h, sp, 2, 0, stp, ids.ctypes.data, 2, -5, 5, hp, 0, None, None, None), INVALID)
    ids = np.array([0, -1], dtype=np.int32)
    refused(ctx, L.gg_rate_hist(ctx._h, sp, 2, 0, stp, ids.ctypes.data, 2, -5, 5, hp, 0, None, None, None), INVALID)
    refused(ctx, L.gg_rate_hist(ctx._h, sp, 2, 0, stp, None, 2, 5, 4, hp, 0, None, None, None), INVALID)
    refused(ctx, L.gg_rate_hist(ctx._h, sp, 2, 0, stp, None, 1, -5, 5, hp, 0, None, None, None), INVALID)
    refused(ctx, L.gg_rate_hist(ctx._h, sp, 2, 0, stp, None, 2, -(1 << 24), 1 << 24, hp, 0, None, None, None), INVALID)
    # more tiles than a plan can index: four segments of 2^44 elements (nothing is read: the check comes first)
    huge = seg_array([(x.data_ptr(), 1 << 44)] * 4)
    refused(ctx, L.gg_fit(ctx._h, huge.ctypes.data, 4, 1, b, a, None, None, None, None, None), WORKSPACE)
    # sampler parameters
    beta = np.array([1.0, 0.0]); alpha = np.array([1.0, 1.0])
    refused(ctx, L.gg_sample(ctx._h, sp, 2, 0, beta.ctypes.data, alpha.ctypes.data, 1, 0, None, None), INVALID)
    beta = np.array([1.0, 1.0]); alpha = np.array([1.0, float("inf")])
    refused(ctx, L.gg_sample(ctx._h, sp, 2, 0, beta.ctypes.data, alpha.ctypes.data, 1, 0, None, None), INVALID)
    torch.cuda.synchronize()
    assert ctx.launch_count == before
    assert bool((out == -3.0).all()) and bool((g == 7.0).all()) and bool((hist == 5).all()) and bool((x == 1.0).all())


def test_fused_and_channel_argument_errors(env):
    ctx, L = env
    from paper_2506_00486_b200 import Segments
    from paper_2506_00486_b200.binding import ChannelArgs
    x = torch.ones(8192, dtype=torch.bfloat16, device="cuda:0")
    g = torch.full((8192,), 7.0, dtype=torch.float32, device="cuda:0")
    step = torch.full((2,), 0.01, dtype=torch.float32, device="cuda:0")
    segs = Segments.slices(x, [0, 4096], [4096, 4000])
    gsegs = Segments.slices(g, [0, 4096], [4096, 4000])
    before = ctx.launch_count

    def status(**change):
        run = ctx.make_fused(segs, grad=gsegs, lam=1e-4, step=step)
        for k, v in change.items():
            setattr(run.args, k, v)
        return L.gg_fused(ctx._h, ctypes.byref(run.args), None), run

    assert status(in_dtype=9)[0] == DTYPE
    assert status(grad_dtype=9)[0] == DTYPE
    assert status(param_mode=5)[0] == INVALID
    assert status(param_mode=1)[0] == INVALID            # given parameters without beta_in / alpha_in
    assert status(reduction=2)[0] == INVALID
    assert status(step_mode=1)[0] == INVALID             # step from alpha without step_out
    assert status(step=None)[0] == INVALID
    assert status(qmin=10, qmax=9)[0] == INVALID
    assert status(n_hist=3)[0] == INVALID                # no ids: one histogram per segment is required
    assert status(beta=None)[0] == INVALID
    ids = np.array([0, 5], dtype=np.int32)
    assert status(hist_id=ids.ctypes.data)[0] == INVALID
    short = Segments.slices(g, [0, 4096], [4096, 3999])
    assert status(grad=short.ptr)[0] == INVALID
    odd = Segments.slices(x, [1, 4096], [4000, 4000])
    odd.array["ptr"][0] += 1                              # one byte past an element boundary
    assert status(segs=odd.ptr)[0] == ALIGN
    # the channel-wise pass
    m = torch.ones((64, 96), dtype=torch.bfloat16, device="cuda:0")
    run = ctx.make_fused_channels(m, lam=1e-4, step=0.01)

    def chan(**change):
        a = ChannelArgs()
        ctypes.memmove(ctypes.byref(a), ctypes.byref(run.args), ctypes.sizeof(a))
        for k, v in change.items():
            setattr(a, k, v)
        return L.gg_fused_channels(ctx._h, ctypes.byref(a), None)

    assert chan(in_dtype=4) == DTYPE
    assert chan(ld=95) == INVALID
    assert chan(rows=-1) == INVALID
    assert chan(step=0.0) == INVALID
    assert chan(step=float("inf")) == INVALID
    assert chan(qmin=3, qmax=2) == INVALID
    assert chan(x=m.data_ptr() + 1) == ALIGN
    assert chan(rows=65536 * 512) == WORKSPACE
    torch.cuda.synchronize()
    assert ctx.launch_count == before
    assert bool((g == 7.0).all())
