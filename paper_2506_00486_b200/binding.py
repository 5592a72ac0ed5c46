"""ctypes binding of libgg_b200.so: argument marshalling only.

Every step of the pass runs in the CUDA library; this module turns torch tensors into the
pointers and sizes of the C interface (include/gg.h) and allocates output tensors.  There is
no CPU fallback: if the library is missing or the device is not a B200-class GPU the calls raise.
"""
import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# GG_B200_LIB selects another build of the same library (the bounds-checking one of build.py --bounds)
_LIB_PATH = os.environ.get("GG_B200_LIB") or os.path.join(_HERE, "libgg_b200.so")

GG_F32, GG_BF16 = 0, 1
GG_SUM, GG_MEAN = 0, 1
GG_PARAMS_FITTED, GG_PARAMS_GIVEN, GG_RATE_EG = 0, 1, 2
GG_STEP_GIVEN, GG_STEP_FROM_ALPHA = 0, 1
FLAG_DEGENERATE, FLAG_BETA_CLAMPED_LO, FLAG_BETA_CLAMPED_HI, FLAG_NONFINITE, FLAG_CLAMPED_SYMBOLS = 1, 2, 4, 8, 16
FLAG_TIMEOUT = 32
HOOK_RESIDENT_MODE, HOOK_EXTRA_ARRIVALS, HOOK_WAIT_CAP, HOOK_CLUSTER_MODE = 0, 1, 2, 3
BETA_LO, BETA_HI = 0.05, 20.0

_SEG_DTYPE = np.dtype([("ptr", np.uint64), ("len", np.int64)])
_P = ctypes.c_void_p


class FusedArgs(ctypes.Structure):
    """Mirror of gg_fused_args."""
    _fields_ = [
        ("segs", _P), ("n_seg", ctypes.c_int32), ("in_dtype", ctypes.c_int32),
        ("beta", _P), ("alpha", _P), ("sum_abs", _P), ("sum_sq", _P), ("count", _P), ("flags", _P),
        ("param_mode", ctypes.c_int32), ("beta_in", _P), ("alpha_in", _P),
        ("lam", ctypes.c_double), ("reduction", ctypes.c_int32),
        ("grad", _P), ("grad_dtype", ctypes.c_int32), ("accumulate_grad", ctypes.c_int32),
        ("penalty", _P),
        ("step_mode", ctypes.c_int32), ("step", _P), ("step_scale", ctypes.c_double), ("step_out", _P),
        ("hist_id", _P), ("n_hist", ctypes.c_int32), ("qmin", ctypes.c_int32), ("qmax", ctypes.c_int32),
        ("hist", _P), ("accumulate_hist", ctypes.c_int32), ("entropy_bits", _P), ("clamped_lo_hi", _P),
        ("eg_k", ctypes.c_int32), ("eg_bits", _P),
    ]


class ChannelArgs(ctypes.Structure):
    """Mirror of gg_channel_args."""
    _fields_ = [
        ("x", _P), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("ld", ctypes.c_int64),
        ("in_dtype", ctypes.c_int32),
        ("beta", _P), ("alpha", _P), ("sum_abs", _P), ("sum_sq", _P), ("count", _P), ("flags", _P),
        ("lam", ctypes.c_double), ("reduction", ctypes.c_int32),
        ("grad", _P), ("grad_ld", ctypes.c_int64), ("grad_dtype", ctypes.c_int32),
        ("accumulate_grad", ctypes.c_int32), ("penalty", _P),
        ("step", ctypes.c_float), ("qmin", ctypes.c_int32), ("qmax", ctypes.c_int32),
        ("hist", _P), ("accumulate_hist", ctypes.c_int32), ("entropy_bits", _P), ("clamped_lo_hi", _P),
    ]


class GGError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"gg status {status}: {text}")
        self.status = status


_lib = None


def lib():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run paper_2506_00486_b200/build.py "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        i32, i64, u32, u64, d = (ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_uint64,
                                 ctypes.c_double)
        L.gg_create.argtypes = [ctypes.POINTER(_P), ctypes.c_int]
        L.gg_destroy.argtypes = [_P]
        L.gg_status_str.argtypes = [ctypes.c_int]
        L.gg_status_str.restype = ctypes.c_char_p
        L.gg_version.restype = ctypes.c_int
        L.gg_last_cuda_error.argtypes = [_P]
        L.gg_last_cuda_error.restype = ctypes.c_char_p
        L.gg_launch_count.argtypes = [_P]
        L.gg_launch_count.restype = i64
        L.gg_plan_stats.argtypes = [_P, i32]
        L.gg_plan_stats.restype = i64
        for name, args in (("gg_alpha_from_std", [d, d]), ("gg_init_alpha", [i64, d, d]),
                           ("gg_diff_entropy_bits", [d, d])):
            getattr(L, name).argtypes = args
            getattr(L, name).restype = d
        L.gg_fit.argtypes = [_P, _P, i32, ctypes.c_int, _P, _P, _P, _P, _P, _P, _P]
        L.gg_penalty_grad.argtypes = [_P, _P, i32, ctypes.c_int, _P, _P, d, ctypes.c_int, _P,
                                      ctypes.c_int, ctypes.c_int, _P, _P]
        L.gg_rate_hist.argtypes = [_P, _P, i32, ctypes.c_int, _P, _P, i32, i32, i32, _P, ctypes.c_int,
                                   _P, _P, _P]
        L.gg_sample.argtypes = [_P, _P, i32, ctypes.c_int, _P, _P, u64, u32, _P, _P]
        L.gg_fused.argtypes = [_P, ctypes.POINTER(FusedArgs), _P]
        L.gg_fused_host.argtypes = [_P, ctypes.POINTER(FusedArgs), i64]
        L.gg_fused_channels.argtypes = [_P, ctypes.POINTER(ChannelArgs), _P]
        L.gg_fused_channels.restype = ctypes.c_int
        L.gg_timing_enable.argtypes = [_P, ctypes.c_int]
        L.gg_timing_read.argtypes = [_P, ctypes.POINTER(d), ctypes.POINTER(i64), ctypes.POINTER(d),
                                     ctypes.POINTER(i64)]
        L.gg_debug_bounds_violations.restype = i64
        L.gg_test_hook.argtypes = [_P, i32, i64]
        L.gg_test_hook.restype = ctypes.c_int
        L.gg_fit_noalloc.argtypes = [ctypes.c_int, _P, i64, ctypes.c_int, _P, _P, _P, _P, _P, _P, _P]
        L.gg_fit_noalloc.restype = ctypes.c_int
        L.gg_fit_noalloc_max_len.restype = i64
        L.gg_eg_rate.argtypes = [_P, _P, i32, i32, i32, i32, _P, _P]
        L.gg_eg_rate_grad.argtypes = [_P, _P, i32, ctypes.c_int, _P, i32, d, i32, i32, _P, ctypes.c_int, ctypes.c_int, _P]
        L.gg_code_stats.argtypes = [_P, _P, i32, i32, i32, i32, _P, _P, _P, _P]
        L.gg_gct_step.argtypes = [_P, _P, i32, ctypes.c_int, _P, _P, _P, i32, i32, i32, d, d, d, i64, _P]
        L.gg_compression_ratio.argtypes = [d, d]
        L.gg_compression_ratio.restype = d
        for name in ("gg_eg_rate", "gg_eg_rate_grad", "gg_code_stats", "gg_gct_step"):
            getattr(L, name).restype = ctypes.c_int
        for name in ("gg_create", "gg_destroy", "gg_fit", "gg_penalty_grad", "gg_rate_hist", "gg_sample",
                     "gg_fused", "gg_fused_host", "gg_timing_enable", "gg_timing_read"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def gg_alpha_from_std(std, beta):
    return lib().gg_alpha_from_std(float(std), float(beta))


def gg_init_alpha(d_in, xi, beta):
    return lib().gg_init_alpha(int(d_in), float(xi), float(beta))


def gg_diff_entropy_bits(alpha, beta):
    return lib().gg_diff_entropy_bits(float(alpha), float(beta))


def gg_fit_noalloc(x, out=None):
    """Moments and fit of one contiguous CUDA tensor through the entry point that allocates nothing.

    For callers that cannot allocate device memory at the time of the call, `out` carries the six
    one-element device tensors (beta, alpha, sum_abs, sum_sq: float64; count: int64; flags: int32)
    prepared beforehand; without it they are created here with torch (which does allocate)."""
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("need a contiguous CUDA tensor")
    dev = x.device
    if out is None:
        out = dict(beta=torch.empty(1, dtype=torch.float64, device=dev), alpha=torch.empty(1, dtype=torch.float64, device=dev),
                   sum_abs=torch.empty(1, dtype=torch.float64, device=dev), sum_sq=torch.empty(1, dtype=torch.float64, device=dev),
                   count=torch.empty(1, dtype=torch.int64, device=dev), flags=torch.empty(1, dtype=torch.int32, device=dev))
    status = lib().gg_fit_noalloc(dev.index or 0, x.data_ptr() if x.numel() else None, x.numel(), _dtype_code(x.dtype),
                                  _ptr(out["beta"]), _ptr(out["alpha"]), _ptr(out["sum_abs"]), _ptr(out["sum_sq"]),
                                  _ptr(out["count"]), _ptr(out["flags"]), _stream_ptr(dev))
    if status != 0:
        raise GGError(status, lib().gg_status_str(status).decode())
    return out


def gg_compression_ratio(bits, fixed_length_bits):
    return lib().gg_compression_ratio(float(bits), float(fixed_length_bits))


def _dtype_code(dt):
    if dt == torch.float32:
        return GG_F32
    if dt == torch.bfloat16:
        return GG_BF16
    raise TypeError(f"unsupported dtype {dt}: the library takes float32 and bfloat16")


class Segments:
    """A host array of gg_seg built once from tensors (kept alive here).

    `Segments(list_of_tensors)`: one segment per tensor (flattened, must be contiguous).
    `Segments.rows(t)`: one segment per row of a contiguous 2-D tensor."""

    def __init__(self, tensors):
        tensors = list(tensors)
        self.tensors = tensors
        self.dtype = tensors[0].dtype if tensors else torch.float32
        arr = np.zeros(len(tensors), dtype=_SEG_DTYPE)
        for i, t in enumerate(tensors):
            if t.dtype != self.dtype:
                raise TypeError("all segments of one call share a dtype")
            if not t.is_contiguous():
                raise ValueError("segments must be contiguous")
            arr["ptr"][i] = t.data_ptr() if t.numel() else 0
            arr["len"][i] = t.numel()
        self.array = arr

    @classmethod
    def rows(cls, t):
        if t.dim() != 2 or not t.is_contiguous():
            raise ValueError("need a contiguous 2-D tensor")
        self = cls.__new__(cls)
        self.tensors = [t]
        self.dtype = t.dtype
        arr = np.zeros(t.shape[0], dtype=_SEG_DTYPE)
        row_bytes = t.shape[1] * t.element_size()
        arr["ptr"] = t.data_ptr() + np.arange(t.shape[0], dtype=np.uint64) * np.uint64(row_bytes)
        arr["len"] = t.shape[1]
        self.array = arr
        return self

    @classmethod
    def slices(cls, flat, offsets, lens):
        """Segments flat[offsets[i] : offsets[i] + lens[i]] of one flat tensor."""
        self = cls.__new__(cls)
        self.tensors = [flat]
        self.dtype = flat.dtype
        arr = np.zeros(len(lens), dtype=_SEG_DTYPE)
        arr["ptr"] = flat.data_ptr() + np.asarray(offsets, dtype=np.uint64) * np.uint64(flat.element_size())
        arr["len"] = np.asarray(lens, dtype=np.int64)
        self.array = arr
        return self

    def __len__(self):
        return len(self.array)

    @property
    def lens(self):
        return self.array["len"]

    @property
    def ptr(self):
        return self.array.ctypes.data

    @property
    def code(self):
        return _dtype_code(self.dtype)

    def device(self):
        return self.tensors[0].device


def _as_segments(x):
    return x if isinstance(x, Segments) else Segments(x)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream_ptr(device):
    return torch.cuda.current_stream(device).cuda_stream


class Context:
    """One gg_ctx on one CUDA device.  Use from one stream at a time."""

    GUARD_BYTES, GUARD_FILL = 256, 0xA5

    def __init__(self, device=0, guard=False):
        """guard=True puts 256 bytes of a fill pattern before and after every output tensor this object allocates
        (fit results, penalties, histograms, entropies, counters); check_guards() then tells whether a kernel
        wrote outside an output."""
        self._guard = bool(guard)
        self._guarded = []
        self.device = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
        if self.device.type != "cuda":
            raise RuntimeError("the GG library runs on CUDA devices only")
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the GG library has no CPU fallback")
        torch.cuda.init()
        with torch.cuda.device(self.device):
            torch.empty(1, device=self.device)          # make sure the primary context exists
        h = _P()
        self._check(lib().gg_create(ctypes.byref(h), self.device.index or 0), None)
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().gg_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, status, h=True):
        if status != 0:
            text = lib().gg_status_str(status).decode()
            if status == 6 and h and getattr(self, "_h", None):
                text += ": " + lib().gg_last_cuda_error(self._h).decode()
            raise GGError(status, text)

    @property
    def launch_count(self):
        return lib().gg_launch_count(self._h)

    @property
    def plan_stats(self):
        """(plans built, plans pointed at other addresses) since the context was created."""
        return lib().gg_plan_stats(self._h, 0), lib().gg_plan_stats(self._h, 1)

    def gg_test_hook(self, what, value):
        """Knobs of the one-launch fitted pass (HOOK_*), for tests and measurements."""
        self._check(lib().gg_test_hook(self._h, int(what), int(value)))

    def _new(self, n, dtype, zero=False):
        shape = (n,) if isinstance(n, int) else tuple(n)
        if not self._guard:
            return (torch.zeros if zero else torch.empty)(shape, dtype=dtype, device=self.device)
        import weakref
        nbytes = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        pad = self.GUARD_BYTES
        raw = torch.full((nbytes + 2 * pad,), self.GUARD_FILL, dtype=torch.uint8, device=self.device)
        body = raw[pad:pad + nbytes]
        if zero:
            body.zero_()
        out = body.view(dtype).view(shape)
        self._guarded.append((weakref.ref(out), raw, nbytes))
        return out

    def check_guards(self):
        """Raises if any byte around a live guarded output has changed (after waiting for the device)."""
        torch.cuda.synchronize(self.device)
        pad, keep = self.GUARD_BYTES, []
        for ref, raw, nbytes in self._guarded:
            if ref() is None:
                continue
            keep.append((ref, raw, nbytes))
            ok = bool((raw[:pad] == self.GUARD_FILL).all()) and bool((raw[pad + nbytes:] == self.GUARD_FILL).all())
            if not ok:
                raise AssertionError(f"a kernel wrote outside an output of {nbytes} bytes")
        self._guarded = keep

    # ------------------------------------------------------------------ gg_fit
    def gg_fit(self, segs):
        """Moments and fit per segment.  Returns a dict of device tensors."""
        segs = _as_segments(segs)
        n = len(segs)
        out = dict(beta=self._new(n, torch.float64), alpha=self._new(n, torch.float64),
                   sum_abs=self._new(n, torch.float64), sum_sq=self._new(n, torch.float64),
                   count=self._new(n, torch.int64), flags=self._new(n, torch.int32))
        self._check(lib().gg_fit(self._h, segs.ptr, n, segs.code, _ptr(out["beta"]), _ptr(out["alpha"]),
                                 _ptr(out["sum_abs"]), _ptr(out["sum_sq"]), _ptr(out["count"]),
                                 _ptr(out["flags"]), _stream_ptr(self.device)))
        return out

    # -------------------------------------------------------- gg_penalty_grad
    def gg_penalty_grad(self, segs, beta, alpha, lam, grad=None, reduction=GG_SUM, accumulate=False,
                        want_penalty=True):
        """Penalty per segment (device float64) and the gradient written into `grad` segments."""
        segs = _as_segments(segs)
        n = len(segs)
        gsegs = None if grad is None else _as_segments(grad)
        pen = self._new(n, torch.float64) if want_penalty else None
        self._check(lib().gg_penalty_grad(
            self._h, segs.ptr, n, segs.code, _ptr(beta), _ptr(alpha), float(lam), int(reduction),
            None if gsegs is None else gsegs.ptr, GG_F32 if gsegs is None else gsegs.code,
            int(bool(accumulate)), _ptr(pen), _stream_ptr(self.device)))
        return pen

    # ------------------------------------------------------------ gg_rate_hist
    def gg_rate_hist(self, segs, step, hist_id=None, n_hist=None, qmin=-32768, qmax=32767, hist=None,
                     accumulate=False):
        """Histogram(s) of the quantised symbols, entropy in bits/symbol, clamp counters."""
        segs = _as_segments(segs)
        n = len(segs)
        n_hist = n if n_hist is None else int(n_hist)
        nb = qmax - qmin + 1
        if hist is None:
            hist = self._new((n_hist, nb), torch.int64)
            if accumulate:
                hist.zero_()
        ent = self._new(n_hist, torch.float64)
        clamped = self._new((n_hist, 2), torch.int64, zero=True)
        hid = None if hist_id is None else np.ascontiguousarray(hist_id, dtype=np.int32)
        self._check(lib().gg_rate_hist(
            self._h, segs.ptr, n, segs.code, _ptr(step), None if hid is None else hid.ctypes.data,
            n_hist, int(qmin), int(qmax), _ptr(hist), int(bool(accumulate)), _ptr(ent), _ptr(clamped),
            _stream_ptr(self.device)))
        return dict(hist=hist, entropy_bits=ent, clamped=clamped)

    # --------------------------------------------------------------- gg_sample
    def gg_sample(self, out, beta, alpha, seed, tensor_id0=0, want_attempts=True):
        """Fills the `out` segments with GG variates; beta, alpha are host sequences."""
        segs = _as_segments(out)
        n = len(segs)
        b = np.ascontiguousarray(beta, dtype=np.float64)
        a = np.ascontiguousarray(alpha, dtype=np.float64)
        if b.size != n or a.size != n:
            raise ValueError("beta and alpha need one entry per segment")
        att = self._new(n, torch.int32) if want_attempts else None
        self._check(lib().gg_sample(self._h, segs.ptr, n, segs.code, b.ctypes.data, a.ctypes.data,
                                    int(seed) & (2 ** 64 - 1), int(tensor_id0) & 0xFFFFFFFF, _ptr(att),
                                    _stream_ptr(self.device)))
        return att

    # ---------------------------------------------------------------- gg_fused
    def make_fused(self, segs, grad=None, lam=1e-4, reduction=GG_SUM, accumulate_grad=False,
                   param_mode=GG_PARAMS_FITTED, beta_in=None, alpha_in=None, want_penalty=True,
                   step=None, step_scale=None, hist_id=None, n_hist=None, qmin=-32768, qmax=32767,
                   want_hist=True, accumulate_hist=False, hist=None, eg_k=0):
        """Allocates the outputs of the fused pass once and returns a callable that enqueues it.

        step: device float32 tensor [n_seg] (GG_STEP_GIVEN); or step_scale: float, step = alpha * scale.
        param_mode=GG_RATE_EG: the gradient and penalty of the Exponential-Golomb rate of order eg_k (Eq. 6-7)
        instead of the GG penalty; out["eg_bits"] holds the mean code length per histogram."""
        segs = _as_segments(segs)
        n = len(segs)
        gsegs = None if grad is None else _as_segments(grad)
        out = dict(beta=self._new(n, torch.float64), alpha=self._new(n, torch.float64),
                   sum_abs=self._new(n, torch.float64), sum_sq=self._new(n, torch.float64),
                   count=self._new(n, torch.int64), flags=self._new(n, torch.int32))
        out["penalty"] = self._new(n, torch.float64) if want_penalty else None
        a = FusedArgs()
        keep = [segs, gsegs, beta_in, alpha_in, step]
        a.segs, a.n_seg, a.in_dtype = segs.ptr, n, segs.code
        for k in ("beta", "alpha", "sum_abs", "sum_sq", "count", "flags", "penalty"):
            setattr(a, k, _ptr(out[k]))
        a.param_mode = int(param_mode)
        a.beta_in, a.alpha_in = _ptr(beta_in), _ptr(alpha_in)
        a.lam, a.reduction = float(lam), int(reduction)
        a.grad = None if gsegs is None else gsegs.ptr
        a.grad_dtype = GG_F32 if gsegs is None else gsegs.code
        a.accumulate_grad = int(bool(accumulate_grad))
        if want_hist:
            n_hist = n if n_hist is None else int(n_hist)
            nb = qmax - qmin + 1
            if hist is None:
                hist = self._new((n_hist, nb), torch.int64, zero=True)
            out["hist"] = hist
            out["entropy_bits"] = self._new(n_hist, torch.float64)
            out["clamped"] = self._new((n_hist, 2), torch.int64, zero=True)
            if step is not None:
                a.step_mode, a.step = GG_STEP_GIVEN, _ptr(step)
                out["step"] = step
            else:
                out["step"] = self._new(n, torch.float32)
                a.step_mode, a.step_scale, a.step_out = GG_STEP_FROM_ALPHA, float(step_scale), _ptr(out["step"])
            hid = None if hist_id is None else np.ascontiguousarray(hist_id, dtype=np.int32)
            keep.append(hid)
            a.hist_id = None if hid is None else hid.ctypes.data
            a.n_hist, a.qmin, a.qmax = n_hist, int(qmin), int(qmax)
            a.hist, a.accumulate_hist = _ptr(hist), int(bool(accumulate_hist))
            a.entropy_bits, a.clamped_lo_hi = _ptr(out["entropy_bits"]), _ptr(out["clamped"])
            if int(param_mode) == GG_RATE_EG:
                out["eg_bits"] = self._new(n_hist, torch.float64)
                a.eg_k, a.eg_bits = int(eg_k), _ptr(out["eg_bits"])

        def run():
            self._check(lib().gg_fused(self._h, ctypes.byref(a), _stream_ptr(self.device)))
            return out

        run.outputs = out
        run.args = a
        run._keep = keep
        return run

    def gg_fused(self, segs, **kw):
        """One-shot form of make_fused(...)()."""
        return self.make_fused(segs, **kw)()

    # ------------------------------------------------------- gg_fused_channels
    def make_fused_channels(self, x, grad=None, lam=1e-4, reduction=GG_SUM, accumulate_grad=False,
                            want_penalty=True, step=None, qmin=-32768, qmax=32767, accumulate_hist=False,
                            hist=None):
        """The fused pass over the COLUMNS of the 2-D tensor x (rows may be strided: x.stride(1) == 1).

        Allocates the per-column outputs once and returns a callable that enqueues the pass.
        step: float, one quantiser step for the matrix; None skips the histogram."""
        if x.dim() != 2 or (x.shape[1] > 1 and x.stride(1) != 1):
            raise ValueError("x must be 2-D with contiguous rows")
        rows, cols = x.shape
        out = dict(beta=self._new(cols, torch.float64), alpha=self._new(cols, torch.float64),
                   sum_abs=self._new(cols, torch.float64), sum_sq=self._new(cols, torch.float64),
                   count=self._new(cols, torch.int64), flags=self._new(cols, torch.int32))
        out["penalty"] = self._new(cols, torch.float64) if want_penalty else None
        a = ChannelArgs()
        a.x, a.rows, a.cols, a.ld, a.in_dtype = _ptr(x), rows, cols, (x.stride(0) if rows > 1 else cols), _dtype_code(x.dtype)
        for k in ("beta", "alpha", "sum_abs", "sum_sq", "count", "flags", "penalty"):
            setattr(a, k, _ptr(out[k]))
        a.lam, a.reduction = float(lam), int(reduction)
        if grad is not None:
            if grad.shape != x.shape or (cols > 1 and grad.stride(1) != 1):
                raise ValueError("grad must have the shape of x and contiguous rows")
            a.grad, a.grad_ld, a.grad_dtype = _ptr(grad), (grad.stride(0) if rows > 1 else cols), _dtype_code(grad.dtype)
        a.accumulate_grad = int(bool(accumulate_grad))
        if step is not None:
            nb = qmax - qmin + 1
            if hist is None:
                hist = self._new(nb, torch.int64, zero=True)
            out["hist"] = hist
            out["entropy_bits"] = self._new(1, torch.float64)
            out["clamped"] = self._new(2, torch.int64, zero=True)
            a.step, a.qmin, a.qmax = float(step), int(qmin), int(qmax)
            a.hist, a.accumulate_hist = _ptr(hist), int(bool(accumulate_hist))
            a.entropy_bits, a.clamped_lo_hi = _ptr(out["entropy_bits"]), _ptr(out["clamped"])

        def run():
            self._check(lib().gg_fused_channels(self._h, ctypes.byref(a), _stream_ptr(self.device)))
            return out

        run.outputs = out
        run.args = a
        run._keep = [x, grad, hist]
        return run

    def gg_fused_channels(self, x, **kw):
        """One-shot form of make_fused_channels(...)()."""
        return self.make_fused_channels(x, **kw)()

    # ----------------------------------------------------------- gg_fused_host
    def make_fused_host(self, segs, grad=None, lam=1e-4, reduction=GG_SUM, step=None, step_scale=None,
                        hist_id=None, n_hist=None, qmin=-32768, qmax=32767, want_hist=True,
                        chunk_bytes=0, pin=True):
        """The fused pass on HOST tensors (CPU torch tensors; pinned ones copy asynchronously).

        Allocates the host outputs once (pinned if `pin`) and returns a callable; each call copies
        the inputs to the device in chunks, runs the pass and returns with all results on the host."""
        segs = _as_segments(segs)
        n = len(segs)
        gsegs = None if grad is None else _as_segments(grad)

        def host(n_, dtype):
            return torch.empty(n_, dtype=dtype, pin_memory=pin)

        out = dict(beta=host(n, torch.float64), alpha=host(n, torch.float64), sum_abs=host(n, torch.float64),
                   sum_sq=host(n, torch.float64), count=host(n, torch.int64), flags=host(n, torch.int32),
                   penalty=host(n, torch.float64))
        a = FusedArgs()
        keep = [segs, gsegs, step]
        a.segs, a.n_seg, a.in_dtype = segs.ptr, n, segs.code
        for k in ("beta", "alpha", "sum_abs", "sum_sq", "count", "flags", "penalty"):
            setattr(a, k, _ptr(out[k]))
        a.param_mode, a.lam, a.reduction = GG_PARAMS_FITTED, float(lam), int(reduction)
        a.grad = None if gsegs is None else gsegs.ptr
        a.grad_dtype = GG_F32 if gsegs is None else gsegs.code
        if want_hist:
            n_hist = n if n_hist is None else int(n_hist)
            nb = qmax - qmin + 1
            out["hist"] = torch.empty((n_hist, nb), dtype=torch.int64, pin_memory=pin)
            out["entropy_bits"] = host(n_hist, torch.float64)
            out["clamped"] = torch.empty((n_hist, 2), dtype=torch.int64, pin_memory=pin)
            if step is not None:
                a.step_mode, a.step = GG_STEP_GIVEN, _ptr(step)
                out["step"] = step
            else:
                out["step"] = host(n, torch.float32)
                a.step_mode, a.step_scale, a.step_out = GG_STEP_FROM_ALPHA, float(step_scale), _ptr(out["step"])
            hid = None if hist_id is None else np.ascontiguousarray(hist_id, dtype=np.int32)
            keep.append(hid)
            a.hist_id = None if hid is None else hid.ctypes.data
            a.n_hist, a.qmin, a.qmax = n_hist, int(qmin), int(qmax)
            a.hist, a.entropy_bits, a.clamped_lo_hi = _ptr(out["hist"]), _ptr(out["entropy_bits"]), _ptr(out["clamped"])

        def run():
            self._check(lib().gg_fused_host(self._h, ctypes.byref(a), int(chunk_bytes)))
            return out

        run.outputs = out
        run._keep = keep
        return run

    def gg_fused_host(self, segs, **kw):
        return self.make_fused_host(segs, **kw)()

    # ------------------------------------------------------------ code lengths
    def gg_eg_rate(self, hist, k=0, qmin=-32768, qmax=32767):
        """Average Exponential-Golomb code length per histogram (device float64)."""
        n_hist = hist.shape[0]
        out = self._new(n_hist, torch.float64)
        self._check(lib().gg_eg_rate(self._h, _ptr(hist), n_hist, int(qmin), int(qmax), int(k), _ptr(out),
                                     _stream_ptr(self.device)))
        return out

    def gg_eg_rate_grad(self, segs, step, lam, grad, k=0, qmin=-32768, qmax=32767, accumulate=False):
        """Writes the gradient of lam * (Exponential-Golomb rate) into the `grad` segments."""
        segs, gsegs = _as_segments(segs), _as_segments(grad)
        self._check(lib().gg_eg_rate_grad(self._h, segs.ptr, len(segs), segs.code, _ptr(step), int(k), float(lam),
                                          int(qmin), int(qmax), gsegs.ptr, gsegs.code, int(bool(accumulate)),
                                          _stream_ptr(self.device)))

    def gg_code_stats(self, hist, k=0, qmin=-32768, qmax=32767):
        """EG, Huffman and fixed-length bits per histogram as numpy arrays (synchronises the stream)."""
        n_hist = hist.shape[0]
        eg, hm, fl = (np.empty(n_hist, dtype=np.float64) for _ in range(3))
        self._check(lib().gg_code_stats(self._h, _ptr(hist), n_hist, int(qmin), int(qmax), int(k), eg.ctypes.data,
                                        hm.ctypes.data, fl.ctypes.data, _stream_ptr(self.device)))
        return dict(eg_bits=eg, hm_bits=hm, fl_bits=fl)

    def gg_gct_step(self, g, ghat, w, step, eta, lam, eps, t, k=0, qmin=-32768, qmax=32767):
        """One GCT step in place: `ghat` (float32 segments) and `w` (float32 segments) are updated."""
        gs, hs, ws = _as_segments(g), _as_segments(ghat), _as_segments(w)
        if hs.dtype != torch.float32 or ws.dtype != torch.float32:
            raise TypeError("ghat and w are float32")
        self._check(lib().gg_gct_step(self._h, gs.ptr, len(gs), gs.code, hs.ptr, ws.ptr, _ptr(step), int(k), int(qmin),
                                      int(qmax), float(eta), float(lam), float(eps), int(t), _stream_ptr(self.device)))

    # ------------------------------------------------------------------ timing
    def timing_enable(self, on=True):
        self._check(lib().gg_timing_enable(self._h, int(bool(on))))

    def timing_read(self):
        """(ms of first sweeps, their count, ms of second sweeps, their count) since the last read."""
        m0, m1 = ctypes.c_double(), ctypes.c_double()
        n0, n1 = ctypes.c_int64(), ctypes.c_int64()
        self._check(lib().gg_timing_read(self._h, ctypes.byref(m0), ctypes.byref(n0), ctypes.byref(m1),
                                         ctypes.byref(n1)))
        return m0.value, n0.value, m1.value, n1.value
