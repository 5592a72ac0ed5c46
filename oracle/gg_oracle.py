"""ctypes front end of the fp64 CPU oracle (oracle/gg_oracle.c).

TEST INFRASTRUCTURE: marshals numpy arrays into the C functions and adds the
few whole-tensor loops (per-segment calls) that the tests need.  No arithmetic
of the method lives here except rounding an fp64 value to bf16 / fp32 storage.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gg_oracle.c")
_LIB = os.path.join(_HERE, "libgg_oracle.so")

FLAG_DEGENERATE = 1
FLAG_BETA_CLAMPED_LO = 2
FLAG_BETA_CLAMPED_HI = 4
FLAG_NONFINITE = 8
BETA_LO = 0.05
BETA_HI = 20.0
SAMPLE_MAX_ATTEMPTS = 64


def build(force=False):
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        d, i64, u64, u32, i32, f32 = (ctypes.c_double, ctypes.c_int64, ctypes.c_uint64,
                                       ctypes.c_uint32, ctypes.c_int32, ctypes.c_float)
        P = ctypes.c_void_p
        for name in ("ggo_log_rho", "ggo_rho"):
            getattr(L, name).restype = d
            getattr(L, name).argtypes = [d]
        for name in ("ggo_alpha_from_std", "ggo_variance", "ggo_mean_abs",
                     "ggo_diff_entropy_nats"):
            getattr(L, name).restype = d
            getattr(L, name).argtypes = [d, d]
        L.ggo_init_alpha.restype = d
        L.ggo_init_alpha.argtypes = [i64, d, d]
        L.ggo_moments.restype = None
        L.ggo_moments.argtypes = [P, i64, P, P, P]
        L.ggo_fit_from_moments.restype = u32
        L.ggo_fit_from_moments.argtypes = [d, d, i64, i64, P, P]
        L.ggo_penalty_grad.restype = None
        L.ggo_penalty_grad.argtypes = [P, i64, d, d, d, P, P]
        L.ggo_quantise_hist.restype = None
        L.ggo_quantise_hist.argtypes = [P, i64, f32, i32, i32, P, P]
        L.ggo_quantise.restype = None
        L.ggo_quantise.argtypes = [P, i64, f32, i32, i32, P]
        L.ggo_entropy_bits.restype = d
        L.ggo_entropy_bits.argtypes = [P, i64]
        L.ggo_philox4x32_10.restype = None
        L.ggo_philox4x32_10.argtypes = [P, P, P]
        L.ggo_sample_one.restype = d
        L.ggo_sample_one.argtypes = [d, d, u64, u32, u64, P]
        L.ggo_sample.restype = None
        L.ggo_sample.argtypes = [d, d, u64, u32, u64, i64, P, P]
        L.ggo_sample_debug.restype = None
        L.ggo_sample_debug.argtypes = [d, u64, u32, u64, u32, P, P, P]
        L.ggo_map.restype = u64
        L.ggo_map.argtypes = [i64]
        L.ggo_eg_length.restype = i32
        L.ggo_eg_length.argtypes = [u64, i32]
        L.ggo_eg_rate.restype = d
        L.ggo_eg_rate.argtypes = [P, i64, f32, i32, i32, i32]
        L.ggo_eg_rate_hist.restype = d
        L.ggo_eg_rate_hist.argtypes = [P, i64, i32, i32]
        L.ggo_eg_rate_grad.restype = None
        L.ggo_eg_rate_grad.argtypes = [P, i64, f32, i32, i32, i32, d, P]
        L.ggo_huffman_bits.restype = d
        L.ggo_huffman_bits.argtypes = [P, i64, P]
        L.ggo_fixed_length_bits.restype = i32
        L.ggo_fixed_length_bits.argtypes = [P, i64]
        L.ggo_gct_step.restype = None
        L.ggo_gct_step.argtypes = [P, P, P, i64, f32, i32, i32, i32, d, d, d, i64, P, P, P]
        _lib = L
    return _lib


def _f32(x):
    a = np.ascontiguousarray(x, dtype=np.float32)
    return a, a.ctypes.data


# ----------------------------------------------------------- closed forms
def log_rho(beta): return lib().ggo_log_rho(float(beta))
def rho(beta): return lib().ggo_rho(float(beta))
def alpha_from_std(std, beta): return lib().ggo_alpha_from_std(float(std), float(beta))
def variance(alpha, beta): return lib().ggo_variance(float(alpha), float(beta))
def mean_abs(alpha, beta): return lib().ggo_mean_abs(float(alpha), float(beta))
def diff_entropy_nats(alpha, beta): return lib().ggo_diff_entropy_nats(float(alpha), float(beta))
def init_alpha(d_in, xi, beta): return lib().ggo_init_alpha(int(d_in), float(xi), float(beta))


# ------------------------------------------------------------- the steps
def moments(x):
    """(sum|x|, sum x^2, n, n_nonfinite) of an fp32 array (bf16 widened by the caller)."""
    a, p = _f32(x)
    s1, s2, bad = ctypes.c_double(), ctypes.c_double(), ctypes.c_int64()
    lib().ggo_moments(p, a.size, ctypes.byref(s1), ctypes.byref(s2), ctypes.byref(bad))
    return s1.value, s2.value, int(a.size), bad.value


def fit_from_moments(sum_abs, sum_sq, n, n_nonfinite=0):
    """(beta, alpha, flags) from the three moments."""
    b, al = ctypes.c_double(), ctypes.c_double()
    fl = lib().ggo_fit_from_moments(float(sum_abs), float(sum_sq), int(n), int(n_nonfinite),
                                    ctypes.byref(b), ctypes.byref(al))
    return b.value, al.value, int(fl)


def fit(x):
    """(beta, alpha, sum_abs, sum_sq, n, flags) of one segment."""
    s1, s2, n, bad = moments(x)
    b, al, fl = fit_from_moments(s1, s2, n, bad)
    return b, al, s1, s2, n, fl


def penalty_grad(x, beta, alpha, lam, want_grad=True):
    """(penalty, grad as fp64 array or None)."""
    a, p = _f32(x)
    g = np.empty(a.size, dtype=np.float64) if want_grad else None
    pen = ctypes.c_double()
    lib().ggo_penalty_grad(p, a.size, float(beta), float(alpha), float(lam),
                           g.ctypes.data if want_grad else None, ctypes.byref(pen))
    return pen.value, g


def quantise_hist(x, step, qmin=-32768, qmax=32767, hist=None, clamped=None):
    """Adds the symbols of x to hist (uint64[qmax-qmin+1]); returns (hist, clamped[2])."""
    a, p = _f32(x)
    nb = qmax - qmin + 1
    if hist is None:
        hist = np.zeros(nb, dtype=np.uint64)
    if clamped is None:
        clamped = np.zeros(2, dtype=np.uint64)
    assert hist.dtype == np.uint64 and hist.size == nb and hist.flags.c_contiguous
    lib().ggo_quantise_hist(p, a.size, np.float32(step).item(), int(qmin), int(qmax),
                            hist.ctypes.data, clamped.ctypes.data)
    return hist, clamped


def quantise(x, step, qmin=-32768, qmax=32767):
    a, p = _f32(x)
    q = np.empty(a.size, dtype=np.int32)
    lib().ggo_quantise(p, a.size, np.float32(step).item(), int(qmin), int(qmax), q.ctypes.data)
    return q


def entropy_bits(hist):
    h = np.ascontiguousarray(hist, dtype=np.uint64)
    return lib().ggo_entropy_bits(h.ctypes.data, h.size)


# ------------------------------------------------ code lengths (Eq. 6-7)
def map_unsigned(q): return int(lib().ggo_map(int(q)))
def eg_length(m, k=0): return int(lib().ggo_eg_length(int(m), int(k)))


def eg_rate(x, step, k=0, qmin=-32768, qmax=32767):
    """Mean k-th order Exponential-Golomb code length of the quantised elements, bits."""
    a, p = _f32(x)
    return lib().ggo_eg_rate(p, a.size, np.float32(step).item(), int(qmin), int(qmax), int(k))


def eg_rate_hist(hist, k=0, qmin=-32768):
    h = np.ascontiguousarray(hist, dtype=np.uint64)
    return lib().ggo_eg_rate_hist(h.ctypes.data, h.size, int(qmin), int(k))


def eg_rate_grad(x, step, lam, k=0, qmin=-32768, qmax=32767):
    a, p = _f32(x)
    g = np.empty(a.size, dtype=np.float64)
    lib().ggo_eg_rate_grad(p, a.size, np.float32(step).item(), int(qmin), int(qmax), int(k), float(lam),
                           g.ctypes.data)
    return g


def huffman_bits(hist):
    h = np.ascontiguousarray(hist, dtype=np.uint64)
    work = np.empty(2 * h.size, dtype=np.uint64)
    return lib().ggo_huffman_bits(h.ctypes.data, h.size, work.ctypes.data)


def fixed_length_bits(hist):
    h = np.ascontiguousarray(hist, dtype=np.uint64)
    return int(lib().ggo_fixed_length_bits(h.ctypes.data, h.size))


def compression_ratio(bits, fixed_bits):
    """C = 1 - bits / FL: the saving of a variable-length code against the fixed-length one."""
    return 1.0 - float(bits) / float(fixed_bits)


def gct_step(g, ghat_prev, w, step, eta, lam, eps, t, k=0, qmin=-32768, qmax=32767):
    """(ghat, w_new) of one GCT step (Algorithm 2), fp64."""
    a, p = _f32(g)
    gp = np.ascontiguousarray(ghat_prev, dtype=np.float64)
    ww = np.ascontiguousarray(w, dtype=np.float64)
    work = np.empty(a.size, dtype=np.float64)
    gh = np.empty(a.size, dtype=np.float64)
    wn = np.empty(a.size, dtype=np.float64)
    lib().ggo_gct_step(p, gp.ctypes.data, ww.ctypes.data, a.size, np.float32(step).item(), int(qmin), int(qmax),
                       int(k), float(eta), float(lam), float(eps), int(t), work.ctypes.data, gh.ctypes.data,
                       wn.ctypes.data)
    return gh, wn


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.empty(4, dtype=np.uint32)
    lib().ggo_philox4x32_10(c.ctypes.data, k.ctypes.data, o.ctypes.data)
    return o


def sample(beta, alpha, seed, tensor_id, n, index0=0, want_attempts=False):
    """n GG variates as fp64 (and the attempts used, uint8)."""
    out = np.empty(int(n), dtype=np.float64)
    att = np.empty(int(n), dtype=np.uint8) if want_attempts else None
    lib().ggo_sample(float(beta), float(alpha), int(seed), int(tensor_id), int(index0), int(n),
                     out.ctypes.data, att.ctypes.data if want_attempts else None)
    return (out, att) if want_attempts else out


def sample_debug(beta, seed, tensor_id, index, attempt=0):
    z, lhs, rhs = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    lib().ggo_sample_debug(float(beta), int(seed), int(tensor_id), int(index), int(attempt),
                           ctypes.byref(z), ctypes.byref(lhs), ctypes.byref(rhs))
    return z.value, lhs.value, rhs.value


# ------------------------------------------------- storage rounding helpers
def round_to_bf16_bits(x64):
    """fp64 -> bf16 bit patterns (uint16): the nearest bf16, ties to even, decided in fp64.

    The two bf16 neighbours of |x| are the truncation c0 of its fp32 rounding and c0 + 1 ulp;
    |x| - c0 and c1 - |x| are exact in fp64, so the comparison is exact."""
    x = np.asarray(x64, dtype=np.float64)
    ax = np.abs(x)
    f_bits = ax.astype(np.float32).view(np.uint32)
    c0_bits = f_bits & np.uint32(0xFFFF0000)
    c1_bits = c0_bits + np.uint32(0x10000)
    with np.errstate(invalid="ignore", over="ignore"):
        c0 = c0_bits.view(np.float32).astype(np.float64)
        c1 = c1_bits.view(np.float32).astype(np.float64)
        d0 = ax - c0
        d1 = c1 - ax
    up = (d1 < d0) | ((d1 == d0) & (((c0_bits >> 16) & 1) == 1))
    up &= np.isfinite(ax)
    mag = (c0_bits >> 16) + up.astype(np.uint32)
    sign = (np.signbit(x).astype(np.uint32) << 15)
    return (mag | sign).astype(np.uint16)


def bf16_bits_to_f32(bits16):
    return (np.asarray(bits16, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)
