"""Comparison helpers of the GPU parity tests (tolerances as stated for the library)."""
import numpy as np

REL_FIT = 1e-5          # fitted beta, alpha
REL_PENALTY = 1e-6      # penalty sums
MAX_ULP = 4             # per-element gradient, fp32 units in the last place
ABS_ENTROPY = 1e-9      # bits per symbol


def _ordered(f32):
    """Map fp32 bit patterns to integers that are monotone in the value (so that differences
    count representable numbers, subnormals included)."""
    i = np.asarray(f32, dtype=np.float32).view(np.int32).astype(np.int64)
    return np.where(i < 0, -(i & 0x7FFFFFFF), i)


def ulp_distance(got_f32, ref_f64):
    """Distance in fp32 ulps between the GPU gradient and the fp64 oracle value rounded to fp32."""
    with np.errstate(over="ignore"):
        ref = np.asarray(ref_f64, dtype=np.float64).astype(np.float32)
    return np.abs(_ordered(got_f32) - _ordered(ref))


def assert_grad_close(got_f32, ref_f64, max_ulp=MAX_ULP):
    d = ulp_distance(got_f32, ref_f64)
    bad = np.flatnonzero(d > max_ulp)
    assert bad.size == 0, (f"{bad.size} of {d.size} gradient entries differ by more than {max_ulp} ulp; "
                           f"worst {d.max()} at {int(d.argmax())}: got {np.asarray(got_f32).reshape(-1)[d.argmax()]!r} "
                           f"ref {np.asarray(ref_f64).reshape(-1)[d.argmax()]!r}")
    return int(d.max()) if d.size else 0


def assert_rel(got, ref, rel, what=""):
    assert abs(got - ref) <= rel * abs(ref), f"{what}: got {got!r} ref {ref!r} rel {abs(got - ref) / abs(ref):.3e}"
