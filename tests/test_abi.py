"""The C interface: every function declared in include/gg.h is exported, and the parts that need
no GPU (status strings, host helpers, argument checks) behave."""
import ctypes
import math
import os
import re

import pytest

import __graft_entry__ as entry
from oracle import gg_oracle as o

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    entry.build()
    from paper_2506_00486_b200 import binding
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gg_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"gg_fit", "gg_penalty_grad", "gg_rate_hist", "gg_sample", "gg_fused", "gg_fused_host",
            "gg_create", "gg_destroy"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_status_strings_and_version(L):
    assert L.gg_version() >= 100
    assert L.gg_status_str(0) == b"ok"
    seen = {L.gg_status_str(i) for i in range(9)}
    assert len(seen) == 9 and b"unknown status" not in seen
    assert L.gg_status_str(99) == b"unknown status"


def test_host_helpers_match_the_paper_formulas(L):
    # Eq. 2 special cases: Gaussian alpha = sigma sqrt 2, Laplace alpha = sigma / sqrt 2
    assert L.gg_alpha_from_std(3.0, 2.0) == pytest.approx(3 * math.sqrt(2), rel=1e-14)
    assert L.gg_alpha_from_std(3.0, 1.0) == pytest.approx(3 / math.sqrt(2), rel=1e-14)
    # Eq. 4-5: shape 2 with the ReLU correction is He initialisation (variance 2/d_in)
    a = L.gg_init_alpha(4096, 2.0, 2.0)
    assert a * a / 2 == pytest.approx(2 / 4096, rel=1e-14)
    for beta in (0.1, 0.5, 1.3, 2.0, 7.0):
        assert L.gg_alpha_from_std(0.02, beta) == pytest.approx(o.alpha_from_std(0.02, beta), rel=1e-13)
        assert L.gg_init_alpha(896, 1.0, beta) == pytest.approx(o.init_alpha(896, 1.0, beta), rel=1e-13)
        assert L.gg_diff_entropy_bits(0.3, beta) == pytest.approx(
            o.diff_entropy_nats(0.3, beta) / math.log(2), rel=1e-13)


def test_calls_fail_cleanly_without_a_context(L):
    # null context / null output are argument errors, not crashes
    assert L.gg_create(None, 0) == 1
    assert L.gg_fit(None, None, 0, 0, None, None, None, None, None, None, None) == 1
    assert L.gg_fused(None, None, None) == 1
    assert L.gg_destroy(None) == 0


def test_create_reports_missing_device_as_an_error(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = ctypes.c_void_p()
    assert L.gg_create(ctypes.byref(h), 0) in (5, 6)
    assert not h.value


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2506_00486_b200 import Context
    with pytest.raises(RuntimeError):
        Context(0)
