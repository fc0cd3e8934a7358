"""CPU checks of the C-ABI boundary: the library builds, loads, and exports every symbol that
include/str.h declares; the host-only schedule helpers agree with the oracle."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2603_00198_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libstr():
    build.build()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "str.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(str_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(libstr):
    names = _declared()
    assert len(names) >= 25
    for n in names:
        assert hasattr(libstr, n), n
    assert set(binding.EXPORTS) <= set(names)


def test_error_strings(libstr):
    assert libstr.str_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert len(libstr.str_strerror(code)) > 3


def test_keep_counts_match_oracle(libstr):
    cases = [([10000] * 4 + [5000] * 4 + [2500] * 4, 32768, 256), ([10000, 1000, 1000], 16384, 256),
             ([5000, 100, 9000], 1000, 144), ([10000, 2500], 100, 144), ([10000, 3162, 1000], 65536, 256),
             ([7071, 7071, 5000], 16384, 0)]
    for alpha, n0, mk in cases:
        assert binding.str_schedule_keep_counts(alpha, n0, mk) == oracle.schedule_keep_counts(alpha, n0, mk)
    with pytest.raises(binding.StrError):
        binding.str_schedule_keep_counts([10001], 10, 0)


def test_sigmoid_schedule_matches_oracle(libstr):
    for x0 in (0.11, 0.24, 0.41):
        bp = binding.str_sigmoid_schedule_bp(62, 20.0, x0, 1.0, 0.125)
        ref = oracle.sigmoid_schedule(62, 20.0, x0, 1.0, 0.125)
        assert all(abs(b - r * 10000) <= 0.5 + 1e-6 for b, r in zip(bp, ref))
        assert bp == sorted(bp, reverse=True)


def test_argument_validation_needs_no_gpu(libstr):
    # null context / null pointers are rejected on the host before anything touches CUDA
    assert libstr.str_topk_select(None, 1, 8, 4, None, None, None, ctypes.c_size_t(0), None) == -1
    assert libstr.str_compact(None, 1, 8, 6, 2, 3, 16, 1, None, None, None, None, None, None, None, None) == -1
    assert libstr.str_destroy(None) == -1
    # the score variants and the FFN activation too
    assert libstr.str_mamba_importance_dynamic(None, None, 8, 2, None, None, None, None, None, None, ctypes.c_size_t(0), None) == -1
    assert libstr.str_attn_importance_ex(None, None, 8, 2, None, None, ctypes.c_float(1.0), 0, None, None, ctypes.c_size_t(0), None) == -1
    assert libstr.str_relu_squared(None, 1, ctypes.c_size_t(8), None, None, None) == -1
    libstr.str_mamba_importance_dynamic_workspace_size.restype = ctypes.c_size_t
    assert libstr.str_mamba_importance_dynamic_workspace_size(None, 8, 2) == 0


def test_newer_entry_points_validate_on_the_host(libstr):
    c_int, c_float, c_size_t = ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    assert libstr.str_score_density(None, 1, 8, None, c_float(0.8), None, None) == -1
    assert libstr.str_attn_prefill_rows(None, None, 4, None, None, None, None, c_float(1.0), None, None, c_size_t(0), None) == -1
    assert libstr.str_stack_prefill_ex(None, None, None, None, None, None, None, None, None, None, c_size_t(0), None) == -1
    assert libstr.str_selftest_wait_timeout(None, ctypes.c_uint(10), None) == -1
    assert libstr.str_mamba_in_proj_conv(None, 1, 1, 8, 64, 8, 32, 32, 1, 4, *([None] * 11)) == -1
    tc, fb = ctypes.c_longlong(), ctypes.c_longlong()
    assert libstr.str_path_counts(None, ctypes.byref(tc), ctypes.byref(fb)) == -1
    # the schedule helper with layer kinds: unknown kinds and missing arrays are refused
    a = (c_int * 3)(10000, 5000, 2500)
    out = (c_int * 3)()
    assert libstr.str_schedule_keep_counts_layers(a, (c_int * 3)(0, 2, 7), 3, 100, 0, out) == -1
    assert libstr.str_schedule_keep_counts_layers(a, None, 3, 100, 0, out) == -1
    assert libstr.str_schedule_keep_counts_layers(a, (c_int * 3)(0, 2, 1), 3, 100, 0, out) == 0 and list(out) == [100, 100, 25]
