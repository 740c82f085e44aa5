"""The C-ABI library loads without a GPU and exports every symbol include/atts.h declares;
argument errors are reported before anything touches a device."""
import ctypes
import os
import re

import pytest

from paper_2509_15148_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "atts.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(atts_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    lib = binding.load()
    names = _declared()
    assert set(names) == set(binding.EXPORTS)
    for name in names:
        assert getattr(lib, name) is not None


def test_strerror_and_version():
    assert binding.version() >= 100
    seen = set()
    for code in range(0, 12):
        s = binding.strerror(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 12
    assert binding.strerror(1234) == "unknown status"


def test_argument_errors_need_no_device():
    lib = binding.load()
    sz = ctypes.c_size_t(0)
    # shape errors are found before the device is probed
    assert lib.atts_score_workspace_bytes(16, 100, 1000, 1, ctypes.byref(sz)) == 2      # d % 64
    assert lib.atts_score_workspace_bytes(16, 0, 1000, 1, ctypes.byref(sz)) == 2
    assert lib.atts_score_workspace_bytes(-1, 64, 1000, 1, ctypes.byref(sz)) == 2
    assert lib.atts_score_workspace_bytes(16, 64, 0, 1, ctypes.byref(sz)) == 2
    assert lib.atts_score_workspace_bytes(16, 64, 1000, 1, None) == 1
    assert lib.atts_calib_workspace_bytes(10, 5, ctypes.byref(sz)) == 0 and sz.value >= 4 * 20
    assert lib.atts_calib_workspace_bytes(-1, 5, ctypes.byref(sz)) == 2
    assert lib.atts_calib_workspace_bytes(1 << 24, 5, ctypes.byref(sz)) == 2
    assert lib.atts_calib_update(None, 10, 12, None, 5, None, None, 0, None) == 5           # capacity first
    assert lib.atts_calib_update(None, 10, 20, None, 5, None, None, 0, None) == 1           # then NULLs
    assert lib.atts_classify(None, 4, 10, 1.5, None, None, None) == 6                      # alpha range
    assert lib.atts_classify(None, 4, 10, 0.0, None, None, None) == 6
    assert lib.atts_classify(None, 4, 10, float("nan"), None, None, None) == 6
    assert lib.atts_classify(None, 4, 10, 0.5, None, None, None) == 1
    assert lib.atts_conformal_rank(None, 4, None, 0, None, None, None) == 1
    assert lib.atts_conformal_rank(None, -1, None, 0, None, None, None) == 2
    assert lib.atts_conformal_rank(None, 0, None, 1 << 24, None, None, None) == 2
    assert lib.atts_score_logprob(None, None, None, None, 8, 64, 100, 1, 7, None, None, None, 0, None) == 6
    assert lib.atts_score_logprob(None, None, None, None, 8, 64, 100, 1, 0, None, None, None, 0, None) == 1
    assert lib.atts_last_device_status(None, None) == 1
    assert lib.atts_calib_index_bytes(524223, ctypes.byref(sz)) == 0 and sz.value % 256 == 0 and sz.value >= 4 * (8192 + 8 * 8191)
    assert lib.atts_calib_index_bytes((1 << 24) - 2, ctypes.byref(sz)) == 0 and sz.value >= 8 * ((1 << 24) - 2)
    assert lib.atts_calib_index_bytes((1 << 24) - 1, ctypes.byref(sz)) == 2                 # beyond the buffer API's range
    assert lib.atts_calib_index_bytes(10, None) == 1
    assert lib.atts_takeover_ids_workspace_bytes(1 << 20, ctypes.byref(sz)) == 0 and sz.value >= 4 * 64 and sz.value % 256 == 0
    assert lib.atts_takeover_ids_workspace_bytes(-1, ctypes.byref(sz)) == 2
    assert lib.atts_takeover_ids(None, 8, None, 8, None, None, 0, None) == 1
    assert lib.atts_takeover_ids(None, 8, None, -1, None, None, 0, None) == 2
    assert lib.atts_conformal_rank_conditional(None, None, 4, None, -1, None, 2, None, None, None, None) == 2   # array length
    assert lib.atts_conformal_rank_conditional(None, None, 4, None, 1 << 31, None, 2, None, None, None, None) == 2
    assert lib.atts_conformal_rank_conditional(None, None, 4, None, 10, None, 2, None, None, None, None) == 1
    assert lib.atts_debug_set_wait(100, 2) == 6 and lib.atts_debug_set_wait(0, 0) == 0
    assert lib.atts_debug_score_form(8, 100, 1000, None) == 1
    assert lib.atts_calib_index_build(None, 10, None, 0, None) == 1
    assert lib.atts_calib_index_build(None, 1 << 24, None, 0, None) == 2
    assert lib.atts_calib_update_indexed(None, 10, 20, None, 5, None, None, 0, None, 0, None) == 1
    assert lib.atts_rank_classify_indexed(None, 4, None, 0, None, None, 5, None, None, None, None, None) == 6
    assert lib.atts_rank_classify_indexed(None, 4, None, 1 << 24, None, None, 0, None, None, None, None, None) == 2


def test_no_device_means_error_not_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    lib = binding.load()
    sz = ctypes.c_size_t(0)
    assert lib.atts_score_workspace_bytes(16, 64, 1000, 1, ctypes.byref(sz)) in (7, 8)
    bits = ctypes.c_uint32(0)
    assert lib.atts_last_device_status(None, ctypes.byref(bits)) in (7, 8)
