"""The allocation-free calibration update gives the same buffer as the workspace version.

atts_calib_update_static exists for callers that cannot obtain device memory at call time: a plug-in
of an engine that has already claimed the GPU's memory, or a loop that must not pay the device-wide
synchronisation of cudaMalloc.  Its scratch is a fixed array inside the library that every call
shares and that keeps the previous call's contents, so the check is made on two calls in a row
(the second starts from a dirty scratch) and against the existing entry point, bit for bit.
This file sorts last so that a run stopping at the first failure has run every other test before it.
"""
import numpy as np
import pytest
import torch

from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, f32_bits, poison, workspace

pytestmark = pytest.mark.gpu


def _both(calib0: np.ndarray, new: np.ndarray, cap: int):
    a = poison((cap,), torch.float32)
    b = poison((cap,), torch.float32)
    n = calib0.size
    if n:
        a[:n] = dev(calib0)
        b[:n] = dev(calib0)
    nw = dev(new) if new.size else None
    ws = workspace(binding.calib_workspace_bytes(n, new.size))
    na = binding.calib_update(a, n, nw, ws)
    nb = binding.calib_update_static(b, n, nw)
    torch.cuda.synchronize()
    return a.cpu().numpy(), na, b.cpu().numpy(), nb


def test_static_update_matches_workspace_update_twice_in_a_row():
    calib = np.sort(inputs.lognormal_scores(1, 5000))
    cap = 5000 + 4096 + 300 + 7
    # first call: large batch, leaves the scratch full of its keys and merged values
    new1 = inputs.lognormal_scores(2, 4096)
    a, na, b, nb = _both(calib, new1, cap)
    assert na == nb == 9096
    assert np.array_equal(f32_bits(a), f32_bits(b))          # poison tail included: nothing written past n + k
    # second call right after, smaller and with ties / special values, on top of the first result
    new2 = np.concatenate([np.round(inputs.lognormal_scores(3, 290), 1),
                           np.array([-0.0, 0.0, np.inf, -np.inf, np.nan, 2.5, 2.5, 2.5, 1e-30, -7.0], np.float32)])
    a2, na2, b2, nb2 = _both(a[:na], new2, cap)
    assert na2 == nb2 == 9396
    assert np.array_equal(f32_bits(a2), f32_bits(b2))
    assert binding.last_device_status() == 0


def test_static_update_edges_and_limits():
    # empty buffer, single element, k = 0
    a, na, b, nb = _both(np.zeros(0, np.float32), inputs.lognormal_scores(4, 1), 4)
    assert na == nb == 1 and np.array_equal(f32_bits(a), f32_bits(b))
    a, na, b, nb = _both(np.sort(inputs.lognormal_scores(5, 9)), np.zeros(0, np.float32), 9)
    assert na == nb == 9 and np.array_equal(f32_bits(a), f32_bits(b))
    # exactly at the limits
    n, k = binding.STATIC_MAX_TOTAL - binding.STATIC_MAX_NEW, binding.STATIC_MAX_NEW
    a, na, b, nb = _both(np.sort(inputs.lognormal_scores(6, n)), inputs.lognormal_scores(7, k), n + k)
    assert na == nb == binding.STATIC_MAX_TOTAL and np.array_equal(f32_bits(a), f32_bits(b))
    # beyond them: a clear error, nothing launched, buffer untouched
    buf = poison((binding.STATIC_MAX_TOTAL + 8,), torch.float32)
    with pytest.raises(binding.AttsError) as e:
        binding.calib_update_static(buf, binding.STATIC_MAX_TOTAL, dev(inputs.lognormal_scores(8, 1)))
    assert e.value.status == 10 and "scratch" in str(e.value)
    with pytest.raises(binding.AttsError) as e:
        binding.calib_update_static(buf, 10, dev(inputs.lognormal_scores(9, binding.STATIC_MAX_NEW + 1)))
    assert e.value.status == 10
    with pytest.raises(binding.AttsError) as e:
        binding.calib_update_static(buf[:12], 10, dev(inputs.lognormal_scores(9, 5)))
    assert e.value.status == 5
    torch.cuda.synchronize()
    assert np.all(f32_bits(buf) == 0xFFFFFFFF)
