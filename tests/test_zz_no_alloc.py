"""The allocation-free calibration update: the oracle's buffer, the same bits as the workspace version, and no
device memory obtained by the call.

atts_calib_update_static exists for callers that cannot obtain device memory at call time: a plug-in
of an engine that has already claimed the GPU's memory, or a loop that must not pay the device-wide
synchronisation of cudaMalloc.  Its scratch is a fixed array inside the library that every call
shares and that keeps the previous call's contents, so the check is made on two calls in a row
(the second starts from a dirty scratch): against the CPU oracle's definition of the update, against the
existing entry point bit for bit, and with the device's free memory read before and after.
This file sorts last so that a run stopping at the first failure has run every other test before it.
"""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, f32_bits, poison, workspace

pytestmark = pytest.mark.gpu


def _both(calib0: np.ndarray, new: np.ndarray, cap: int):
    n = calib0.size
    a = poison((cap,), torch.float32)
    copies = [poison((cap,), torch.float32) for _ in range(3)]    # every buffer exists before free memory is read
    if n:
        a[:n] = dev(calib0)
        for c in copies:
            c[:n] = a[:n]
    nw = dev(new) if new.size else None
    ws = workspace(binding.calib_workspace_bytes(n, new.size))
    na = binding.calib_update(a, n, nw, ws)
    torch.cuda.synchronize()
    # Free device memory is a figure of the whole GPU, so a reading that moved is taken again on a fresh copy; the
    # call itself must leave it where it was.
    unchanged = False
    for b in copies:
        free_before = torch.cuda.mem_get_info()[0]
        nb = binding.calib_update_static(b, n, nw)
        torch.cuda.synchronize()
        unchanged = torch.cuda.mem_get_info()[0] == free_before
        if unchanged:
            break
    assert unchanged                                             # the call obtained no device memory
    return a.cpu().numpy(), na, b.cpu().numpy(), nb


def _check(calib0, new, cap):
    a, na, b, nb = _both(calib0, new, cap)
    want = orc.calib_update(calib0, new)
    assert na == nb == want.size
    assert np.array_equal(f32_bits(b[:nb]), f32_bits(want))   # the definition: sorted union, canonical bits
    assert np.array_equal(f32_bits(a), f32_bits(b))           # and the workspace version, poison tail included
    return b[:nb]


def test_static_update_matches_oracle_and_workspace_update_twice_in_a_row():
    binding.calib_update_static(poison((8,), torch.float32), 0, dev(inputs.lognormal_scores(1, 2)))   # start-up call
    torch.cuda.synchronize()
    calib = np.sort(inputs.lognormal_scores(1, 5000))
    cap = 5000 + 4096 + 300 + 7
    # first call: large batch, leaves the scratch full of its merged values
    merged = _check(calib, inputs.lognormal_scores(2, 4096), cap)
    assert merged.size == 9096
    # second call right after, smaller and with ties / special values, on top of the first result
    new2 = np.concatenate([np.round(inputs.lognormal_scores(3, 290), 1),
                           np.array([-0.0, 0.0, np.inf, -np.inf, np.nan, 2.5, 2.5, 2.5, 1e-30, -7.0], np.float32)])
    merged2 = _check(merged, new2, cap)
    assert merged2.size == 9396
    assert binding.last_device_status() == 0


def test_static_update_edges_and_limits():
    # empty buffer, single element, k = 0
    _check(np.zeros(0, np.float32), inputs.lognormal_scores(4, 1), 4)
    _check(np.sort(inputs.lognormal_scores(5, 9)), np.zeros(0, np.float32), 9)
    # exactly at the limits
    n, k = binding.STATIC_MAX_TOTAL - binding.STATIC_MAX_NEW, binding.STATIC_MAX_NEW
    out = _check(np.sort(inputs.lognormal_scores(6, n)), inputs.lognormal_scores(7, k), n + k)
    assert out.size == binding.STATIC_MAX_TOTAL
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
