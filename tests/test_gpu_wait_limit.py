"""The bounded waits of the fused scoring kernel: a wait that cannot be satisfied runs out, the kernel returns on its
own, the condition is reported as ATTS_ERR_TIMEOUT and cleared, and the next call is correct.

Nothing is broken to get there: the library's diagnostic switch makes the kernel's producer issue no loads, so the
first wait for data has nothing to wait for and nothing is in flight when it gives up (no trap, no bad address, no
endless loop; every other role of the kernel sees the raised flag or runs out itself)."""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, dev_bf16, poison, workspace

pytestmark = pytest.mark.gpu


# the first shape runs on CTA pairs (two tiles' worth of rows, few vocabulary tiles), the second on single CTAs
# (one row block against many vocabulary tiles)
@pytest.mark.parametrize("M,d,V,form", [(512, 512, 8192, 2), (128, 128, 65536, 1)])
def test_expired_wait_is_reported_and_the_context_stays_usable(M, d, V, form):
    assert binding.debug_score_form(M, d, V) == form
    Hb, Wb = inputs.hidden(11, M, d), inputs.lm_head(12, V, d)
    ids = inputs.zipf_ids(13, M, V)
    off = np.array([0, M // 2, M], np.int32)
    H, W, ids_d, off_d = dev_bf16(Hb), dev_bf16(Wb), dev(ids), dev(off)
    ws = workspace(binding.score_workspace_bytes(M, d, V, 2))
    lp, sc = poison((M,), torch.float32), poison((2,), torch.float32)
    assert binding.last_device_status() == 0
    try:
        binding.debug_set_wait(2_000_000, withhold_loads=True)       # about a millisecond
        binding.score_logprob(H, W, ids_d, off_d, lp, sc, ws)         # returns: the call only enqueues
        with pytest.raises(binding.AttsError) as err:
            binding.last_device_status()                              # waits for the stream: the kernel has returned
        assert err.value.status == 9 and "wait" in str(err.value)
    finally:
        binding.debug_set_wait(0, withhold_loads=False)
    assert binding.last_device_status() == 0                          # reported once, then cleared
    lp2, sc2 = poison((M,), torch.float32), poison((2,), torch.float32)
    binding.score_logprob(H, W, ids_d, off_d, lp2, sc2, ws)
    assert binding.last_device_status() == 0
    want = orc.token_logprob(Hb, Wb, ids)
    assert np.abs(lp2.cpu().numpy().astype(np.float64) - want).max() <= 2e-3
    assert np.abs(sc2.cpu().numpy() - orc.sample_score(want, off)).max() <= 2e-3


def test_wait_setting_argument_errors():
    lib = binding.load()
    assert lib.atts_debug_set_wait(100, 2) == 6
    assert lib.atts_debug_set_wait(0, 0) == 0
