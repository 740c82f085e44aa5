"""The whole step can be captured once in a CUDA graph and replayed on new inputs: no call of the path
synchronises, allocates or depends on host state other than its arguments."""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, dev_bf16, f32_bits, host_u32, poison, workspace

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,T,d,V,n0", [(8, 64, 512, 8192, 256), (24, 50, 256, 3000, 100)])
def test_step_captured_in_a_graph_matches_eager_and_oracle(N, T, d, V, n0):
    M = N * T
    Wb = inputs.lm_head(1, V, d)
    W = dev_bf16(Wb)
    off = dev(inputs.seg_offsets(N, T))
    H = torch.zeros((M, d), dtype=torch.bfloat16, device="cuda")
    ids = torch.zeros(M, dtype=torch.int32, device="cuda")
    calib = torch.zeros(n0 + N, device="cuda")
    lp = poison((M,), torch.float32)
    sc = poison((N,), torch.float32)
    numer = poison((N,), torch.int32)
    p = poison((N,), torch.float32)
    stage = poison((N,), torch.uint8)
    counts = poison((3,), torch.int32)
    ws_s = workspace(binding.score_workspace_bytes(M, d, V, N))
    ws_c = workspace(binding.calib_workspace_bytes(n0, N))
    binding.load()
    binding.conformal_rank(sc, calib, 0, numer, None)          # first use outside the capture (device set-up)
    torch.cuda.synchronize()

    def step():
        binding.score_logprob(H, W, ids, off, lp, sc, ws_s)
        binding.conformal_rank(sc, calib, n0, numer, p)
        binding.classify(numer, n0, 0.2, stage, counts)
        return binding.calib_update(calib, n0, sc, ws_c)

    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        step()                                                   # warm-up on the side stream
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        n1 = step()
    assert n1 == n0 + N
    for seed in (11, 12):
        Hb = inputs.hidden(seed, M, d)
        idn = inputs.zipf_ids(seed + 100, M, V)
        cal0 = (np.sort(inputs.lognormal_scores(seed + 200, n0)) + np.float32(6.0)).astype(np.float32)
        H.copy_(dev_bf16(Hb))
        ids.copy_(dev(idn))
        calib[:n0] = dev(cal0)
        g.replay()
        torch.cuda.synchronize()
        got = dict(lp=lp.cpu().numpy(), sc=sc.cpu().numpy(), numer=host_u32(numer).copy(), p=p.cpu().numpy(),
                   stage=stage.cpu().numpy(), counts=host_u32(counts).copy(), calib=calib.cpu().numpy())
        want_lp = orc.token_logprob(Hb, Wb, idn)
        assert np.abs(got["lp"] - want_lp).max() <= 2e-3
        want_numer = orc.conformal_numer_sorted(got["sc"], cal0)
        assert np.array_equal(got["numer"], want_numer)
        assert np.array_equal(f32_bits(got["p"]), f32_bits(orc.pvalue(want_numer, n0)))
        ws, wc = orc.classify(want_numer, n0, 0.2)
        assert np.array_equal(got["stage"], ws) and np.array_equal(got["counts"], wc)
        assert np.array_equal(f32_bits(got["calib"]), f32_bits(orc.calib_update(cal0, got["sc"])))
        # the same inputs run eagerly give the same bits
        calib[:n0] = dev(cal0)
        step()
        torch.cuda.synchronize()
        assert np.array_equal(f32_bits(lp), f32_bits(got["lp"]))
        assert np.array_equal(f32_bits(calib), f32_bits(got["calib"]))
    assert binding.last_device_status() == 0
