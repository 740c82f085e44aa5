"""Randomised GPU parity through the C-ABI: many small and mid-sized problems with sizes drawn around the kernels' mode
switches and values drawn from several families (LogNormal, heavily rounded, packed into a sliver, huge and tiny
magnitudes, arbitrary bit patterns with NaNs and denormals).  Seeds are fixed, so every run sees the same problems.
Integer and bit results are compared exactly, log-probs within 2e-3."""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, dev_bf16, f32_bits, host_u32, poison, workspace

pytestmark = pytest.mark.gpu

POOL = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-38, -1e-38, 3.0, 3e38, -3e38], np.float32)


def draw(rng, n, kind):
    if kind == 0:
        v = np.exp(rng.standard_normal(n)).astype(np.float32)
    elif kind == 1:
        v = np.round(np.exp(rng.standard_normal(n)), int(rng.integers(0, 3))).astype(np.float32)
    elif kind == 2:
        v = (1.0 + 1e-5 * rng.standard_normal(n)).astype(np.float32)
    elif kind == 3:
        v = (rng.standard_normal(n) * 10.0 ** int(rng.integers(-30, 30))).astype(np.float32)
    else:
        v = rng.integers(0, 2 ** 32, n, dtype=np.uint64).astype(np.uint32).view(np.float32).copy()
    if n >= 4 and rng.random() < 0.5:
        idx = rng.choice(n, size=min(n, 5), replace=False)
        v[idx] = rng.choice(POOL, size=idx.size)
    return v


def test_randomised_rank_index_update_and_budget_report():
    rng = np.random.default_rng(777)
    for case in range(48):
        n = int(rng.choice([1, 2, 3, 100, 4095, 4096, 8191, 8192, 8193, 20000, 65527, 65536, 100001, 300000, 524223, 524224, 1000003]))
        Nc = int(rng.choice([1, 17, 4096, 16384, 65536, 65536 + 48, 200000]))
        kc, ks = int(rng.integers(0, 5)), int(rng.integers(0, 5))
        calib = orc.calib_update(np.zeros(0, np.float32), draw(rng, n, kc))
        scores = draw(rng, Nc, ks if rng.random() < 0.5 else kc)
        want = orc.conformal_numer_sorted(scores, calib)
        c, s = dev(calib), dev(scores)
        numer, p = poison((Nc,), torch.int32), poison((Nc,), torch.float32)
        binding.conformal_rank(s, c, n, numer, p)
        torch.cuda.synchronize()
        assert np.array_equal(host_u32(numer), want), ("rank", case, n, Nc, kc, ks)
        assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want, n))), ("p", case, n, Nc)
        index = workspace(binding.calib_index_bytes(n))
        binding.calib_index_build(c, n, index)
        alphas = (0.05, 0.3) if Nc % 16 == 0 else (0.3,)
        stage, counts = poison((len(alphas), Nc), torch.uint8), poison((len(alphas), 3), torch.int32)
        numer2 = poison((Nc,), torch.int32)
        binding.rank_classify_indexed(s, c, n, index, alphas, numer2, None, stage, counts)
        torch.cuda.synchronize()
        assert np.array_equal(host_u32(numer2), want), ("indexed", case, n, Nc, kc, ks)
        for a, alpha in enumerate(alphas):
            want_stage, want_counts = orc.classify(want, n, alpha)
            assert np.array_equal(stage[a].cpu().numpy(), want_stage), ("stage", case, n, Nc, alpha)
            assert np.array_equal(host_u32(counts[a]), want_counts), ("counts", case, n, Nc, alpha)
        ids, count = poison((Nc,), torch.int32), poison((1,), torch.int32)
        binding.takeover_ids(stage[0], ids, count, workspace(binding.takeover_ids_workspace_bytes(Nc)))
        torch.cuda.synchronize()
        want_ids = np.flatnonzero(orc.classify(want, n, alphas[0])[0] == 3)
        assert host_u32(count)[0] == want_ids.size and np.array_equal(ids.cpu().numpy()[:want_ids.size], want_ids)
        k = int(rng.choice([0, 1, 64, 4096, 5000, 20000]))
        if True:
            new = draw(rng, k, int(rng.integers(0, 5)))
            buf = poison((n + k + 8,), torch.float32)
            buf[:n] = c
            index2 = workspace(binding.calib_index_bytes(n + k))
            binding.calib_index_build(buf, n, index2)
            n2 = binding.calib_update_indexed(buf, n, dev(new) if k else None, index2,
                                              workspace(binding.calib_workspace_bytes(n, k)))
            want_buf = orc.calib_update(calib, new)
            torch.cuda.synchronize()
            assert n2 == n + k and np.array_equal(f32_bits(buf[:n2]), f32_bits(want_buf)), ("update", case, n, k)
            assert np.all(f32_bits(buf[n2:]) == 0xFFFFFFFF)
            binding.rank_classify_indexed(s, buf, n2, index2, (), numer2)
            torch.cuda.synchronize()
            assert np.array_equal(host_u32(numer2), orc.conformal_numer_sorted(scores, want_buf)), ("indexed after update", case)
    assert binding.last_device_status() == 0


def test_randomised_scoring_shapes_modes_and_row_factors():
    rng = np.random.default_rng(778)
    worst = 0.0
    for case in range(60):
        M = int(rng.choice([1, 2, 127, 128, 129, 255, 256, 257, 300, 640, 1000, 1500]))
        d = 64 * int(rng.choice([1, 2, 3, 5, 8, 16]))
        V = int(rng.choice([1, 2, 31, 32, 33, 255, 256, 257, 511, 513, 1000, 4099, 9000]))
        seed = int(rng.integers(0, 1 << 30))
        scale = float(rng.choice([0.02, 0.2, 1.0]))
        Wb = inputs.f32_to_bf16_bits((np.random.default_rng(seed).standard_normal((V, d)) * scale).astype(np.float32))
        Hb = inputs.hidden(seed + 1, M, d)
        ids = rng.integers(0, V, size=M).astype(np.int32)
        ids[int(rng.integers(0, M))] = V - 1
        S = int(rng.choice([1, 2, 5, 40]))
        cuts = np.sort(rng.integers(0, M + 1, size=S - 1)) if S > 1 else np.zeros(0, np.int64)
        off = np.concatenate([[0], cuts, [M]]).astype(np.int32)
        mode = int(rng.integers(0, 4))
        H, W = dev_bf16(Hb), dev_bf16(Wb)
        lp, sc = poison((M,), torch.float32), poison((S,), torch.float32)
        ws = workspace(binding.score_workspace_bytes(M, d, V, S))
        if rng.random() < 0.3:
            factor = (0.5 + rng.random(M)).astype(np.float32)
            binding.score_logprob_scaled(H, W, dev(ids), dev(factor), dev(off), lp, sc, ws, mode)
            want = orc.token_logprob_scaled(Hb, Wb, ids, factor)
        else:
            binding.score_logprob(H, W, dev(ids), dev(off), lp, sc, ws, mode)
            want = orc.token_logprob(Hb, Wb, ids)
        assert binding.last_device_status() == 0
        err = float(np.abs(lp.cpu().numpy().astype(np.float64) - want).max())
        worst = max(worst, err)
        assert err <= 2e-3, (case, M, d, V, scale, err)
        want_sc = orc.sample_score(want, off, mode)
        lens = np.diff(off.astype(np.int64))
        got = sc.cpu().numpy()
        assert np.all(np.isnan(got[lens == 0]))
        tol = 2e-3 * (np.maximum(lens, 1) if mode in (1, 3) else np.ones_like(lens))
        assert np.all(np.abs(got[lens > 0] - want_sc[lens > 0]) <= tol[lens > 0]), (case, M, d, V, mode)
    assert worst > 0.0
