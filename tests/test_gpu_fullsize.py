"""GPU parity at the full sizes of the 7B-, 32B- and 70B-target shapes, in the launch configuration the
benchmark times.  The oracle cannot score every row in float64 (up to 1e14 flop), so it scores a seeded
sample: every row of one whole draft sample (for the per-sample score) plus rows scattered over the rest
of the batch.  Each sampled row still spans the whole vocabulary and the whole hidden dimension."""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, dev_bf16, f32_bits, host_u32, poison, workspace

pytestmark = pytest.mark.gpu

TOL = 2e-3


@pytest.mark.parametrize("name,scattered", [("7b", 192), ("32b", 192), ("70b", 128)])
def test_full_shape_sampled_rows(name, scattered):
    c = inputs.CONFIGS[name]
    N, T, d, V = c["N"], c["T"], c["d"], c["V"]
    M = N * T
    Wb = inputs.lm_head(inputs.BASE_SEED, V, d)
    Hb = inputs.hidden(inputs.BASE_SEED + 1, M, d)
    ids = inputs.zipf_ids(inputs.BASE_SEED + 2, M, V)
    off = inputs.seg_offsets(N, T)
    # directed ids on a few rows: both ends of the vocabulary and tile edges of the last tiles
    ids[:8] = np.array([0, 255, 256, V - 1, V - 2, (V // 256) * 256 - 1, (V // 256) * 256 % V, V // 2], np.int32)
    lp = poison((M,), torch.float32)
    sc = poison((N,), torch.float32)
    ws = workspace(binding.score_workspace_bytes(M, d, V, N))
    binding.score_logprob(dev_bf16(Hb), dev_bf16(Wb), dev(ids), dev(off), lp, sc, ws)
    assert binding.last_device_status() == 0
    lp_h, sc_h = lp.cpu().numpy(), sc.cpu().numpy()
    assert np.isfinite(lp_h).all() and np.isfinite(sc_h).all()

    rng = np.random.default_rng(7)
    sample = int(rng.integers(0, N))
    rows = np.concatenate([np.arange(8), np.arange(sample * T, (sample + 1) * T),
                           rng.choice(M, size=scattered, replace=False)])
    rows = np.unique(rows)
    want = orc.token_logprob(Hb[rows], Wb, ids[rows])
    err = np.abs(lp_h[rows].astype(np.float64) - want)
    assert err.max() <= TOL, f"{name}: max |logprob error| {err.max():.3e}"
    srows = np.arange(sample * T, (sample + 1) * T)
    want_score = orc.sample_score(want[np.searchsorted(rows, srows)], np.array([0, T]))[0]
    assert abs(float(sc_h[sample]) - want_score) <= TOL
    # properties that hold for every row: log-probs are negative and no smaller than the uniform bound minus the
    # logit spread allows; every sample's score equals the mean of the kernel's own token log-probs
    assert (lp_h <= 0).all()
    means = -lp_h.astype(np.float64).reshape(N, T).mean(axis=1)
    assert np.abs(means - sc_h).max() <= 1e-5

    # ---- the configuration's conformal step on the kernel's own fp32 scores, bit for bit against the oracle.
    # The calibration buffer (n scores "from the same generator on another seed") is filled by scoring n / N
    # calibration batches of the same distribution drawn on the device, through the same entry points.
    n_cal, alphas = c["n"], c["alphas"]
    gen = torch.Generator(device="cuda")
    gen.manual_seed(inputs.BASE_SEED + 100)
    W_d, off_d = dev_bf16(Wb), dev(off)
    cdf = torch.cumsum(torch.arange(1, V + 1, device="cuda", dtype=torch.float64) ** -1.1, 0)
    cdf /= cdf[-1].clone()
    calib = poison((n_cal + N,), torch.float32)
    ws_c = workspace(binding.calib_workspace_bytes(n_cal, N))
    Hc = torch.empty((M, d), dtype=torch.bfloat16, device="cuda")
    sc_c = poison((N,), torch.float32)
    n_fill, cal_host = 0, np.zeros(0, np.float32)
    for _ in range(n_cal // N):
        for r0 in range(0, M, 8192):
            x = torch.randn(min(8192, M - r0), d, device="cuda", generator=gen)
            Hc[r0:r0 + x.shape[0]] = (x / x.pow(2).mean(1, keepdim=True).sqrt()).to(torch.bfloat16)
        u = torch.rand(M, device="cuda", dtype=torch.float64, generator=gen)
        idc = torch.searchsorted(cdf, u, right=True).clamp_(max=V - 1).to(torch.int32)
        binding.score_logprob(Hc, W_d, idc, off_d, None, sc_c, ws)
        n_fill = binding.calib_update(calib, n_fill, sc_c, ws_c)
        cal_host = orc.calib_update(cal_host, sc_c.cpu().numpy())
    assert n_fill == n_cal
    assert np.array_equal(f32_bits(calib[:n_cal]), f32_bits(cal_host))
    numer = poison((N,), torch.int32)
    p = poison((N,), torch.float32)
    stage = poison((N,), torch.uint8)
    counts = poison((3,), torch.int32)
    binding.conformal_rank(sc, calib, n_cal, numer, p)
    want_numer = orc.conformal_numer_sorted(sc_h, cal_host)
    assert np.array_equal(host_u32(numer), want_numer)
    assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want_numer, n_cal)))
    assert np.array_equal(want_numer, orc.conformal_numer_count(sc_h, cal_host))
    for alpha in alphas:
        binding.classify(numer, n_cal, alpha, stage, counts)
        want_stage, want_counts = orc.classify(want_numer, n_cal, alpha)
        assert np.array_equal(stage.cpu().numpy(), want_stage)
        assert np.array_equal(host_u32(counts), want_counts)
        # exchangeable test and calibration samples: the number taken over by the target is Binomial(N, ~alpha)
        assert want_counts[2] <= alpha * N + 5 * np.sqrt(alpha * (1 - alpha) * N) + 1
    n_after = binding.calib_update(calib, n_cal, sc, ws_c)
    assert n_after == n_cal + N
    assert np.array_equal(f32_bits(calib), f32_bits(orc.calib_update(cal_host, sc_h)))
    assert binding.last_device_status() == 0


def test_conformal_stress_at_maximum_buffer_size():
    """Last step of the conformal-only workload: 2^20 candidates against n = 323,584, three alphas, insert 4,096."""
    cfg = inputs.CONFORMAL_STRESS
    Nc, k = cfg["Nc"], cfg["k"]
    n = cfg["n0"] + k * (cfg["steps"] - 1)
    scores = inputs.lognormal_scores(inputs.BASE_SEED + 1, Nc)
    calib = np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, n))
    new = inputs.lognormal_scores(inputs.BASE_SEED + 3 + cfg["steps"] - 1, k)
    buf = poison((n + k,), torch.float32)
    buf[:n] = dev(calib)
    numer = poison((Nc,), torch.int32)
    p = poison((Nc,), torch.float32)
    stage = poison((Nc,), torch.uint8)
    counts = poison((3,), torch.int32)
    binding.conformal_rank(dev(scores), buf, n, numer, p)
    want_numer = orc.conformal_numer_sorted(scores, calib)
    assert np.array_equal(host_u32(numer), want_numer)
    assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want_numer, n)))
    idx = np.random.default_rng(1).choice(Nc, size=256, replace=False)
    assert np.array_equal(want_numer[idx], orc.conformal_numer_count(scores[idx], calib))
    for alpha in cfg["alphas"]:
        binding.classify(numer, n, alpha, stage, counts)
        want_stage, want_counts = orc.classify(want_numer, n, alpha)
        assert np.array_equal(stage.cpu().numpy(), want_stage)
        assert np.array_equal(host_u32(counts), want_counts)
        assert abs(want_counts[2] / Nc - alpha) < 0.01       # rejection rate tracks alpha
    n2 = binding.calib_update(buf, n, dev(new), workspace(binding.calib_workspace_bytes(n, k)))
    assert n2 == n + k
    assert np.array_equal(f32_bits(buf), f32_bits(orc.calib_update(calib, new)))


def test_conformal_stress_whole_sequence_with_index_in_one_graph():
    """The conformal-only workload in the form the benchmark times: all 64 steps (rank + three alphas through the
    calibration index, then the indexed update) captured in one CUDA graph and replayed.  The last step's ranks,
    p-values, stages and counts and the final buffer are compared with the oracle, which replays the 64 inserts."""
    cfg = inputs.CONFORMAL_STRESS
    Nc, n0, k, steps, alphas = cfg["Nc"], cfg["n0"], cfg["k"], cfg["steps"], cfg["alphas"]
    scores = inputs.lognormal_scores(inputs.BASE_SEED + 1, Nc)
    calib0 = np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, n0))
    news_h = [inputs.lognormal_scores(inputs.BASE_SEED + 3 + t, k) for t in range(steps)]
    cap = n0 + k * steps
    s_dev, c0_dev, news = dev(scores), dev(calib0), [dev(x) for x in news_h]
    buf = poison((cap,), torch.float32)
    numer, p = poison((Nc,), torch.int32), poison((Nc,), torch.float32)
    stage, counts = poison((len(alphas), Nc), torch.uint8), poison((len(alphas), 3), torch.int32)
    index = workspace(binding.calib_index_bytes(cap))
    ws = workspace(binding.calib_workspace_bytes(cap, k))

    def sequence():
        buf[:n0] = c0_dev
        binding.calib_index_build(buf, n0, index)
        n = n0
        for t in range(steps):
            binding.rank_classify_indexed(s_dev, buf, n, index, alphas, numer, p, stage, counts)
            n = binding.calib_update_indexed(buf, n, news[t], index, ws)
        return n

    assert sequence() == cap                       # eager once (also the device set-up)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        sequence()
    for t in (numer, p, stage, counts):
        t.view(torch.uint8).fill_(0xFF)
    g.replay()
    torch.cuda.synchronize()
    calib = calib0
    for t in range(steps - 1):
        calib = orc.calib_update(calib, news_h[t])
    want_numer = orc.conformal_numer_sorted(scores, calib)     # the last step ranks against n = cap - k entries
    assert np.array_equal(host_u32(numer), want_numer)
    assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want_numer, calib.size)))
    for a, alpha in enumerate(alphas):
        want_stage, want_counts = orc.classify(want_numer, calib.size, alpha)
        assert np.array_equal(stage[a].cpu().numpy(), want_stage)
        assert np.array_equal(host_u32(counts[a]), want_counts)
    assert np.array_equal(f32_bits(buf), f32_bits(orc.calib_update(calib, news_h[-1])))
    assert binding.last_device_status() == 0


def test_conformal_stress_every_step_eager_with_index():
    """All 64 steps of the conformal-only workload through the indexed calls, launched one by one, with the
    numerators, p-value bits, the three rows of stage bytes, their counts and the buffer checked against the
    oracle after every step (the oracle replays the same inserts)."""
    cfg = inputs.CONFORMAL_STRESS
    Nc, n0, k, steps, alphas = cfg["Nc"], cfg["n0"], cfg["k"], cfg["steps"], cfg["alphas"]
    scores = inputs.lognormal_scores(inputs.BASE_SEED + 1, Nc)
    calib = np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, n0))
    cap = n0 + k * steps
    s_dev = dev(scores)
    buf = poison((cap,), torch.float32)
    buf[:n0] = dev(calib)
    numer, p = poison((Nc,), torch.int32), poison((Nc,), torch.float32)
    stage, counts = poison((len(alphas), Nc), torch.uint8), poison((len(alphas), 3), torch.int32)
    index = workspace(binding.calib_index_bytes(cap))
    ws = workspace(binding.calib_workspace_bytes(cap, k))
    binding.calib_index_build(buf, n0, index)
    n = n0
    for t in range(steps):
        new = inputs.lognormal_scores(inputs.BASE_SEED + 3 + t, k)
        for out in (numer, p, stage, counts):
            out.view(torch.uint8).fill_(0xFF)
        binding.rank_classify_indexed(s_dev, buf, n, index, alphas, numer, p, stage, counts)
        n_next = binding.calib_update_indexed(buf, n, dev(new), index, ws)
        torch.cuda.synchronize()
        want_numer = orc.conformal_numer_sorted(scores, calib)
        assert np.array_equal(host_u32(numer), want_numer), t
        assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want_numer, n))), t
        for a, alpha in enumerate(alphas):
            want_stage, want_counts = orc.classify(want_numer, n, alpha)
            assert np.array_equal(stage[a].cpu().numpy(), want_stage), (t, alpha)
            assert np.array_equal(host_u32(counts[a]), want_counts), (t, alpha)
        calib = orc.calib_update(calib, new)
        assert n_next == calib.size
        assert np.array_equal(f32_bits(buf[:n_next]), f32_bits(calib)), t
        n = n_next
    assert n == cap and np.all(np.diff(calib) >= 0)
    assert binding.last_device_status() == 0


def test_takeover_ids_at_the_largest_range_size():
    """Budget report on 2^24 + 3 stage bytes, where the kernel works in ranges of 32 KB over several turns per block:
    mostly 10 % of the samples in stage 3, with a stretch in which all are (more positions than a range can stage: the
    direct path), a stretch in which none is, other byte values, and a stage array that does not start on a 16-byte
    boundary.  Expected positions by the definition, vectorised (numpy), which the oracle's loop is checked against on
    a slice."""
    Nc = (1 << 24) + 3
    rng = np.random.default_rng(99)
    stage_h = np.where(rng.random(Nc) < 0.1, 3, 2).astype(np.uint8)
    stage_h[3_000_000:3_200_000] = 3
    stage_h[9_000_000:9_300_000] = 2
    stage_h[12_000_001:12_100_000] = rng.integers(0, 256, 99_999).astype(np.uint8)
    want = np.flatnonzero(stage_h == 3).astype(np.int32)
    assert np.array_equal(orc.takeover_ids(stage_h[2_990_000:3_010_000]) + 2_990_000, want[(want >= 2_990_000) & (want < 3_010_000)])
    ws = workspace(binding.takeover_ids_workspace_bytes(Nc))
    for shift in (0, 5):
        st = poison((Nc + 16,), torch.uint8)
        st[shift:shift + Nc] = dev(stage_h)
        ids, count = poison((want.size + 3,), torch.int32), poison((1,), torch.int32)
        binding.takeover_ids(st[shift:shift + Nc], ids[:want.size], count, ws)
        torch.cuda.synchronize()
        assert host_u32(count)[0] == want.size
        got = ids.cpu().numpy()
        assert np.array_equal(got[:want.size], want)
        assert np.all(got.view(np.uint32)[want.size:] == 0xFFFFFFFF)
    assert binding.last_device_status() == 0
