"""GPU parity of the extension entry points (threshold form, conditional coverage, row-scaled scoring)
against the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, dev_bf16, f32_bits, host_u32, poison, workspace

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("alpha", [0.01, 0.1, 0.25, 0.9])
@pytest.mark.parametrize("Nc,n", [(5, 8), (4099, 400), (300000, 65536)])
def test_threshold_classify_equals_rank_classify(alpha, Nc, n):
    calib = np.sort(np.round(inputs.lognormal_scores(10 + n, n), 2))             # ties
    scores = np.round(inputs.lognormal_scores(20 + Nc, Nc), 2)
    scores[: min(Nc, 4)] = np.array([np.nan, np.inf, -np.inf, calib[-1]], np.float32)[: min(Nc, 4)]
    c_dev, s_dev = dev(calib), dev(scores)
    tau = poison((1,), torch.float32)
    binding.threshold(c_dev, n, alpha, tau)
    stage = poison((Nc,), torch.uint8)
    counts = poison((3,), torch.int32)
    binding.classify_threshold(s_dev, tau, stage, counts)
    torch.cuda.synchronize()
    want_tau = orc.threshold(calib, alpha)
    assert f32_bits(tau)[0] == f32_bits(np.array([want_tau], np.float32))[0]
    want_stage, want_counts = orc.classify_by_threshold(scores, want_tau)
    assert np.array_equal(stage.cpu().numpy(), want_stage)
    assert np.array_equal(host_u32(counts), want_counts)
    # the same bytes as the rank route
    numer = poison((Nc,), torch.int32)
    stage2 = poison((Nc,), torch.uint8)
    binding.conformal_rank(s_dev, c_dev, n, numer, None)
    binding.classify(numer, n, alpha, stage2, None)
    torch.cuda.synchronize()
    assert torch.equal(stage, stage2)


def test_conditional_rank_and_classify_bit_exact():
    rng = np.random.default_rng(3)
    G = 300
    sizes = rng.integers(0, 130, size=G)
    sizes[:3] = [0, 1, 128]
    groups = [np.sort(np.round(inputs.lognormal_scores(100 + g, int(sizes[g])), 1)) for g in range(G)]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    calib = np.concatenate(groups).astype(np.float32)
    Nc = 20000
    gid = rng.integers(0, G, size=Nc).astype(np.int32)
    gid[:3] = [0, 1, 2]
    scores = np.round(inputs.lognormal_scores(7, Nc), 1)
    scores[5] = np.nan
    numer = poison((Nc,), torch.int32)
    denom = poison((Nc,), torch.int32)
    p = poison((Nc,), torch.float32)
    binding.conformal_rank_conditional(dev(scores), dev(gid), dev(calib), dev(off), numer, denom, p)
    want_numer, want_denom = orc.conformal_numer_conditional(scores, gid, groups)
    assert np.array_equal(host_u32(numer), want_numer)
    assert np.array_equal(host_u32(denom), want_denom)
    want_p = (want_numer.astype(np.float64) / want_denom.astype(np.float64)).astype(np.float32)
    want_p[want_numer == 0] = np.nan
    assert np.array_equal(f32_bits(p), f32_bits(want_p))
    for alpha in (0.1, 0.25, 0.5):
        stage = poison((Nc,), torch.uint8)
        counts = poison((3,), torch.int32)
        binding.classify_conditional(numer, denom, alpha, stage, counts)
        want_stage, want_counts = orc.classify_conditional(want_numer, want_denom, alpha)
        assert np.array_equal(stage.cpu().numpy(), want_stage)
        assert np.array_equal(host_u32(counts), want_counts)
    assert binding.last_device_status() == 0
    # a group id out of range is flagged, not fatal
    gid2 = gid.copy()
    gid2[10] = G
    binding.conformal_rank_conditional(dev(scores), dev(gid2), dev(calib), dev(off), numer, denom, None)
    assert binding.last_device_status() & binding.DEV_GROUP_ID_RANGE
    assert host_u32(numer)[10] == 0
    # a calibration array that is not 32-byte aligned (no 256-bit loads), with candidates in random and in grouped order
    shifted = dev(np.concatenate([np.zeros(1, np.float32), calib]))[1:]
    for order in (np.arange(Nc), np.argsort(gid, kind="stable")):
        binding.conformal_rank_conditional(dev(scores[order]), dev(gid[order]), shifted, dev(off), numer, denom, None)
        assert np.array_equal(host_u32(numer), want_numer[order])
    binding.conformal_rank_conditional(dev(scores[order]), dev(gid[order]), dev(calib), dev(off), numer, denom, None)
    assert np.array_equal(host_u32(numer), want_numer[order])
    # offsets that do not describe a part of the calibration array (decreasing, negative, beyond its end) are
    # flagged like a bad group id and never used as addresses; the other groups are unaffected
    for g_bad, (a, b) in ((7, (int(off[8]) + 5, int(off[8]))), (9, (-4, int(off[10]))), (G - 1, (int(off[G - 1]), int(off[G]) + 1000))):
        off2 = off.copy()
        if g_bad == G - 1:
            off2[G] = b
        else:
            off2[g_bad] = a
        hit = (gid == g_bad) | ((gid == g_bad - 1) if g_bad != G - 1 else False)
        binding.conformal_rank_conditional(dev(scores), dev(gid), dev(calib), dev(off2), numer, denom, None)
        assert binding.last_device_status() & binding.DEV_GROUP_ID_RANGE
        got = host_u32(numer)
        assert np.array_equal(got[~hit], want_numer[~hit])
        assert np.all(got[gid == g_bad] == 0)
    # ragged tails and arrays that are not 16-byte aligned take the scalar loads and stores
    for start, stop in ((0, Nc - 1), (1, Nc), (3, Nc - 2), (0, 3)):
        m = stop - start
        numer3, denom3, p3 = poison((m + 4,), torch.int32), poison((m + 4,), torch.int32), poison((m + 4,), torch.float32)
        shift = start % 4
        binding.conformal_rank_conditional(dev(scores)[start:stop], dev(gid)[start:stop], dev(calib), dev(off),
                                           numer3[shift:shift + m], denom3[shift:shift + m], p3[shift:shift + m])
        assert np.array_equal(host_u32(numer3)[shift:shift + m], want_numer[start:stop])
        assert np.array_equal(host_u32(denom3)[shift:shift + m], want_denom[start:stop])
        assert np.array_equal(f32_bits(p3)[shift:shift + m], f32_bits(want_p[start:stop]))
        assert np.all(host_u32(numer3)[shift + m:] == 0xFFFFFFFF) and np.all(host_u32(numer3)[:shift] == 0xFFFFFFFF)
    assert binding.last_device_status() == 0


def test_conditional_rank_warps_with_nothing_to_search():
    """Whole warps whose candidates have no entries to search: empty calibration sets, scores that are all NaN, and a
    single group; then a mix in which only some warps have work."""
    def run(scores, gid, groups):
        off = np.concatenate([[0], np.cumsum([len(x) for x in groups])]).astype(np.int32)
        calib = np.concatenate(groups).astype(np.float32) if off[-1] else np.zeros(1, np.float32)
        Nc = scores.size
        numer, denom, p = poison((Nc,), torch.int32), poison((Nc,), torch.int32), poison((Nc,), torch.float32)
        binding.conformal_rank_conditional(dev(scores), dev(gid), dev(calib), dev(off), numer, denom, p)
        torch.cuda.synchronize()
        wn, wd = orc.conformal_numer_conditional(scores, gid, groups)
        assert np.array_equal(host_u32(numer), wn) and np.array_equal(host_u32(denom), wd)

    empty = np.zeros(0, np.float32)
    scores = inputs.lognormal_scores(21, 1000)
    run(scores, np.zeros(1000, np.int32), [empty])                                   # one group, no calibration scores
    run(scores, (np.arange(1000) % 5).astype(np.int32), [empty] * 5)                 # every group empty
    run(np.full(1000, np.nan, np.float32), np.zeros(1000, np.int32), [np.sort(inputs.lognormal_scores(22, 40))])
    groups = [empty, np.sort(inputs.lognormal_scores(23, 30)), empty, np.sort(inputs.lognormal_scores(24, 700))]
    gid = np.sort(np.random.default_rng(5).integers(0, 4, size=3000)).astype(np.int32)
    run(inputs.lognormal_scores(25, 3000), gid, groups)                              # warps of empty and of large groups
    assert binding.last_device_status() == 0


@pytest.mark.parametrize("M,d,V", [(300, 192, 1000), (1000, 512, 5000), (4096, 1024, 8192)])
def test_rms_inv_and_scaled_scoring(M, d, V):
    rng = np.random.default_rng(M)
    raw = rng.standard_normal((M, d)).astype(np.float32) * rng.uniform(0.2, 6.0, size=(M, 1)).astype(np.float32)
    Hb = inputs.f32_to_bf16_bits(raw)                                   # un-normalised hidden states
    Wb = inputs.lm_head(2, V, d)
    ids = inputs.zipf_ids(3, M, V)
    off = np.array([0, M // 2, M], np.int32)
    H = dev_bf16(Hb)
    rs = poison((M,), torch.float32)
    binding.rms_inv(H, 1e-6, rs)
    torch.cuda.synchronize()
    want_rs = orc.rms_inv(Hb, 1e-6)
    assert np.abs(rs.cpu().numpy() / want_rs - 1).max() < 1e-5
    lp = poison((M,), torch.float32)
    sc = poison((2,), torch.float32)
    ws = workspace(binding.score_workspace_bytes(M, d, V, 2))
    binding.score_logprob_scaled(H, dev_bf16(Wb), dev(ids), rs, dev(off), lp, sc, ws)
    assert binding.last_device_status() == 0
    # the oracle gets the device's fp32 row factors, so that only the scoring arithmetic is compared
    want = orc.token_logprob_scaled(Hb, Wb, ids, rs.cpu().numpy().astype(np.float64))
    assert np.abs(lp.cpu().numpy() - want).max() <= 2e-3
    assert np.abs(sc.cpu().numpy() - orc.sample_score(want, off)).max() <= 2e-3
    # scale 1 reproduces the unscaled entry point bit for bit
    ones = torch.ones(M, device="cuda")
    lp1 = poison((M,), torch.float32)
    lp2 = poison((M,), torch.float32)
    binding.score_logprob_scaled(H, dev_bf16(Wb), dev(ids), ones, dev(off), lp1, sc, ws)
    binding.score_logprob(H, dev_bf16(Wb), dev(ids), dev(off), lp2, sc, ws)
    torch.cuda.synchronize()
    assert torch.equal(lp1, lp2)


@pytest.mark.parametrize("M,d,V,cuts", [(300, 192, 5000, (0, 1700, 1701, 5000)), (1000, 256, 4096, (0, 1024, 2048, 3072, 4096)),
                                        (130, 64, 600, (0, 600)), (4096, 1024, 30000, (0, 9999, 20480, 30000))])
def test_vocabulary_sliced_scoring_equals_the_full_definition(M, d, V, cuts):
    """W split by rows into G slices (as on G tensor-parallel ranks), each scored on its own, the [M, 3] blocks
    stacked in rank order and merged: the result is the log-softmax over the whole vocabulary."""
    Hb, Wb = inputs.hidden(1, M, d), inputs.lm_head(2, V, d)
    ids = inputs.zipf_ids(3, M, V)
    ids[:6] = np.array([0, cuts[1] - 1, cuts[1] % V, V - 1, cuts[-2], cuts[-2] - 1 if cuts[-2] > 0 else 0], np.int32)
    off = np.array([0, M // 3, M], np.int32)
    H, idd = dev_bf16(Hb), dev(ids)
    G = len(cuts) - 1
    stats = poison((G, M, 3), torch.float32)
    for g in range(G):
        a, b = cuts[g], cuts[g + 1]
        Wg = dev_bf16(Wb[a:b])
        ws = workspace(binding.score_workspace_bytes(M, d, b - a, 0))
        binding.score_slice(H, Wg, idd, a, stats[g], ws)
    lp = poison((M,), torch.float32)
    sc = poison((2,), torch.float32)
    binding.score_combine(stats, dev(off), lp, sc, workspace(4 * M + 512))
    assert binding.last_device_status() == 0
    want = orc.token_logprob(Hb, Wb, ids)
    assert np.abs(lp.cpu().numpy() - want).max() <= 2e-3
    assert np.abs(sc.cpu().numpy() - orc.sample_score(want, off)).max() <= 2e-3
    # exactly one slice holds each token's logit
    held = torch.isfinite(stats[:, :, 2]).sum(dim=0).cpu().numpy()
    assert (held == 1).all()
    # an id beyond every slice is flagged and gives NaN
    bad = ids.copy()
    bad[7] = V
    for g in range(G):
        a, b = cuts[g], cuts[g + 1]
        binding.score_slice(H, dev_bf16(Wb[a:b]), dev(bad), a, stats[g], workspace(binding.score_workspace_bytes(M, d, b - a, 0)))
    binding.score_combine(stats, dev(off), lp, sc, workspace(4 * M + 512))
    assert binding.last_device_status() & binding.DEV_TOKEN_ID_RANGE
    assert np.isnan(lp.cpu().numpy()[7])


@pytest.mark.parametrize("Nc", [0, 1, 15, 16, 4095, 4096, 4097, 70001, (1 << 20) + 5])
def test_takeover_ids_bit_exact(Nc):
    """Positions of the samples the target takes over and the budget B, against the oracle: random stages, all stage 3,
    none, arbitrary byte values, an output too short for all of them, and a stage array that is not 16-byte aligned."""
    rng = np.random.default_rng(Nc + 1)
    cases = [rng.choice(np.array([1, 2, 3], np.uint8), size=Nc, p=[0.05, 0.7, 0.25]),
             np.full(Nc, 3, np.uint8), np.full(Nc, 2, np.uint8),
             # every byte value, threes made frequent: only the byte 3 itself counts (0x83, 0x13, 0x02, 0x07 do not)
             np.where(rng.random(Nc) < 0.3, 3, rng.integers(0, 256, Nc)).astype(np.uint8)]
    ws = workspace(binding.takeover_ids_workspace_bytes(Nc))
    for stage_h in cases:
        want = orc.takeover_ids(stage_h) if Nc < 200000 else np.flatnonzero(stage_h == 3).astype(np.int32)
        for shift, cap in ((0, Nc), (1, Nc), (0, want.size // 2)):
            st = poison((Nc + 16,), torch.uint8)
            st[shift:shift + Nc] = dev(stage_h) if Nc else st[:0]
            ids = poison((cap + 3,), torch.int32)
            count = poison((1,), torch.int32)
            binding.takeover_ids(st[shift:shift + Nc], ids[:cap], count, ws)
            torch.cuda.synchronize()
            assert host_u32(count)[0] == want.size
            got = ids.cpu().numpy()
            m = min(cap, want.size)
            assert np.array_equal(got[:m], want[:m])
            assert np.all(got.view(np.uint32)[m:] == 0xFFFFFFFF)        # nothing written past what fits
    if Nc >= 200000:   # the shortcut above is the oracle's definition: checked on a sample of positions
        assert np.array_equal(orc.takeover_ids(cases[0][:5000]), np.flatnonzero(cases[0][:5000] == 3))
    assert binding.last_device_status() == 0


def test_takeover_ids_follow_classify():
    n, Nc, alpha = 4096, 64, 0.25
    calib = np.sort(inputs.lognormal_scores(11, n))
    scores = inputs.lognormal_scores(12, Nc)
    numer, stage, counts = poison((Nc,), torch.int32), poison((Nc,), torch.uint8), poison((3,), torch.int32)
    binding.conformal_rank(dev(scores), dev(calib), n, numer, None)
    binding.classify(numer, n, alpha, stage, counts)
    ids, count = poison((Nc,), torch.int32), poison((1,), torch.int32)
    binding.takeover_ids(stage, ids, count, workspace(binding.takeover_ids_workspace_bytes(Nc)))
    torch.cuda.synchronize()
    want_stage, want_counts = orc.classify(orc.conformal_numer_sorted(scores, calib), n, alpha)
    want = orc.takeover_ids(want_stage)
    assert host_u32(count)[0] == want_counts[2] == want.size
    assert np.array_equal(ids.cpu().numpy()[:want.size], want)


def test_conditional_rank_randomised_groups_and_alignments():
    """Sixty random problems: group counts and sizes from empty to thousands of entries (staged and unstaged warps),
    sorted and shuffled group ids, rounded values (ties), a NaN score, and output arrays at every 4-byte alignment."""
    rng = np.random.default_rng(20250131)
    for case in range(60):
        G = int(rng.choice([1, 2, 7, 100, 3000]))
        sizes = rng.integers(0, int(rng.choice([1, 8, 64, 600, 3000])) + 1, size=G)
        digits = int(rng.integers(0, 4))
        groups = [np.sort(np.round(inputs.lognormal_scores(5000 + 100 * case + g % 97, int(z)), digits)) for g, z in enumerate(sizes)]
        off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
        calib = np.concatenate(groups).astype(np.float32) if off[-1] else np.zeros(1, np.float32)
        Nc = int(rng.choice([1, 5, 127, 128, 129, 5000, 40001]))
        gid = rng.integers(0, G, size=Nc).astype(np.int32)
        if rng.random() < 0.6:
            gid = np.sort(gid)
        scores = np.round(inputs.lognormal_scores(9000 + case, Nc), digits)
        if Nc > 3:
            scores[int(rng.integers(0, Nc))] = np.nan
        shift = int(rng.integers(0, 4))
        numer, denom, p = poison((Nc + 4,), torch.int32), poison((Nc + 4,), torch.int32), poison((Nc + 4,), torch.float32)
        s, g = poison((Nc + 4,), torch.float32), poison((Nc + 4,), torch.int32)
        s[shift:shift + Nc] = dev(scores)
        g[shift:shift + Nc] = dev(gid)
        binding.conformal_rank_conditional(s[shift:shift + Nc], g[shift:shift + Nc], dev(calib), dev(off),
                                           numer[shift:shift + Nc], denom[shift:shift + Nc], p[shift:shift + Nc])
        torch.cuda.synchronize()
        wn, wd = orc.conformal_numer_conditional(scores, gid, groups)
        assert np.array_equal(host_u32(numer)[shift:shift + Nc], wn), (case, G, Nc, shift)
        assert np.array_equal(host_u32(denom)[shift:shift + Nc], wd), (case, G, Nc, shift)
        wp = (wn.astype(np.float64) / wd.astype(np.float64)).astype(np.float32)
        wp[wn == 0] = np.nan
        assert np.array_equal(f32_bits(p)[shift:shift + Nc], f32_bits(wp)), (case, G, Nc, shift)
    assert binding.last_device_status() == 0
