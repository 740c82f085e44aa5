"""GPU parity: rank / p-value, classify and calibration update through the C-ABI, against the CPU
oracle, bit for bit, on the same fp32 score arrays."""
import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import binding, inputs
from tests.gpu_util import dev, f32_bits, host_u32, poison, workspace

pytestmark = pytest.mark.gpu


def gpu_rank(scores: np.ndarray, calib: np.ndarray, want_p=True):
    s, c = dev(scores), dev(calib) if calib.size else None
    numer = poison((scores.size,), torch.int32)
    p = poison((scores.size,), torch.float32) if want_p else None
    binding.conformal_rank(s, c, calib.size, numer, p)
    torch.cuda.synchronize()
    return host_u32(numer), (p.cpu().numpy() if want_p else None)


def gpu_classify(numer: np.ndarray, n: int, alpha: float):
    nm = dev(numer)
    stage = poison((numer.size,), torch.uint8)
    counts = poison((3,), torch.int32)
    binding.classify(nm, n, alpha, stage, counts)
    torch.cuda.synchronize()
    return stage.cpu().numpy(), host_u32(counts)


def gpu_update(calib: np.ndarray, new: np.ndarray, cap: int):
    buf = poison((cap,), torch.float32)
    buf[:calib.size] = dev(calib) if calib.size else buf[:0]
    ws = workspace(binding.calib_workspace_bytes(calib.size, new.size))
    n2 = binding.calib_update(buf, calib.size, dev(new) if new.size else None, ws)
    torch.cuda.synchronize()
    return buf.cpu().numpy(), n2


def check_rank(scores, calib):
    numer, p = gpu_rank(scores, calib)
    want = orc.conformal_numer_sorted(scores, calib)
    assert np.array_equal(numer, want)
    assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want, calib.size)))
    return numer


@pytest.mark.parametrize("Nc,n", [(1, 1), (5, 0), (1023, 7), (4096, 256), (4099, 8192), (70001, 8193),
                                   (33333, 65536), (20011, 327680), (1000, 1000001)])
def test_rank_pvalue_bit_exact(Nc, n):
    scores = inputs.lognormal_scores(100 + Nc, Nc)
    calib = np.sort(inputs.lognormal_scores(200 + n, n))
    numer = check_rank(scores, calib)
    # sampled outputs against the literal double-sum definition
    idx = np.random.default_rng(0).choice(Nc, size=min(Nc, 64), replace=False)
    assert np.array_equal(numer[idx], orc.conformal_numer_count(scores[idx], calib))


def test_rank_ties_extremes_and_special_values():
    calib = np.sort(np.round(inputs.lognormal_scores(1, 50000), 1))     # heavy ties
    scores = np.concatenate([np.round(inputs.lognormal_scores(2, 9000), 1), calib[::97],
                             np.array([0.0, -0.0, -1.0, 1e30, np.inf, -np.inf, np.nan], np.float32)])
    check_rank(scores, calib)
    calib = orc.calib_update(np.zeros(0, np.float32),
                             np.array([-np.inf, -1.0, -0.0, 0.0, 5.0, np.inf, np.nan, np.nan], np.float32))
    scores = np.array([np.nan, 0.0, -0.0, np.inf, -np.inf, 6.0, 5.0, -1.0], np.float32)
    numer = check_rank(scores, calib)
    assert np.array_equal(numer, orc.conformal_numer_count(scores, calib))
    # every score of the buffer ranked against itself: n - i + 1 for distinct values
    calib = np.unique(inputs.lognormal_scores(3, 20000))
    numer, _ = gpu_rank(calib, calib)
    assert np.array_equal(numer, np.arange(calib.size + 1, 1, -1, dtype=np.uint32))


@pytest.mark.parametrize("n", [2, 4096, 8191, 8192, 70000])
def test_rank_many_candidates_tied_clustered_and_special_data(n):
    """Many candidates against plain, heavily tied, clustered (outliers), constant and special-valued buffers."""
    Nc = (1 << 17) + 37
    base = inputs.lognormal_scores(700 + n, n)
    cases = {
        "plain": base,
        "ties": np.round(base, 1),
        "outliers": np.concatenate([base[: n - 2], np.array([1e30, -1e30], np.float32)]) if n > 2 else base,
        "constant": np.full(n, 2.5, np.float32),
        "special": np.concatenate([base[: max(n - 5, 0)], np.array([np.inf, -np.inf, np.nan, 0.0, -0.0], np.float32)[: min(n, 5)]]),
    }
    scores = np.concatenate([inputs.lognormal_scores(800 + n, Nc - 8),
                             np.array([0.0, -0.0, 2.5, np.inf, -np.inf, np.nan, 1e30, -1e30], np.float32)])
    for name, vals in cases.items():
        calib = orc.calib_update(np.zeros(0, np.float32), vals)
        numer, p = gpu_rank(scores, calib)
        assert np.array_equal(numer, orc.conformal_numer_sorted(scores, calib)), name
        idx = np.concatenate([np.arange(Nc - 8, Nc), np.arange(0, Nc - 8, 4099)])
        assert np.array_equal(numer[idx], orc.conformal_numer_count(scores[idx], calib)), name


@pytest.mark.parametrize("Nc,n", [(1 << 16, 1), ((1 << 16) + 3, 3), (1 << 18, 1000), (300007, 8191), (70001, 4096)])
def test_rank_bucket_form_bit_exact(Nc, n):
    """Many candidates against a small buffer take the bucket form of the rank kernel: smooth data (nearly every
    bucket holds at most one entry), then data packed into a sliver of the key range beside far outliers (most
    candidates search inside one bucket), with and without the p-value output and with fused thresholds."""
    smooth = np.sort(inputs.lognormal_scores(40 + n, n))
    packed = np.float32(1.0) + np.float32(1e-4) * inputs.lognormal_scores(41 + n, n)
    if n >= 3:
        packed[:2] = np.array([-3e38, 3e38], np.float32)
    packed = np.sort(packed)
    for calib, scores in ((smooth, inputs.lognormal_scores(42 + Nc, Nc)),
                          (packed, np.float32(1.0) + np.float32(1e-4) * inputs.lognormal_scores(43 + Nc, Nc))):
        scores[:6] = np.array([np.nan, -np.inf, np.inf, 0.0, -0.0, calib[n // 2]], np.float32)
        numer = check_rank(scores, calib)
        idx = np.concatenate([np.arange(6), np.arange(6, Nc, 2503)])
        assert np.array_equal(numer[idx], orc.conformal_numer_count(scores[idx], calib))
        numer_only, _ = gpu_rank(scores, calib, want_p=False)
        assert np.array_equal(numer_only, numer)
    Nf = Nc - Nc % 16
    alphas = (0.05, 0.1, 0.2)
    s, c = dev(scores[:Nf]), dev(calib)
    out_numer, p = poison((Nf,), torch.int32), poison((Nf,), torch.float32)
    stage, counts = poison((3, Nf), torch.uint8), poison((3, 3), torch.int32)
    binding.rank_classify(s, c, n, alphas, out_numer, p, stage, counts)
    torch.cuda.synchronize()
    assert np.array_equal(host_u32(out_numer), numer[:Nf])
    for a, alpha in enumerate(alphas):
        want_stage, want_counts = orc.classify(numer[:Nf], n, alpha)
        assert np.array_equal(stage[a].cpu().numpy(), want_stage)
        assert np.array_equal(host_u32(counts[a]), want_counts)


def test_rank_buffer_not_32_byte_aligned():
    # the kernel's 256-bit loads need a 32-byte aligned buffer; any other 4-byte aligned pointer takes the scalar path
    n, Nc = 100000, 1 << 17
    calib = np.sort(inputs.lognormal_scores(31, n))
    scores = inputs.lognormal_scores(32, Nc)
    want = orc.conformal_numer_sorted(scores, calib)
    for shift in (0, 1, 3, 8):
        buf = torch.empty(n + 16, device="cuda")
        buf[shift:shift + n] = dev(calib)
        numer = poison((Nc,), torch.int32)
        binding.conformal_rank(dev(scores), buf[shift:], n, numer, None)
        torch.cuda.synchronize()
        assert np.array_equal(host_u32(numer), want), shift


def test_rank_without_pvalue_output_and_empty_input():
    calib = np.sort(inputs.lognormal_scores(5, 300))
    scores = inputs.lognormal_scores(6, 77)
    numer, _ = gpu_rank(scores, calib, want_p=False)
    assert np.array_equal(numer, orc.conformal_numer_sorted(scores, calib))
    binding.conformal_rank(torch.empty(0, device="cuda"), dev(calib), calib.size, torch.empty(0, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("alpha", [0.05, 0.1, 0.2, 0.25, 0.4, 0.999])
@pytest.mark.parametrize("Nc,n", [(3, 9), (4096 + 5, 255), (100000, 65536)])
def test_classify_bit_exact(alpha, Nc, n):
    rng = np.random.default_rng(Nc + n)
    numer = rng.integers(0, n + 2, size=Nc).astype(np.uint32)
    ka = orc.k_alpha(alpha, n)
    numer[: min(Nc, 3)] = np.array([ka, ka + 1, 0], np.uint32)[: min(Nc, 3)]     # both sides of the threshold
    stage, counts = gpu_classify(numer, n, alpha)
    want_stage, want_counts = orc.classify(numer, n, alpha)
    assert np.array_equal(stage, want_stage)
    assert np.array_equal(counts, want_counts)


def test_classify_boundary_cases_and_no_counts():
    stage, counts = gpu_classify(np.array([1, 2], np.uint32), 9, 0.1)     # alpha (n + 1) = 1 exactly
    assert stage.tolist() == [3, 2] and counts.tolist() == [0, 1, 1]
    stage, counts = gpu_classify(np.array([1, 2, 9], np.uint32), 8, 0.1)  # k_alpha = 0: nobody rejected
    assert stage.tolist() == [2, 2, 2] and counts.tolist() == [0, 3, 0]
    numer = dev(np.arange(40, dtype=np.uint32))
    stage = poison((40,), torch.uint8)
    binding.classify(numer, 50, 0.25, stage, None)
    torch.cuda.synchronize()
    assert np.array_equal(stage.cpu().numpy(), orc.classify(np.arange(40, dtype=np.uint32), 50, 0.25)[0])
    counts = poison((3,), torch.int32)
    binding.classify(numer[:0], 50, 0.25, stage[:0], counts)              # empty input still zeroes the counts
    torch.cuda.synchronize()
    assert host_u32(counts).tolist() == [0, 0, 0]


@pytest.mark.parametrize("n,k", [(0, 1), (0, 300), (1, 1), (256, 8), (4096, 64), (1000, 4097), (65536, 4096),
                                  (323584, 4096), (5000, 16384), (100, 40000), (7, 0),
                                  (602112, 4096), (602113, 4096), (700000, 100), (20, 16385),
                                  (20000, 1000), (28672, 3000), (28673, 10), (28000, 4096), (5, 8)])
def test_calib_update_bit_exact(n, k):
    calib = np.sort(inputs.lognormal_scores(300 + n, n))
    new = inputs.lognormal_scores(400 + k, k)
    buf, n2 = gpu_update(calib, new, n + k + 5)
    assert n2 == n + k
    want = orc.calib_update(calib, new)
    assert np.array_equal(f32_bits(buf[:n2]), f32_bits(want))
    assert np.all(f32_bits(buf[n2:]) == 0xFFFFFFFF)     # nothing written past the new fill


@pytest.mark.parametrize("Nc,n,alphas", [(16, 9, (0.1,)), (4096 + 16, 255, (0.05, 0.1)), (1 << 20, 65536, (0.05, 0.1, 0.2)),
                                         (100000 - 100000 % 16, 327680, (0.05, 0.1, 0.2, 0.4)), (37, 500, (0.25,))])
def test_fused_rank_classify_equals_separate_calls(Nc, n, alphas):
    scores = inputs.lognormal_scores(500 + Nc, Nc)
    scores[: min(Nc, 2)] = np.array([np.nan, -1.0], np.float32)[: min(Nc, 2)]
    calib = np.sort(inputs.lognormal_scores(600 + n, n))
    s, c = dev(scores), dev(calib)
    numer = poison((Nc,), torch.int32)
    p = poison((Nc,), torch.float32)
    stage = poison((len(alphas), Nc), torch.uint8)
    counts = poison((len(alphas), 3), torch.int32)
    binding.rank_classify(s, c, n, alphas, numer, p, stage, counts)
    torch.cuda.synchronize()
    want_numer = orc.conformal_numer_sorted(scores, calib)
    assert np.array_equal(host_u32(numer), want_numer)
    assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want_numer, n)))
    for a, alpha in enumerate(alphas):
        want_stage, want_counts = orc.classify(want_numer, n, alpha)
        assert np.array_equal(stage[a].cpu().numpy(), want_stage)
        assert np.array_equal(host_u32(counts[a]), want_counts)
        # and byte for byte what the two separate entry points give
        st2, c2 = gpu_classify(host_u32(numer), n, alpha)
        assert np.array_equal(stage[a].cpu().numpy(), st2) and np.array_equal(host_u32(counts[a]), c2)


def test_calib_update_duplicates_and_special_values():
    calib = orc.calib_update(np.zeros(0, np.float32), np.round(inputs.lognormal_scores(1, 3000), 1))
    weird_nan = np.array([0x7F800001, 0xFFC00123], np.uint32).view(np.float32)
    new = np.concatenate([np.round(inputs.lognormal_scores(2, 500), 1),
                          np.array([-0.0, 0.0, np.inf, -np.inf, 3.0, 3.0], np.float32), weird_nan])
    buf, n2 = gpu_update(calib, new, calib.size + new.size)
    assert np.array_equal(f32_bits(buf[:n2]), f32_bits(orc.calib_update(calib, new)))
    # a second insert on top of a buffer that already holds NaNs
    buf2, n3 = gpu_update(buf[:n2], new, n2 + new.size)
    assert np.array_equal(f32_bits(buf2[:n3]), f32_bits(orc.calib_update(buf[:n2], new)))


def test_calib_update_small_in_place_path_special_values():
    # few new scores into a small buffer: the single-block in-place kernel; ties, zeros, infinities, NaNs
    calib = orc.calib_update(np.zeros(0, np.float32), np.concatenate(
        [np.round(inputs.lognormal_scores(1, 2000), 1), np.array([np.nan, np.inf, -np.inf, -0.0], np.float32)]))
    weird_nan = np.array([0x7F800001, 0xFFC00123], np.uint32).view(np.float32)
    new = np.concatenate([np.round(inputs.lognormal_scores(2, 40), 1),
                          np.array([-0.0, 0.0, np.inf, -np.inf, 3.0, 3.0], np.float32), weird_nan])
    buf, n2 = gpu_update(calib, new, calib.size + new.size + 3)
    assert np.array_equal(f32_bits(buf[:n2]), f32_bits(orc.calib_update(calib, new)))
    assert np.all(f32_bits(buf[n2:]) == 0xFFFFFFFF)
    # a non-canonical old buffer (-0.0 stored) is canonicalised on the way
    old = np.array([-1.0, -0.0, 0.0, 2.0], np.float32)
    buf, n2 = gpu_update(old, np.array([1.0], np.float32), 5)
    assert np.array_equal(f32_bits(buf[:n2]), f32_bits(orc.calib_update(old, np.array([1.0], np.float32))))


def test_calib_update_capacity_error_leaves_buffer_untouched():
    buf = dev(np.sort(inputs.lognormal_scores(1, 16)))
    before = buf.clone()
    ws = workspace(binding.calib_workspace_bytes(16, 4))
    with pytest.raises(binding.AttsError) as e:
        binding.calib_update(buf, 16, dev(inputs.lognormal_scores(2, 4)), ws)
    assert e.value.status == 5
    torch.cuda.synchronize()
    assert torch.equal(buf, before)


def test_conformal_stress_sequence_bit_exact():
    """The conformal-only workload at reduced length: rank, classify at three alphas, merge-insert, repeated,
    every step's outputs against the oracle."""
    cfg = inputs.CONFORMAL_STRESS
    Nc, n0, k, steps = cfg["Nc"], cfg["n0"], cfg["k"], 6
    scores = inputs.lognormal_scores(inputs.BASE_SEED + 1, Nc)
    calib = np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, n0))
    cap = n0 + k * steps
    buf = poison((cap,), torch.float32)
    buf[:n0] = dev(calib)
    s_dev = dev(scores)
    numer = poison((Nc,), torch.int32)
    p = poison((Nc,), torch.float32)
    stage = poison((Nc,), torch.uint8)
    counts = poison((3,), torch.int32)
    ws = workspace(binding.calib_workspace_bytes(cap, k))
    n = n0
    stage_f = poison((len(cfg["alphas"]), Nc), torch.uint8)
    counts_f = poison((len(cfg["alphas"]), 3), torch.int32)
    for t in range(steps):
        binding.rank_classify(s_dev, buf, n, cfg["alphas"], numer, p, stage_f, counts_f)
        fused = (host_u32(numer).copy(), stage_f.cpu().numpy().copy(), host_u32(counts_f).copy())
        numer.view(torch.uint8).fill_(0xFF)
        binding.conformal_rank(s_dev, buf, n, numer, p)
        want_numer = orc.conformal_numer_sorted(scores, calib)
        assert np.array_equal(host_u32(numer), want_numer)
        assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want_numer, n)))
        assert np.array_equal(fused[0], want_numer)
        for a, alpha in enumerate(cfg["alphas"]):
            binding.classify(numer, n, alpha, stage, counts)
            want_stage, want_counts = orc.classify(want_numer, n, alpha)
            assert np.array_equal(stage.cpu().numpy(), want_stage)
            assert np.array_equal(host_u32(counts), want_counts)
            assert np.array_equal(fused[1][a], want_stage) and np.array_equal(fused[2][a], want_counts)
        new = inputs.lognormal_scores(inputs.BASE_SEED + 3 + t, k)
        n = binding.calib_update(buf, n, dev(new), ws)
        calib = orc.calib_update(calib, new)
        assert n == calib.size
        assert np.array_equal(f32_bits(buf[:n]), f32_bits(calib))
    assert binding.last_device_status() == 0


def test_randomised_sizes_and_value_mixes():
    """Thirty random problems: random sizes around the kernels' mode switches, values rounded to force ties,
    a sprinkling of special values; every output compared with the oracle bit for bit."""
    rng = np.random.default_rng(20240607)
    pool = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-38, -1e-38, 3.0], np.float32)
    for case in range(30):
        n = int(rng.choice([0, 1, 2, 255, 8190, 8191, 8192, 20000, 28672, 28673, 70001]))
        k = int(rng.choice([0, 1, 7, 64, 500, 4096, 4097]))
        Nc = int(rng.choice([1, 3, 4, 1000, 4095, 65535, 65536, 131072 + 5]))
        digits = int(rng.choice([1, 3, 6]))
        calib_raw = np.round(inputs.lognormal_scores(1000 + case, n), digits)
        new = np.round(inputs.lognormal_scores(2000 + case, k), digits)
        scores = np.round(inputs.lognormal_scores(3000 + case, Nc), digits)
        for arr in (calib_raw, new, scores):
            if arr.size >= 4 and rng.random() < 0.5:
                idx = rng.choice(arr.size, size=min(arr.size, 6), replace=False)
                arr[idx] = rng.choice(pool, size=idx.size)
        calib = orc.calib_update(np.zeros(0, np.float32), calib_raw)
        numer, p = gpu_rank(scores, calib)
        want = orc.conformal_numer_sorted(scores, calib)
        assert np.array_equal(numer, want), (case, n, Nc)
        assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want, n))), (case, n, Nc)
        alpha = float(rng.choice([0.05, 0.1, 0.37, 0.5]))
        stage, counts = gpu_classify(numer, n, alpha)
        ws, wc = orc.classify(want, n, alpha)
        assert np.array_equal(stage, ws) and np.array_equal(counts, wc), (case, n, Nc, alpha)
        buf, n2 = gpu_update(calib, new, n + k + 2)
        assert n2 == n + k
        assert np.array_equal(f32_bits(buf[:n2]), f32_bits(orc.calib_update(calib, new))), (case, n, k)


def _index_for(calib_dev, n, cap=None):
    ix = workspace(binding.calib_index_bytes(cap if cap is not None else n))
    binding.calib_index_build(calib_dev, n, ix)
    return ix


@pytest.mark.parametrize("Nc,n", [(1 << 17, 8192), (100003, 8255), (1 << 16, 65536), (70001, 65543), (1 << 18, 327680),
                                   (16384, 524223), (20000, 100), (100, 70000), (0, 9000), (16384, 65527), (16384, 65528),
                                   (1 << 16, 524224), (1 << 15, 262143), (1 << 15, 262144), (1 << 15, 2097151),
                                   (1 << 15, 2097152), (1 << 15, 4193792), (1 << 15, 16776703), (1 << 15, 16777214)])
def test_indexed_rank_equals_definition_and_plain_call(Nc, n):
    """The indexed rank gives the numerators and p-value bits of the definition, on smooth data, on heavily tied data
    and with special values at both ends of the buffer, with and without fused thresholds."""
    for variant in ("smooth", "ties", "special"):
        raw = inputs.lognormal_scores(900 + n, n)
        scores = inputs.lognormal_scores(901 + Nc, Nc)
        if variant == "ties":
            raw, scores = np.round(raw, 1), np.round(scores, 1)
        if variant == "special":
            raw[:6] = np.array([-np.inf, -0.0, 0.0, np.inf, np.nan, np.nan], np.float32)
        if Nc >= 8:
            scores[:8] = np.array([np.nan, -np.inf, np.inf, 0.0, -0.0, raw[n // 2], 1e30, -1e30], np.float32)
        calib = orc.calib_update(np.zeros(0, np.float32), raw)
        c, s = dev(calib), dev(scores)
        ix = _index_for(c, n)
        numer, p = poison((Nc,), torch.int32), poison((Nc,), torch.float32)
        binding.rank_classify_indexed(s, c, n, ix, (), numer, p)
        torch.cuda.synchronize()
        want = orc.conformal_numer_sorted(scores, calib)
        assert np.array_equal(host_u32(numer), want), variant
        assert np.array_equal(f32_bits(p), f32_bits(orc.pvalue(want, n))), variant
        if Nc:
            idx = np.arange(0, Nc, max(Nc // 50, 1))
            assert np.array_equal(want[idx], orc.conformal_numer_count(scores[idx], calib)), variant
    Nf = Nc - Nc % 16
    if Nf:
        alphas = (0.05, 0.1, 0.2)
        numer2, stage, counts = poison((Nf,), torch.int32), poison((3, Nf), torch.uint8), poison((3, 3), torch.int32)
        binding.rank_classify_indexed(s[:Nf], c, n, ix, alphas, numer2, None, stage, counts)
        torch.cuda.synchronize()
        assert np.array_equal(host_u32(numer2), want[:Nf])
        for a, alpha in enumerate(alphas):
            ws, wc = orc.classify(want[:Nf], n, alpha)
            assert np.array_equal(stage[a].cpu().numpy(), ws) and np.array_equal(host_u32(counts[a]), wc)
    assert binding.last_device_status() == 0


def test_indexed_update_sequence_keeps_buffer_and_index_in_step():
    """A growing buffer: every update through the indexed entry point leaves the oracle's buffer and an index with
    which the next rank is exact (small in-place path, general path, a slice-by-slice insert, an empty insert)."""
    Nc = 1 << 16
    scores = inputs.lognormal_scores(77, Nc)
    s = dev(scores)
    calib = np.sort(inputs.lognormal_scores(78, 5000))
    cap = 5000 + 64 + 4096 + 40000 + 0 + 3000 + 8
    buf = poison((cap,), torch.float32)
    buf[:calib.size] = dev(calib)
    ix = _index_for(buf, calib.size, cap)
    n = calib.size
    for step, k in enumerate((64, 4096, 40000, 0, 3000)):
        new = inputs.lognormal_scores(80 + step, k)
        ws = workspace(binding.calib_workspace_bytes(n, k))
        n2 = binding.calib_update_indexed(buf, n, dev(new) if k else None, ix, ws)
        calib = orc.calib_update(calib, new)
        assert n2 == calib.size
        n = n2
        numer = poison((Nc,), torch.int32)
        binding.rank_classify_indexed(s, buf, n, ix, (), numer)
        torch.cuda.synchronize()
        assert np.array_equal(f32_bits(buf[:n]), f32_bits(calib)), step
        assert np.array_equal(host_u32(numer), orc.conformal_numer_sorted(scores, calib)), step
    assert binding.last_device_status() == 0


def test_stale_index_is_refused_and_argument_errors():
    n, Nc = 20000, 1 << 15
    calib = np.sort(inputs.lognormal_scores(90, n + 64))
    c, s = dev(calib), dev(inputs.lognormal_scores(91, Nc))
    ix = _index_for(c, n, n + 64 + 5000)
    numer = poison((Nc,), torch.int32)
    binding.rank_classify_indexed(s, c, n + 64, ix, (), numer)           # index describes n, not n + 64
    with pytest.raises(binding.AttsError) as err:
        binding.last_device_status()
    assert err.value.status == 11
    assert np.all(host_u32(numer) == 0xFFFFFFFF)                         # nothing was written
    assert binding.last_device_status() == 0                             # the bit was cleared
    # an update through an index that does not describe the fill it starts from changes nothing and is reported
    buf = poison((n + 64 + 5000,), torch.float32)
    buf[:n + 64] = c
    new = dev(inputs.lognormal_scores(92, 5000))
    binding.calib_update_indexed(buf, n + 64, new, ix, workspace(binding.calib_workspace_bytes(n + 64, 5000)))
    with pytest.raises(binding.AttsError) as err:
        binding.last_device_status()
    assert err.value.status == 11
    assert np.array_equal(f32_bits(buf[:n + 64]), f32_bits(calib)) and np.all(f32_bits(buf[n + 64:]) == 0xFFFFFFFF)
    # the fill it does describe is still served, from the index's own copy of the buffer
    binding.rank_classify_indexed(s, c, n, ix, (), numer)
    torch.cuda.synchronize()
    assert np.array_equal(host_u32(numer), orc.conformal_numer_sorted(inputs.lognormal_scores(91, Nc), calib[:n]))
    with pytest.raises(binding.AttsError) as err:                        # index too small for this n
        binding.calib_index_build(c, n + 64, ix[:1024])
    assert err.value.status == 4


def test_indexed_update_may_overlap_the_rank_of_the_fill_it_starts_from():
    """Rank of fill n on one stream, the update n -> n + k on another, with no ordering between them: the rank sees the
    buffer as it was (ranks against the old fill), the update leaves the new one; the next rank waits for the update,
    the next update for this rank.  Several steps, every result against the oracle."""
    Nc, n, k, steps = 1 << 17, 90000, 4096, 5
    calib = np.sort(inputs.lognormal_scores(310, n))
    scores = inputs.lognormal_scores(311, Nc)
    news = [inputs.lognormal_scores(312 + t, k) for t in range(steps)]
    s, nws = dev(scores), [dev(x) for x in news]
    cap = n + k * steps
    buf = poison((cap,), torch.float32)
    buf[:n] = dev(calib)
    ix = _index_for(buf, n, cap)
    ws = workspace(binding.calib_workspace_bytes(cap, k))
    numers = [poison((Nc,), torch.int32) for _ in range(steps)]
    main, side = torch.cuda.current_stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    ranked, merged = [], []
    fill = n
    for t in range(steps):
        if t:
            main.wait_event(merged[t - 1])                   # the rank of fill n_t needs the update that produced it
        binding.rank_classify_indexed(s, buf, fill, ix, (), numers[t])
        ev = torch.cuda.Event()
        ev.record(main)
        ranked.append(ev)
        with torch.cuda.stream(side):
            if t:
                side.wait_event(ranked[t - 1])               # this update overwrites what the previous rank read
            fill = binding.calib_update_indexed(buf, fill, nws[t], ix, ws)
            ev = torch.cuda.Event()
            ev.record(side)
            merged.append(ev)
    torch.cuda.synchronize()
    want = calib
    for t in range(steps):
        assert np.array_equal(host_u32(numers[t]), orc.conformal_numer_sorted(scores, want)), t
        want = orc.calib_update(want, news[t])
    assert fill == cap and np.array_equal(f32_bits(buf), f32_bits(want))
    assert binding.last_device_status() == 0


@pytest.mark.parametrize("n,k", [(70000, 4096), (40000, 16384), (300000, 20000), (5000, 600), (0, 3000), (100000, 385)])
def test_update_with_skewed_batches(n, k):
    """New scores that all fall into one stretch of the buffer (beyond its largest entry, below its smallest, one
    repeated value, a narrow band, everything NaN): the block that owns that stretch sorts them all.  Plain and
    indexed update against the oracle."""
    calib = np.sort(inputs.lognormal_scores(400 + n, n))
    top = float(calib[-1]) if n else 1.0
    mid = float(calib[n // 2]) if n else 1.0
    batches = {
        "above": top + 1.0 + inputs.lognormal_scores(401, k),
        "below": -inputs.lognormal_scores(402, k),
        "equal": np.full(k, mid, np.float32),
        "band": (mid + 1e-4 * inputs.lognormal_scores(403, k)).astype(np.float32),
        "nan": np.full(k, np.nan, np.float32),
        "two_values": np.where(np.arange(k) % 2 == 0, np.float32(mid), np.float32(top + 2.0)).astype(np.float32),
    }
    for name, new in batches.items():
        new = new.astype(np.float32)
        want = orc.calib_update(calib, new)
        for indexed in (False, True):
            buf = poison((n + k + 5,), torch.float32)
            if n:
                buf[:n] = dev(calib)
            ws = workspace(binding.calib_workspace_bytes(n, k))
            if indexed:
                ix = _index_for(buf, n, n + k)
                n2 = binding.calib_update_indexed(buf, n, dev(new), ix, ws)
            else:
                n2 = binding.calib_update(buf, n, dev(new), ws)
            torch.cuda.synchronize()
            assert n2 == n + k
            assert np.array_equal(f32_bits(buf[:n2]), f32_bits(want)), (name, indexed)
            assert np.all(f32_bits(buf[n2:]) == 0xFFFFFFFF), (name, indexed)
    assert binding.last_device_status() == 0
