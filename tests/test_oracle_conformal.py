"""Pins for the conformal half of the CPU oracle (rank, p-value, stages, calibration update)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pvalue_worked_examples.txt")


def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            c, s, num, den, alpha, stage = [x.strip() for x in line.split("|")]
            rows.append((np.array([float(v) for v in c.split(",")], dtype=np.float32), float(s), int(num),
                         int(den), float(alpha), int(stage)))
    return rows


def test_hand_worked_examples():
    rows = _golden_rows()
    assert len(rows) >= 10
    for calib, s, num, den, alpha, stage in rows:
        sc = np.array([s], dtype=np.float32)
        assert orc.conformal_numer_count(sc, calib)[0] == num
        assert orc.conformal_numer_sorted(sc, np.sort(calib))[0] == num
        assert calib.size + 1 == den
        assert orc.pvalue(np.array([num], np.uint32), calib.size)[0] == np.float32(num / den)
        st, counts = orc.classify(np.array([num], np.uint32), calib.size, alpha)
        assert st[0] == stage
        assert counts[stage - 1] == 1 and counts.sum() == 1


def _python_numer(s, calib):
    return [1 + sum(1 for c in calib if (c >= x) or math.isnan(c)) if not math.isnan(x) else 0 for x in s]


@pytest.mark.parametrize("seed", range(4))
def test_count_and_sorted_agree_with_python_loop(seed):
    rng = np.random.default_rng(seed)
    n, Nc = int(rng.integers(0, 40)), 50
    calib = np.round(rng.standard_normal(n) * 2, 1).astype(np.float32)   # rounded: many ties
    s = np.round(rng.standard_normal(Nc) * 2, 1).astype(np.float32)
    want = _python_numer(s.tolist(), calib.tolist())
    assert orc.conformal_numer_count(s, calib).tolist() == want
    assert orc.conformal_numer_sorted(s, np.sort(calib)).tolist() == want


def test_rank_closed_forms():
    calib = np.sort(inputs.lognormal_scores(1, 500))
    assert np.unique(calib).size == calib.size
    n = calib.size
    # ranking the distinct sorted buffer against itself: numer(calib[i]) = n - i + 1
    assert orc.conformal_numer_sorted(calib, calib).tolist() == [n - i + 1 for i in range(n)]
    lo = np.array([calib[0] / 2, -1.0, -np.inf], np.float32)
    hi = np.array([calib[-1] * 2, np.inf], np.float32)
    assert orc.conformal_numer_sorted(lo, calib).tolist() == [n + 1] * 3      # p = 1
    assert orc.conformal_numer_sorted(hi, calib).tolist() == [1, 1]           # p = 1 / (n + 1)
    assert orc.pvalue(np.array([n + 1, 1], np.uint32), n).tolist() == [1.0, np.float32(1 / (n + 1))]
    # empty calibration set: numer 1, p = 1
    assert orc.conformal_numer_sorted(np.array([0.3], np.float32), np.zeros(0, np.float32)).tolist() == [1]
    assert orc.pvalue(np.array([1], np.uint32), 0)[0] == 1.0
    # monotone non-increasing in s
    s = np.sort(inputs.lognormal_scores(2, 2000))
    num = orc.conformal_numer_sorted(s, calib).astype(np.int64)
    assert np.all(np.diff(num) <= 0)


def test_rank_matches_torch_searchsorted():
    calib = np.sort(np.round(inputs.lognormal_scores(3, 3000), 2))   # with duplicates
    s = np.round(inputs.lognormal_scores(4, 5000), 2)
    idx = torch.searchsorted(torch.from_numpy(calib), torch.from_numpy(s), right=False).numpy()
    assert np.array_equal(orc.conformal_numer_sorted(s, calib), (calib.size - idx + 1).astype(np.uint32))
    # a candidate equal to a calibration value counts the whole tie block (indicator is "<=")
    calib = np.array([1, 2, 2, 2, 3], np.float32)
    assert orc.conformal_numer_sorted(np.array([2.0], np.float32), calib)[0] == 1 + 4
    assert orc.conformal_numer_count(np.array([2.0], np.float32), calib)[0] == 1 + 4


def test_special_values():
    calib = np.array([-np.inf, -1.0, -0.0, 0.0, 5.0, np.inf, np.nan, np.nan], np.float32)
    s = np.array([np.nan, 0.0, -0.0, np.inf, -np.inf, 6.0], np.float32)
    want = [0, 1 + 6, 1 + 6, 1 + 3, 1 + 8, 1 + 3]
    assert orc.conformal_numer_count(s, calib).tolist() == want
    assert orc.conformal_numer_sorted(s, calib).tolist() == want
    p = orc.pvalue(np.array(want, np.uint32), calib.size)
    assert math.isnan(p[0]) and p[4] == 1.0
    st, counts = orc.classify(np.array(want, np.uint32), calib.size, 0.5)   # k_alpha = 4
    assert st.tolist() == [1, 2, 2, 3, 2, 3]
    assert counts.tolist() == [1, 3, 2]


def test_pvalue_rounding_is_single_float32_division():
    n = 4096
    num = np.arange(1, n + 2, dtype=np.uint32)
    want = torch.from_numpy(num.astype(np.float32)) / torch.tensor(float(n + 1), dtype=torch.float32)
    assert np.array_equal(orc.pvalue(num, n), want.numpy())


def test_pvalues_uniform_under_exchangeability():
    """Proposition 1: with distinct exchangeable scores the numerator is uniform on {1..n+1}."""
    n, reps = 19, 20000
    rng = np.random.default_rng(123)
    x = rng.standard_normal((reps, n + 1)).astype(np.float32)
    hist = np.zeros(n + 2, dtype=np.int64)
    for r in range(reps):
        num = orc.conformal_numer_count(x[r, :1], x[r, 1:])[0]
        hist[num] += 1
    assert hist[0] == 0
    expected = reps / (n + 1)
    chi2 = ((hist[1:] - expected) ** 2 / expected).sum()
    assert chi2 < 50.0   # 19 degrees of freedom: P(chi2 > 50) ~ 1e-4
    # and therefore P(p <= alpha) = floor(alpha (n + 1)) / (n + 1) <= alpha
    for alpha in (0.05, 0.1, 0.25, 0.4):
        ka = orc.k_alpha(alpha, n)
        rate = hist[1:ka + 1].sum() / reps
        assert abs(rate - ka / (n + 1)) < 5 * math.sqrt(alpha / reps) + 1e-9
        assert ka / (n + 1) <= alpha + 1e-12


@pytest.mark.parametrize("alpha", [0.05, 0.1, 0.2, 0.25, 0.4])
def test_rejection_rate_tracks_alpha(alpha):
    """Take-over fraction ~ alpha on exchangeable synthetic scores (synthetic analogue of Fig. budget)."""
    n, Nc = 4096, 200000
    calib = np.sort(inputs.lognormal_scores(10, n))
    s = inputs.lognormal_scores(11, Nc)
    stage, counts = orc.classify(orc.conformal_numer_sorted(s, calib), n, alpha)
    rate = counts[2] / Nc
    tol = 5 * math.sqrt(alpha * (1 - alpha) / (n + 2)) + 1 / (n + 1) + 5 * math.sqrt(alpha * (1 - alpha) / Nc)
    assert abs(rate - alpha) <= tol
    assert counts.sum() == Nc and counts[0] == 0


def test_k_alpha_boundaries():
    assert orc.k_alpha(0.1, 9) == 1        # alpha (n + 1) = 1 exactly
    assert orc.k_alpha(0.25, 3) == 1       # 0.25 * 4 = 1
    assert orc.k_alpha(0.1, 8) == 0        # n + 1 < 1 / alpha: nobody can be rejected
    assert orc.k_alpha(0.05, 65536) == 3276
    assert orc.k_alpha(0.2, 65536) == 13107
    st, counts = orc.classify(np.array([1, 2], np.uint32), 9, 0.1)
    assert st.tolist() == [3, 2]           # p = 0.1 = alpha is rejected, p = 0.2 accepted
    st, counts = orc.classify(np.array([1, 2, 9], np.uint32), 8, 0.1)
    assert st.tolist() == [2, 2, 2] and counts.tolist() == [0, 3, 0]


def test_classify_equals_classic_threshold_form_and_is_monotone_in_alpha():
    """For distinct scores, stage 3 <=> s is strictly above the k_alpha-th largest calibration score
    (the quantile-threshold construction of the classic set-up, Eqs. quantile / pred_set)."""
    n = 999
    calib = np.sort(inputs.lognormal_scores(20, n))
    s = inputs.lognormal_scores(21, 5000)
    num = orc.conformal_numer_sorted(s, calib)
    prev = -1
    for alpha in (0.01, 0.05, 0.1, 0.3, 0.77):
        ka = orc.k_alpha(alpha, n)
        stage, counts = orc.classify(num, n, alpha)
        tau = calib[n - ka] if ka >= 1 else np.inf      # k_alpha-th largest
        assert np.array_equal(stage == 3, s > tau)
        assert counts[2] >= prev
        prev = counts[2]
        assert counts.sum() == s.size


def test_calib_update_matches_torch_sort_and_preserves_multiset():
    calib = np.sort(inputs.lognormal_scores(30, 1000))
    new = inputs.lognormal_scores(31, 333)
    got = orc.calib_update(calib, new)
    want = torch.sort(torch.cat([torch.from_numpy(calib), torch.from_numpy(new)])).values.numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(np.sort(got.view(np.uint32)), np.sort(np.concatenate([calib, new]).view(np.uint32)))
    # k = 0 changes nothing; one batch == two halves
    assert np.array_equal(orc.calib_update(calib, np.zeros(0, np.float32)), calib)
    two = orc.calib_update(orc.calib_update(calib, new[:100]), new[100:])
    assert np.array_equal(two.view(np.uint32), got.view(np.uint32))
    # empty buffer: plain sort
    assert np.array_equal(orc.calib_update(np.zeros(0, np.float32), new), np.sort(new))


def test_calib_update_canonicalises_zero_and_nan():
    weird_nan = np.array([0x7F800001, 0xFFC00123], np.uint32).view(np.float32)
    new = np.concatenate([np.array([-0.0, 3.0, -np.inf, 0.0, np.inf], np.float32), weird_nan])
    got = orc.calib_update(np.array([-1.0, 1.0], np.float32), new)
    want_bits = np.array([-np.inf, -1.0, 0.0, 0.0, 1.0, 3.0, np.inf], np.float32).view(np.uint32).tolist()
    want_bits += [0x7FC00000, 0x7FC00000]
    assert got.view(np.uint32).tolist() == want_bits


def test_rank_before_insert_semantics():
    """A batch is ranked against the buffer as it was, then inserted: afterwards each of its scores
    finds itself in the buffer, so its numerator grows by the number of batch scores >= it."""
    calib = np.sort(inputs.lognormal_scores(40, 256))
    batch = inputs.lognormal_scores(41, 8)
    before = orc.conformal_numer_sorted(batch, calib).astype(np.int64)
    after = orc.conformal_numer_sorted(batch, orc.calib_update(calib, batch)).astype(np.int64)
    extra = np.array([(batch >= b).sum() for b in batch])
    assert np.array_equal(after - before, extra)
