"""Pins for the oracle's extension functions: threshold form, conditional p-values, row-scaled scoring."""
import math

import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import inputs


@pytest.mark.parametrize("alpha", [0.01, 0.1, 0.25, 0.5, 0.9])
def test_threshold_is_kth_largest_and_matches_rank_rule_with_ties(alpha):
    calib = np.sort(np.round(inputs.lognormal_scores(1, 400), 1))            # heavy ties
    ka = orc.k_alpha(alpha, calib.size)
    tau = orc.threshold(calib, alpha)
    if ka >= 1:
        assert tau == sorted(calib.tolist())[-ka]
        assert tau == torch.kthvalue(torch.from_numpy(calib), calib.size - ka + 1).values.item()
    else:
        assert math.isinf(tau)
    s = np.concatenate([np.round(inputs.lognormal_scores(2, 3000), 1), np.array([np.nan, np.inf, -np.inf], np.float32)])
    by_rank, c_rank = orc.classify(orc.conformal_numer_sorted(s, calib), calib.size, alpha)
    by_tau, c_tau = orc.classify_by_threshold(s, tau)
    assert np.array_equal(by_rank, by_tau) and np.array_equal(c_rank, c_tau)
    # brute force of the rule itself: rejected iff fewer than k_alpha calibration scores are >= s
    for x, st in zip(s[:200].tolist(), by_tau[:200].tolist()):
        assert (st == 3) == (sum(1 for c in calib.tolist() if c >= x) < ka)


def test_threshold_small_buffer_cannot_reject():
    calib = np.arange(8, dtype=np.float32)
    assert math.isinf(orc.threshold(calib, 0.1))                             # floor(0.1 * 9) = 0
    st, counts = orc.classify_by_threshold(np.array([100.0, -1.0], np.float32), orc.threshold(calib, 0.1))
    assert st.tolist() == [2, 2]


def test_conditional_hand_example_and_reduction_to_marginal():
    groups = [np.array([1.0, 2.0, 3.0], np.float32), np.array([0.5, 0.5], np.float32), np.zeros(0, np.float32)]
    s = np.array([2.0, 2.5, 0.5, 0.6, 7.0, np.nan], np.float32)
    g = np.array([0, 0, 1, 1, 2, 0])
    numer, denom = orc.conformal_numer_conditional(s, g, groups)
    assert numer.tolist() == [3, 2, 3, 1, 1, 0]        # worked by hand from (1 + #{own group >= s})
    assert denom.tolist() == [4, 4, 3, 3, 1, 4]
    st, counts = orc.classify_conditional(numer, denom, 0.5)   # k = 2, 2, 1, 1, 0, 2
    assert st.tolist() == [2, 3, 2, 3, 2, 1]
    # one group only: the marginal p-value
    calib = inputs.lognormal_scores(3, 77)
    s = inputs.lognormal_scores(4, 50)
    numer, denom = orc.conformal_numer_conditional(s, np.zeros(50, np.int64), [calib])
    assert np.array_equal(numer, orc.conformal_numer_count(s, calib)) and np.all(denom == 78)
    a, _ = orc.classify_conditional(numer, denom, 0.2)
    b, _ = orc.classify(numer, 77, 0.2)
    assert np.array_equal(a, b)


def test_conditional_pvalues_uniform_within_group():
    """Proposition 2: within a group of size m with distinct exchangeable scores the numerator is uniform on 1..m+1."""
    m, reps = 15, 16000
    rng = np.random.default_rng(5)
    x = rng.standard_normal((reps, m + 1)).astype(np.float32) + rng.standard_normal((reps, 1)).astype(np.float32) * 5
    hist = np.zeros(m + 2, np.int64)
    numer, denom = orc.conformal_numer_conditional(x[:, 0], np.arange(reps), [x[r, 1:] for r in range(reps)])
    for v in numer:
        hist[v] += 1
    exp = reps / (m + 1)
    assert hist[0] == 0 and ((hist[1:] - exp) ** 2 / exp).sum() < 45.0     # 15 dof
    st, counts = orc.classify_conditional(numer, denom, 0.25)
    assert abs(counts[2] / reps - 4 / 16) < 0.02


def test_rms_inv_and_scaled_logprob_match_torch_rms_norm():
    M, d, V = 9, 32, 40
    Hb = inputs.f32_to_bf16_bits(np.random.default_rng(1).standard_normal((M, d)).astype(np.float32) * 3)
    Wb = inputs.lm_head(2, V, d)
    ids = inputs.zipf_ids(3, M, V)
    eps = 1e-6
    r = orc.rms_inv(Hb, eps)
    H = torch.from_numpy(inputs.bf16_bits_to_f32(Hb)).double()
    W = torch.from_numpy(inputs.bf16_bits_to_f32(Wb)).double()
    Hn = torch.nn.functional.rms_norm(H, (d,), eps=eps)
    np.testing.assert_allclose(r[:, None] * H.numpy(), Hn.numpy(), rtol=1e-13)
    nll = torch.nn.functional.cross_entropy(Hn @ W.T, torch.from_numpy(ids).long(), reduction="none")
    np.testing.assert_allclose(orc.token_logprob_scaled(Hb, Wb, ids, r), -nll.numpy(), atol=1e-12)
    # scale 1 is the unscaled function; a scale that sends logits to zero gives the uniform distribution
    np.testing.assert_allclose(orc.token_logprob_scaled(Hb, Wb, ids, np.ones(M)), orc.token_logprob(Hb, Wb, ids), atol=1e-13)
    np.testing.assert_allclose(orc.token_logprob_scaled(Hb, Wb, ids, np.zeros(M)), -math.log(V), atol=1e-13)


def test_takeover_ids_hand_example_library_routine_and_budget():
    # worked by hand: stages 2 3 1 3 3 2 -> the target takes over samples 1, 3 and 4; B = 3
    assert orc.takeover_ids(np.array([2, 3, 1, 3, 3, 2], np.uint8)).tolist() == [1, 3, 4]
    assert orc.takeover_ids(np.zeros(0, np.uint8)).size == 0
    assert orc.takeover_ids(np.array([1, 2, 2], np.uint8)).size == 0
    # against a library routine, and against the count classify reports as the budget
    calib = np.sort(inputs.lognormal_scores(5, 999))
    s = inputs.lognormal_scores(6, 5000)
    s[::97] = np.nan
    for alpha in (0.05, 0.25, 0.6):
        stage, counts = orc.classify(orc.conformal_numer_sorted(s, calib), calib.size, alpha)
        ids = orc.takeover_ids(stage)
        assert np.array_equal(ids, torch.nonzero(torch.from_numpy(stage) == 3).flatten().numpy())
        assert ids.size == counts[2]
        assert np.all(np.diff(ids) > 0)
        # exactly the samples with p <= alpha (Eq. prediction_set's complement), none without a score
        p = orc.pvalue(orc.conformal_numer_sorted(s, calib), calib.size)
        assert set(ids.tolist()) == {j for j in range(s.size) if p[j] <= alpha}
