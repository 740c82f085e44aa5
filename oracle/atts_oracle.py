"""CPU oracle for the ATTS verification hot path (numpy, float64).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
path computes, written from the paper's definitions.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it; the library's
product path never does, and this file imports nothing from the CUDA package.

What is computed, and where the paper defines it:

* ``token_logprob``  - log q_t(y_i | prefix): the target model's logits for a
  draft token are turned into a log-probability by the full softmax over the
  vocabulary (Verification paragraph of Sec. 3.3; the loss l of Eq. 2 is the
  negative log-likelihood).
* ``sample_score``   - the unnormalised conformity score s = -l of a draft
  sample (Sec. 3.2, "Online Calibration", the unnumbered equation before
  Eq. p-value).  Reading adopted: the score handed to the conformal layer is
  the NLL of the draft sample under the target, averaged over its tokens
  (mode 0); sum and the opposite sign are modes 1-3.
* ``conformal_numer_*`` / ``pvalue`` - the marginal conformal p-value,
  Eq. (p-value) and Proposition 1: (1 + #{calibration scores >= s}) / (n + 1).
* ``k_alpha`` / ``classify`` - accept iff p > alpha (Eq. prediction_set and
  the sentence after Eq. p-value); the three pipeline stages of Sec. 3.3.
* ``calib_update``   - the online calibration set grows by the new scores
  (Sec. 3.2, "Online Calibration"); it is kept as an ascending array.

Parity pins (tests/test_oracle_*.py): every function here is pinned to
something other than itself - brute-force softmax in Python floats, closed
forms, torch's float64 cross_entropy / searchsorted / sort, the uniformity of
p-values stated by Proposition 1, and hand-worked examples under
tests/golden/.  No function is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

STAGE_DRAFT = 1      # nothing was verified (no score): the sample stays a draft
STAGE_ACCEPTED = 2   # verified, p > alpha: the draft continuation is kept
STAGE_TARGET = 3     # verified, p <= alpha: the target model takes over

CANONICAL_NAN_BITS = np.uint32(0x7FC00000)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float64, exactly (bf16 is the top half of a float32)."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def logits(hidden_bits: np.ndarray, lm_head_bits: np.ndarray, vocab_slab: int = 8192) -> np.ndarray:
    """z[i, v] = sum_k h[i, k] * w[v, k] in float64 (Sec. 3.3, Verification: "computing the logits").

    The matrix product is a library dgemm.  It is issued per slab of vocabulary
    rows only to bound the memory of the float64 copy of W; every logit is still
    one plain dot product over the whole hidden dimension.
    """
    H = bf16_bits_to_f64(hidden_bits)
    V = lm_head_bits.shape[0]
    z = np.empty((H.shape[0], V), dtype=np.float64)
    for a in range(0, V, vocab_slab):
        b = min(a + vocab_slab, V)
        z[:, a:b] = H @ bf16_bits_to_f64(lm_head_bits[a:b]).T
    return z


def token_logprob(hidden_bits: np.ndarray, lm_head_bits: np.ndarray, token_ids: np.ndarray) -> np.ndarray:
    """log-softmax of each row's logits at that row's draft token, float64.

    logp_i = z[i, y_i] - (max_v z[i, v] + log sum_v exp(z[i, v] - max_v z[i, v])).
    No temperature, bias or soft-cap; every vocabulary row takes part.
    A token id outside [0, V) is a caller error and raises.
    """
    ids = np.asarray(token_ids, dtype=np.int64)
    V = lm_head_bits.shape[0]
    if ids.size and (ids.min() < 0 or ids.max() >= V):
        raise ValueError("token id out of range")
    z = logits(hidden_bits, lm_head_bits)
    mx = z.max(axis=1)
    lse = mx + np.log(np.exp(z - mx[:, None]).sum(axis=1))
    return z[np.arange(z.shape[0]), ids] - lse


def sample_score(token_logprob_: np.ndarray, seg_offsets: np.ndarray, mode: int = 0) -> np.ndarray:
    """Per-sample score from token log-probs (Sec. 3.2: s = -l, l the NLL of the sample).

    Sample k owns tokens [o_k, o_{k+1}).  mode 0: mean NLL (default reading);
    1: summed NLL; 2: mean log-likelihood; 3: summed log-likelihood.
    An empty sample has no score: NaN.
    """
    lp = np.asarray(token_logprob_, dtype=np.float64)
    off = np.asarray(seg_offsets, dtype=np.int64)
    S = off.size - 1
    out = np.full(S, np.nan, dtype=np.float64)
    for k in range(S):
        a, b = int(off[k]), int(off[k + 1])
        if b <= a:
            continue
        tot = float(np.sum(lp[a:b]))
        if mode in (0, 2):
            tot /= (b - a)
        out[k] = -tot if mode in (0, 1) else tot
    return out


def _canonical(x: np.ndarray) -> np.ndarray:
    """float32 copy with -0.0 -> +0.0 and every NaN -> the one quiet NaN 0x7FC00000."""
    x = np.array(x, dtype=np.float32, copy=True)
    x[x == 0.0] = np.float32(0.0)
    bits = x.view(np.uint32)
    bits[np.isnan(x)] = CANONICAL_NAN_BITS
    return x


def conformal_numer_count(scores: np.ndarray, calib: np.ndarray) -> np.ndarray:
    """Numerator of Eq. (p-value) by the literal double sum: 1 + #{i : s <= calib_i}.

    The calibration scores need not be sorted here.  Readings: a tie counts
    (the indicator is "<="); a NaN calibration score counts for every candidate
    (it behaves like +infinity, which only makes p larger, i.e. conservative);
    a NaN candidate has no score: numerator 0.
    """
    s = np.asarray(scores, dtype=np.float32)
    c = np.asarray(calib, dtype=np.float32)
    out = np.zeros(s.size, dtype=np.uint32)
    c_nan = int(np.isnan(c).sum())
    c_ok = c[~np.isnan(c)]
    for j in range(s.size):
        if np.isnan(s[j]):
            continue
        out[j] = 1 + int(np.count_nonzero(s[j] <= c_ok)) + c_nan
    return out


def conformal_numer_sorted(scores: np.ndarray, calib_sorted: np.ndarray) -> np.ndarray:
    """The same numerator when the calibration array is ascending (NaNs last).

    #{i : calib_i >= s} = n - (number of calib_i < s) = n - lower_bound(calib, s);
    the lower bound is numpy's searchsorted (a library binary search).
    """
    s = np.asarray(scores, dtype=np.float32)
    c = np.asarray(calib_sorted, dtype=np.float32)
    n = c.size
    n_fin = n - int(np.isnan(c).sum())
    below = np.searchsorted(c[:n_fin], s, side="left")
    numer = (n - below + 1).astype(np.uint32)
    numer[np.isnan(s)] = 0
    return numer


def pvalue(numer: np.ndarray, n: int) -> np.ndarray:
    """p = numer / (n + 1) (Eq. p-value), rounded once to float32; no score -> NaN."""
    num = np.asarray(numer, dtype=np.uint32)
    p = (num.astype(np.float64) / float(n + 1)).astype(np.float32)
    p[num == 0] = np.float32(np.nan)
    return p


def k_alpha(alpha: float, n: int) -> int:
    """Largest numerator that is still rejected: p <= alpha <=> numer <= floor(alpha * (n + 1))."""
    return int(np.floor(np.float64(alpha) * np.float64(n + 1)))


def classify(numer: np.ndarray, n: int, alpha: float):
    """Ordinal stage per sample and the three stage counts.

    A candidate is accepted iff p > alpha (Eq. prediction_set); the target model
    takes over the others (Sec. 3.3).  Stage 1: no score; 2: accepted; 3: target.
    The count of stage 3 is the budget B of the "Budget Prediction" paragraph.
    """
    num = np.asarray(numer, dtype=np.uint32)
    ka = k_alpha(alpha, n)
    stage = np.full(num.size, STAGE_ACCEPTED, dtype=np.uint8)
    stage[num == 0] = STAGE_DRAFT
    stage[(num >= 1) & (num <= ka)] = STAGE_TARGET
    counts = np.array([(stage == 1).sum(), (stage == 2).sum(), (stage == 3).sum()], dtype=np.uint32)
    return stage, counts


def takeover_ids(stage: np.ndarray) -> np.ndarray:
    """The samples the target model takes over in this turn ("Budget Prediction", Sec. 3.2: the B candidates that
    are rejected; "Target Sampling", Sec. 3.3: the candidates the target continues): the positions whose stage is 3,
    in input order.  Their number is the budget B."""
    out = []
    for j, st in enumerate(np.asarray(stage, dtype=np.uint8).tolist()):
        if st == STAGE_TARGET:
            out.append(j)
    return np.array(out, dtype=np.int32)


def calib_update(calib_sorted: np.ndarray, new_scores: np.ndarray) -> np.ndarray:
    """Online calibration: the set grows by the new scores and stays ascending (Sec. 3.2).

    Grow-only multiset, no eviction.  Values are canonicalised first (-0 -> +0,
    one NaN pattern) so that equal values are equal bit patterns and the result
    is unique; numpy's sort puts NaNs last.
    """
    allv = np.concatenate([_canonical(calib_sorted), _canonical(new_scores)])
    return np.sort(allv, kind="stable")


# ----------------------------------------------------------------------------------------------
# Extensions beyond the marginal path ("next" rows): threshold form, conditional coverage, row scale.
# ----------------------------------------------------------------------------------------------

def threshold(calib_sorted: np.ndarray, alpha: float) -> np.float32:
    """Score threshold equivalent to the rank rule: tau = the k_alpha-th largest calibration score.

    numer <= k_alpha  <=>  fewer than k_alpha calibration scores are >= s  <=>  s > (k_alpha-th largest), ties
    included; this is the quantile-threshold construction of the classic set-up (Eqs. quantile / pred_set) read
    for the rejection side.  k_alpha = 0 (nobody can be rejected) gives +inf.
    """
    c = np.asarray(calib_sorted, dtype=np.float32)
    ka = k_alpha(alpha, c.size)
    if ka < 1:
        return np.float32(np.inf)
    return c[c.size - ka]


def classify_by_threshold(scores: np.ndarray, tau: np.float32):
    """Stage from one comparison per sample: 3 if s > tau, else 2; a NaN score is stage 1."""
    s = np.asarray(scores, dtype=np.float32)
    stage = np.full(s.size, STAGE_ACCEPTED, dtype=np.uint8)
    with np.errstate(invalid="ignore"):
        stage[s > np.float32(tau)] = STAGE_TARGET
    stage[np.isnan(s)] = STAGE_DRAFT
    counts = np.array([(stage == 1).sum(), (stage == 2).sum(), (stage == 3).sum()], dtype=np.uint32)
    return stage, counts


def conformal_numer_conditional(scores: np.ndarray, group_ids: np.ndarray, calib_groups):
    """Conditional conformal p-value (Proposition 2; Sec. 3.2, last sentence of the p-value paragraph): a
    candidate is ranked only against the calibration scores of its own input.

    calib_groups[g] holds input g's calibration scores (any order).  Reading adopted (the appendix flips the
    indicator and mixes denominators): the same count as the marginal form, 1 + #{calib in own group >= s},
    over |group| + 1.  Returns (numer, denom) as uint32; a NaN candidate has numer 0.
    """
    s = np.asarray(scores, dtype=np.float32)
    g = np.asarray(group_ids, dtype=np.int64)
    numer = np.zeros(s.size, dtype=np.uint32)
    denom = np.zeros(s.size, dtype=np.uint32)
    for j in range(s.size):
        c = np.asarray(calib_groups[g[j]], dtype=np.float32)
        denom[j] = c.size + 1
        numer[j] = conformal_numer_count(s[j:j + 1], c)[0]
    return numer, denom


def classify_conditional(numer: np.ndarray, denom: np.ndarray, alpha: float):
    """Accept iff p > alpha with each candidate's own denominator: reject iff 1 <= numer <= floor(alpha * denom)."""
    num = np.asarray(numer, dtype=np.uint32)
    ka = np.floor(np.float64(alpha) * np.asarray(denom, dtype=np.float64)).astype(np.int64)
    stage = np.full(num.size, STAGE_ACCEPTED, dtype=np.uint8)
    stage[num == 0] = STAGE_DRAFT
    stage[(num >= 1) & (num.astype(np.int64) <= ka)] = STAGE_TARGET
    counts = np.array([(stage == 1).sum(), (stage == 2).sum(), (stage == 3).sum()], dtype=np.uint32)
    return stage, counts


def rms_inv(hidden_bits: np.ndarray, eps: float) -> np.ndarray:
    """1 / sqrt(mean_k h[i, k]^2 + eps) per row, float64: the row factor of an RMS normalisation."""
    H = bf16_bits_to_f64(hidden_bits)
    return 1.0 / np.sqrt((H * H).mean(axis=1) + float(eps))


def token_logprob_scaled(hidden_bits: np.ndarray, lm_head_bits: np.ndarray, token_ids: np.ndarray,
                         row_scale: np.ndarray) -> np.ndarray:
    """token_logprob with every row of logits multiplied by row_scale[i] before the softmax: the LM head applied
    to an RMS-normalised hidden state, z_i = r_i * (W h_i), with the norm's gain folded into W by the caller."""
    ids = np.asarray(token_ids, dtype=np.int64)
    z = logits(hidden_bits, lm_head_bits) * np.asarray(row_scale, dtype=np.float64)[:, None]
    mx = z.max(axis=1)
    lse = mx + np.log(np.exp(z - mx[:, None]).sum(axis=1))
    return z[np.arange(z.shape[0]), ids] - lse
