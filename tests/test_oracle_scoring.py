"""Pins for the scoring half of the CPU oracle (token log-probs, sample scores).

Each test fixes the oracle to something other than its own formula: a
brute-force softmax in Python floats, closed forms, torch's float64
cross_entropy, invariances of the softmax.  They are chosen so that a dropped
term, a wrong sign, a transposed operand or a mis-decoded bf16 fails one.
"""
import math

import numpy as np
import pytest
import torch

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import inputs


def _bits(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_bf16_decode_known_patterns():
    bits = np.array([0x3F80, 0xC000, 0x3DCC, 0x0000, 0x8000, 0x7F80, 0x0080, 0x4049], dtype=np.uint16)
    want = [1.0, -2.0, 0.099609375, 0.0, -0.0, math.inf, 2.0 ** -126, 3.140625]
    got = orc.bf16_bits_to_f64(bits)
    assert got.dtype == np.float64
    assert list(got) == want
    assert math.copysign(1.0, got[4]) == -1.0


def test_bf16_encode_round_to_nearest_even():
    # 1 + 2^-8 is exactly half way between bf16 neighbours 1.0 and 1 + 2^-7: ties to even -> 1.0
    assert _bits([1.0 + 2.0 ** -8])[0] == 0x3F80
    # 1 + 3 * 2^-8 is half way between 1 + 2^-7 (odd) and 1 + 2^-6 (even) -> up
    assert _bits([1.0 + 3 * 2.0 ** -8])[0] == 0x3F82
    assert _bits([1.0 + 2.0 ** -8 + 2.0 ** -20])[0] == 0x3F81
    x = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    back = inputs.bf16_bits_to_f32(_bits(x))
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    t = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(_bits(x), t)


def _brute_logprob(H, W, ids):
    """Full softmax over the vocabulary in Python floats with math.fsum."""
    out = []
    for i in range(len(H)):
        z = [math.fsum(float(H[i][k]) * float(W[v][k]) for k in range(len(H[i]))) for v in range(len(W))]
        tot = math.fsum(math.exp(zz) for zz in z)
        out.append(z[ids[i]] - math.log(tot))
    return np.array(out)


@pytest.mark.parametrize("M,d,V,seed", [(5, 16, 64, 0), (7, 3, 11, 1), (1, 1, 2, 2), (4, 8, 1, 3)])
def test_logprob_matches_bruteforce_softmax(M, d, V, seed):
    rng = np.random.default_rng(seed)
    Hb = _bits(rng.standard_normal((M, d)))
    Wb = _bits(rng.standard_normal((V, d)))
    ids = rng.integers(0, V, size=M).astype(np.int32)
    H = inputs.bf16_bits_to_f32(Hb).astype(np.float64)
    W = inputs.bf16_bits_to_f32(Wb).astype(np.float64)
    want = _brute_logprob(H.tolist(), W.tolist(), ids.tolist())
    got = orc.token_logprob(Hb, Wb, ids)
    assert got.dtype == np.float64
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def test_logprob_matches_torch_cross_entropy_float64():
    rng = np.random.default_rng(11)
    M, d, V = 33, 24, 301
    Hb, Wb = _bits(rng.standard_normal((M, d))), _bits(rng.standard_normal((V, d)) * 0.5)
    ids = rng.integers(0, V, size=M).astype(np.int32)
    Ht = torch.from_numpy(Hb.view(np.int16)).view(torch.bfloat16).double()
    Wt = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).double()
    nll = torch.nn.functional.cross_entropy(Ht @ Wt.T, torch.from_numpy(ids).long(), reduction="none")
    np.testing.assert_allclose(orc.token_logprob(Hb, Wb, ids), -nll.numpy(), rtol=0, atol=1e-12)


def test_logprob_closed_forms():
    M, d, V = 6, 8, 40
    rng = np.random.default_rng(3)
    Hb = _bits(rng.standard_normal((M, d)))
    ids = rng.integers(0, V, size=M).astype(np.int32)
    # zero weights: uniform distribution
    got = orc.token_logprob(Hb, np.zeros((V, d), dtype=np.uint16), ids)
    np.testing.assert_allclose(got, -math.log(V), atol=1e-13)
    # all vocabulary rows identical: uniform as well, whatever the row
    Wb = np.tile(_bits(rng.standard_normal((1, d))), (V, 1))
    np.testing.assert_allclose(orc.token_logprob(Hb, Wb, ids), -math.log(V), atol=1e-12)
    # V = d, W = c * I, h = e_j: logit c at column j, 0 elsewhere
    c, n = 2.0, 16
    Wb = _bits(c * np.eye(n))
    Hb = _bits(np.eye(n))
    on = orc.token_logprob(Hb, Wb, np.arange(n, dtype=np.int32))
    np.testing.assert_allclose(on, c - math.log(math.exp(c) + n - 1), atol=1e-13)
    off = orc.token_logprob(Hb, Wb, ((np.arange(n) + 1) % n).astype(np.int32))
    np.testing.assert_allclose(off, 0.0 - math.log(math.exp(c) + n - 1), atol=1e-13)


def test_logprob_is_a_distribution_and_permutation_invariant():
    rng = np.random.default_rng(5)
    d, V = 12, 50
    hb = _bits(rng.standard_normal((1, d)))
    Wb = _bits(rng.standard_normal((V, d)))
    Hrep = np.repeat(hb, V, axis=0)
    lp = orc.token_logprob(Hrep, Wb, np.arange(V, dtype=np.int32))
    assert abs(np.exp(lp).sum() - 1.0) < 1e-12
    perm = rng.permutation(V)
    inv = np.empty(V, dtype=np.int64)
    inv[perm] = np.arange(V)
    lp_perm = orc.token_logprob(Hrep, Wb[perm], inv.astype(np.int32))
    np.testing.assert_allclose(lp_perm, lp, atol=1e-12)


def test_logprob_large_logits_do_not_overflow():
    # logits of +-600: a naive exp overflows float64 only above ~709, the max-shift must hold anyway
    d = 4
    Hb = _bits(np.full((1, d), 16.0))
    Wb = _bits(np.array([[16.0] * d, [-16.0] * d, [0.0] * d]))   # logits 1024, -1024, 0
    lp = orc.token_logprob(np.repeat(Hb, 3, 0), Wb, np.array([0, 1, 2], dtype=np.int32))
    np.testing.assert_allclose(lp, [0.0, -2048.0, -1024.0], atol=1e-9)


def test_logprob_rejects_bad_ids():
    Hb, Wb = np.zeros((2, 4), np.uint16), np.zeros((3, 4), np.uint16)
    with pytest.raises(ValueError):
        orc.token_logprob(Hb, Wb, np.array([0, 3], dtype=np.int32))
    with pytest.raises(ValueError):
        orc.token_logprob(Hb, Wb, np.array([-1, 0], dtype=np.int32))


def test_sample_score_modes_and_invariants():
    lp = np.array([-1.0, -2.0, -3.0, -0.5, -0.25, -4.0])
    off = np.array([0, 3, 3, 6], dtype=np.int32)
    s0 = orc.sample_score(lp, off, 0)
    np.testing.assert_allclose(s0[[0, 2]], [2.0, (0.5 + 0.25 + 4.0) / 3])
    assert math.isnan(s0[1])
    np.testing.assert_allclose(orc.sample_score(lp, off, 1)[[0, 2]], [6.0, 4.75])
    np.testing.assert_allclose(orc.sample_score(lp, off, 2)[[0, 2]], [-2.0, -4.75 / 3])
    np.testing.assert_allclose(orc.sample_score(lp, off, 3)[[0, 2]], [-6.0, -4.75])
    # identical tokens: the mean score is minus that log-prob, whatever the length
    same = np.full(17, -1.375)
    assert orc.sample_score(same, np.array([0, 17]), 0)[0] == 1.375
    # two equal-length samples joined into one: the mean of their scores
    rng = np.random.default_rng(2)
    lp = -rng.random(64)
    two = orc.sample_score(lp, np.array([0, 32, 64]), 0)
    one = orc.sample_score(lp, np.array([0, 64]), 0)
    assert abs(one[0] - two.mean()) < 1e-15
    # a single-token sample scores minus that token's log-prob
    assert orc.sample_score(np.array([-0.75]), np.array([0, 1]), 0)[0] == 0.75


def test_score_equals_log_perplexity_on_generated_inputs():
    # mean NLL = log PPL; checked through torch's mean-reduced cross_entropy on a small generated batch
    N, T, d, V = 3, 5, 64, 97
    Hb = inputs.hidden(7, N * T, d)
    Wb = inputs.lm_head(8, V, d)
    ids = inputs.zipf_ids(9, N * T, V)
    lp = orc.token_logprob(Hb, Wb, ids)
    sc = orc.sample_score(lp, inputs.seg_offsets(N, T), 0)
    Ht = torch.from_numpy(inputs.bf16_bits_to_f32(Hb)).double()
    Wt = torch.from_numpy(inputs.bf16_bits_to_f32(Wb)).double()
    for k in range(N):
        ce = torch.nn.functional.cross_entropy(Ht[k * T:(k + 1) * T] @ Wt.T,
                                               torch.from_numpy(ids[k * T:(k + 1) * T]).long())
        assert abs(sc[k] - ce.item()) < 1e-12
