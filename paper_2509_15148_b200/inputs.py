"""Seeded synthetic input generators (numpy only).

These arrays stand in for the draft/target pairs of the paper's experiments
(Experimental Setup): a target model's final hidden states for the tokens of
parallel draft samples, its LM-head matrix, the draft token ids, and scalar
scores for the conformal-only workloads.  The module draws random numbers and
converts dtypes; it contains none of the method's arithmetic (no logits, no
log-sum-exp, no ranks), so both the CPU oracle's tests and the CUDA path's
tests can be fed from it without sharing any computation.

Recipe (every array is a pure function of its seed and shape):

* Large matrices are drawn in slabs of ``SLAB_ROWS`` rows; slab ``j`` uses
  ``numpy.random.default_rng([seed, j])`` (PCG64), so slabs can be produced by
  a thread pool and any row range can be regenerated on its own.
* ``lm_head``: float32 standard normals times 0.02 (standard deviation 0.02),
  rounded to bf16 (round to nearest, ties to even).
* ``hidden``: float32 standard normals, each row divided by its root mean
  square (no epsilon, no gain) in float32, rounded to bf16.
* ``zipf_ids``: ``P(id = r)`` proportional to ``(r + 1) ** -s`` for
  ``r = 0 .. V-1`` by inverse CDF on a float64 cumulative table.
* ``lognormal_scores``: ``exp(standard normal)`` in float32.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

SLAB_ROWS = 2048


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _slabbed(seed: int, rows: int, cols: int, fn, row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    row_end = rows if row_end is None else row_end
    out = np.empty((row_end - row_begin, cols), dtype=np.uint16)
    first, last = row_begin // SLAB_ROWS, (max(row_end, row_begin + 1) - 1) // SLAB_ROWS

    def work(j: int) -> None:
        a, b = j * SLAB_ROWS, min((j + 1) * SLAB_ROWS, rows)
        rng = np.random.default_rng([seed, j])
        x = rng.standard_normal((b - a, cols), dtype=np.float32)
        bits = f32_to_bf16_bits(fn(x))
        lo, hi = max(a, row_begin), min(b, row_end)
        if hi > lo:
            out[lo - row_begin:hi - row_begin] = bits[lo - a:hi - a]

    jobs = list(range(first, last + 1))
    workers = max(1, min(len(jobs), os.cpu_count() or 1, 16))
    if workers == 1:
        for j in jobs:
            work(j)
    else:
        with ThreadPoolExecutor(workers) as ex:
            list(ex.map(work, jobs))
    return out


def lm_head(seed: int, V: int, d: int, row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    """LM-head matrix W [V, d] as bf16 bits, entries ~ N(0, 0.02**2). Optional row range."""
    return _slabbed(seed, V, d, lambda x: x * np.float32(0.02), row_begin, row_end)


def hidden(seed: int, M: int, d: int, row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    """Hidden states H [M, d] as bf16 bits: Gaussian rows scaled to unit root mean square."""
    def rms_rows(x: np.ndarray) -> np.ndarray:
        r = np.sqrt(np.mean(x * x, axis=1, dtype=np.float32, keepdims=True))
        return x / r
    return _slabbed(seed, M, d, rms_rows, row_begin, row_end)


def zipf_ids(seed: int, M: int, V: int, s: float = 1.1) -> np.ndarray:
    """Token ids [M] int32 with P(id = r) proportional to (r + 1) ** -s over r in [0, V)."""
    w = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    u = np.random.default_rng(seed).random(M)
    ids = np.searchsorted(cdf, u, side="right")
    return np.minimum(ids, V - 1).astype(np.int32)


def seg_offsets(N: int, T: int) -> np.ndarray:
    """Segment offsets [N + 1] int32 for N samples of T tokens each."""
    return (np.arange(N + 1, dtype=np.int64) * T).astype(np.int32)


def ragged_seg_offsets(seed: int, N: int, T_max: int, allow_empty: bool = True) -> np.ndarray:
    """Segment offsets for N samples with lengths uniform in [0 or 1, T_max] (early end tokens)."""
    lo = 0 if allow_empty else 1
    lens = np.random.default_rng(seed).integers(lo, T_max + 1, size=N)
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)


def lognormal_scores(seed: int, n: int, mu: float = 0.0, sigma: float = 1.0) -> np.ndarray:
    """Scores [n] float32 ~ LogNormal(mu, sigma)."""
    z = np.random.default_rng(seed).standard_normal(n)
    return np.exp(mu + sigma * z).astype(np.float32)


# The five workload shapes (N samples x T tokens, hidden d, vocab V, calibration n, alphas).
CONFIGS = {
    "tiny": dict(N=8, T=64, d=512, V=8192, n=256, alphas=(0.1,)),
    "7b": dict(N=16, T=256, d=3584, V=152064, n=1024, alphas=(0.1,)),
    "32b": dict(N=64, T=1024, d=5120, V=152064, n=4096, alphas=(0.1,)),
    "70b": dict(N=32, T=512, d=8192, V=128256, n=4096, alphas=(0.05, 0.1)),
}
CONFORMAL_STRESS = dict(Nc=1 << 20, n0=1 << 16, k=4096, steps=64, alphas=(0.05, 0.1, 0.2))
BASE_SEED = 1234
