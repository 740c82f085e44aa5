"""Data-parallel plumbing for more than one GPU (host logic only; no arithmetic of the method).

The path shards by samples: every rank scores its own draft samples against a replicated LM head and
a replicated calibration buffer.  The one exchange per step is an all-gather of the ranks' new
scores, after which every rank merge-inserts the same scores in the same order, so the replicated
buffers stay bit-identical without any further traffic.
"""
from __future__ import annotations


def sample_range(n_samples: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous block [begin, end) of a batch of n_samples that `rank` scores (sizes differ by at most 1)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_samples, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_seed(base_seed: int, rank: int, stream: int = 0) -> int:
    """Seed of a rank's synthetic batch: distinct per rank and per stream of random numbers."""
    return base_seed + stream + 1000 * rank


def all_gather_scores(local_scores, world: int, dist=None):
    """Concatenation over ranks (in rank order) of equally sized 1-D score tensors; identity when world == 1."""
    if world == 1:
        return local_scores
    import torch
    parts = [torch.empty_like(local_scores) for _ in range(world)]
    dist.all_gather(parts, local_scores.contiguous())
    return torch.cat(parts)


def vocab_range(V: int, world: int, rank: int, align: int = 256) -> tuple[int, int]:
    """Rows [begin, end) of the LM head that `rank` holds when the vocabulary is sharded: equal slices rounded up
    to a multiple of `align` rows (one vocabulary tile), the last rank taking what is left (possibly nothing)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    per = -(-V // world)
    per = -(-per // align) * align
    begin = min(rank * per, V)
    return begin, min(begin + per, V)


def all_gather_slice_stats(local_stats, world: int, dist=None):
    """[M, 3] per rank -> [world, M, 3] in rank order (the layout atts_score_combine reads)."""
    import torch
    if world == 1:
        return local_stats.unsqueeze(0)
    parts = [torch.empty_like(local_stats) for _ in range(world)]
    dist.all_gather(parts, local_stats.contiguous())
    return torch.stack(parts)
