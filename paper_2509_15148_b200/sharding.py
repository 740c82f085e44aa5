"""Data-parallel plumbing for more than one GPU (host logic only; no arithmetic of the method).

The path shards by samples: every rank scores its own draft samples against a replicated LM head and
a replicated calibration buffer.  The one exchange per step is an all-gather of the ranks' new
scores, after which every rank merge-inserts the same scores in the same order, so the replicated
buffers stay bit-identical without any further traffic.
"""
from __future__ import annotations


def free_port() -> int:
    """A TCP port that is free on the loopback interface right now."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_command(script: str, script_args: list[str], n_ranks: int, port: int, python: str,
                   environ: dict) -> tuple[list[str], dict]:
    """Command line and environment that start `script` as n_ranks processes on this node, one per GPU, with a
    loopback rendezvous (torch.distributed.run).  NCCL's communicator lines are switched on unless the caller has
    set NCCL_DEBUG already, so that the number of ranks of the communicator can be read from the log."""
    if n_ranks < 2:
        raise ValueError("one rank needs no launcher")
    cmd = [python, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), script] + list(script_args)
    env = dict(environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    return cmd, env


def needs_launch(n_ranks: int, environ: dict) -> bool:
    """True when more than one rank is asked for and this process was not started by a launcher already."""
    return n_ranks > 1 and "WORLD_SIZE" not in environ


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
