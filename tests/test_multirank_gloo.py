"""World-size-2 check (gloo, CPU) of the data-parallel host logic: sample sharding, the score
all-gather, and that every rank ends up with the same calibration buffer as one process would."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import atts_oracle as orc
from paper_2509_15148_b200 import inputs, sharding


def test_sample_range_partitions_the_batch():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            spans = [sharding.sample_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    assert len({sharding.rank_seed(1234, r, s) for r in range(8) for s in range(3)}) == 24


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    calib = np.sort(inputs.lognormal_scores(50, 300))                     # replicated buffer
    n = calib.size
    stages = []
    for step in range(3):
        local = inputs.lognormal_scores(sharding.rank_seed(60 + 10 * step, rank), 16)   # this rank's 16 scores
        numer = orc.conformal_numer_sorted(local, calib)                  # rank against the buffer as it was
        stages.append(orc.classify(numer, n, 0.1)[0])
        allv = sharding.all_gather_scores(torch.from_numpy(local), world, dist).numpy()
        calib = orc.calib_update(calib, allv)                             # every rank inserts all ranks' scores
        n = calib.size
    np.save(os.path.join(out_dir, f"calib_{rank}.npy"), calib)
    np.save(os.path.join(out_dir, f"stage_{rank}.npy"), np.concatenate(stages))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_keep_identical_buffers(tmp_path):
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    bufs = [np.load(tmp_path / f"calib_{r}.npy") for r in range(world)]
    assert np.array_equal(bufs[0].view(np.uint32), bufs[1].view(np.uint32))
    # one process doing the same inserts in rank order gets the same buffer
    calib = np.sort(inputs.lognormal_scores(50, 300))
    want_stage = {r: [] for r in range(world)}
    for step in range(3):
        locals_ = [inputs.lognormal_scores(sharding.rank_seed(60 + 10 * step, r), 16) for r in range(world)]
        for r in range(world):
            want_stage[r].append(orc.classify(orc.conformal_numer_sorted(locals_[r], calib), calib.size, 0.1)[0])
        calib = orc.calib_update(calib, np.concatenate(locals_))
    assert calib.size == 300 + 3 * 32
    assert np.array_equal(bufs[0].view(np.uint32), calib.view(np.uint32))
    for r in range(world):
        assert np.array_equal(np.load(tmp_path / f"stage_{r}.npy"), np.concatenate(want_stage[r]))


def test_vocab_range_partitions_the_vocabulary():
    for V in (1, 255, 256, 257, 8192, 152064, 128256):
        for world in (1, 2, 3, 8):
            spans = [sharding.vocab_range(V, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == V
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            assert all(a % 256 == 0 for a, _ in spans if a < V)


def _vocab_worker(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    M, d, V = 40, 32, 700
    Hb, Wb = inputs.hidden(1, M, d), inputs.lm_head(2, V, d)
    ids = inputs.zipf_ids(3, M, V)
    a, b = sharding.vocab_range(V, world, rank)
    # this rank's triple per token over its slice of the vocabulary (float64 stand-in for atts_score_slice)
    z = orc.logits(Hb, Wb[a:b]) if b > a else np.full((M, 0), -np.inf)
    mx = z.max(axis=1) if b > a else np.full(M, -np.inf)
    sm = np.exp(z - mx[:, None]).sum(axis=1) if b > a else np.zeros(M)
    g = np.where((ids >= a) & (ids < b), z[np.arange(M), np.clip(ids - a, 0, max(b - a - 1, 0))] if b > a else -np.inf, -np.inf)
    local = torch.from_numpy(np.stack([mx, sm, g], axis=1))
    allst = sharding.all_gather_slice_stats(local, world, dist).numpy()          # [world, M, 3]
    assert allst.shape == (world, M, 3)
    Mx = allst[:, :, 0].max(axis=0)
    lse = Mx + np.log((allst[:, :, 1] * np.exp(allst[:, :, 0] - Mx)).sum(axis=0))
    lp = allst[:, :, 2].max(axis=0) - lse
    np.save(os.path.join(out_dir, f"lp_{rank}.npy"), lp)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_vocabulary_sharded_scoring(tmp_path):
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_vocab_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    want = orc.token_logprob(inputs.hidden(1, 40, 32), inputs.lm_head(2, 700, 32), inputs.zipf_ids(3, 40, 700))
    for r in range(world):
        np.testing.assert_allclose(np.load(tmp_path / f"lp_{r}.npy"), want, atol=1e-12)


def test_launcher_host_logic():
    """`bench.py --gpus N` started plainly starts its own N ranks; under a launcher, or with one GPU, it does not."""
    assert not sharding.needs_launch(1, {})
    assert sharding.needs_launch(2, {})
    assert not sharding.needs_launch(2, {"WORLD_SIZE": "2", "RANK": "0"})
    cmd, env = sharding.launch_command("/x/bench.py", ["--gpus", "2", "--steps", "5"], 2, 29517, "/usr/bin/python",
                                       {"PATH": "/bin", "NCCL_DEBUG": "WARN"})
    assert cmd[:3] == ["/usr/bin/python", "-m", "torch.distributed.run"]
    assert "--nproc-per-node=2" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29517"
    assert cmd[-5:] == ["/x/bench.py", "--gpus", "2", "--steps", "5"]
    assert env["NCCL_DEBUG"] == "WARN" and env["PATH"] == "/bin"          # the caller's settings win
    _, env2 = sharding.launch_command("/x/bench.py", [], 4, 1, "py", {})
    assert env2["NCCL_DEBUG"] == "INFO"
    try:
        sharding.launch_command("/x/bench.py", [], 1, 1, "py", {})
        raise AssertionError("one rank must not be launched")
    except ValueError:
        pass
    port = sharding.free_port()
    assert 1024 <= port < 65536
