#!/usr/bin/env python
"""Benchmark of the ATTS verification hot path.

One step = one pass of the whole path over one batch of synthetic input at the 32B-target shape
(N = 64 parallel draft samples x T = 1024 tokens, hidden 5120, vocabulary 152064, online
calibration buffer starting at n = 4096, alpha = 0.1):

    atts_score_logprob -> atts_conformal_rank -> atts_classify -> atts_calib_update

The metric is draft tokens scored per second over the whole job.  `python bench.py --gpus N
--steps K --warmup W` prints one JSON line on rank 0.  For N > 1 it runs one rank per GPU: started
plainly it launches the N ranks itself (torch.distributed.run, loopback rendezvous); started under
torchrun it is one of them.
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_15148_b200 import inputs  # noqa: E402

WORKLOAD = "32b"   # the bench line's workload; --workload picks another shape for profiling runs
ALPHA = 0.1
METRIC = "draft tokens scored/s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
KERNELS_PER_STEP = 6  # lmhead_lse, lse_combine, segment_score, rank, classify, small_update (n + k small: one block)
# DRAM bytes per launch of the fused kernel on this workload, from an ncu capture (profiles/), valid only for
# the kernel source it was taken on: (sha256 of csrc/lmhead_lse.cuh, dram__bytes_read.sum + dram__bytes_write.sum).
K1_TRAFFIC = ("63ed8c15ce1c5157e25ce877a7cba86bd55c145fefd26b445bb2b96233c252f6", 8.680e10)


def k1_traffic_bytes():
    import hashlib
    path = os.path.join(ROOT, "paper_2509_15148_b200", "csrc", "lmhead_lse.cuh")
    try:
        digest = hashlib.sha256(open(path, "rb").read()).hexdigest()
    except OSError:
        return None
    return K1_TRAFFIC[1] if K1_TRAFFIC[0] == digest else None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons with nvidia-smi while a timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_rows_plan(M: int, T: int, whole_samples: int, scattered: int, seed: int) -> np.ndarray:
    """Token rows the oracle scores out of a batch of M: the first `whole_samples` samples completely, plus
    `scattered` rows drawn by a seeded permutation from the rest (every row spans the whole vocabulary and hidden
    dimension, so every tile column is exercised by every row)."""
    head = np.arange(min(whole_samples * T, M))
    rest = np.arange(head.size, M)
    pick = np.random.default_rng(seed).permutation(rest)[:scattered] if rest.size else rest
    return np.concatenate([head, np.sort(pick)]).astype(np.int64)


def oracle_step(orc, H_rows, Wb, ids_rows, whole_rows, T, scores_rest, calib, alpha):
    """One pass of the oracle over a bounded sample: the given token rows scored (the first `whole_rows` of them are
    whole samples of T tokens and give sample scores), then rank / p-value / stage / insert on the batch's scores
    (`scores_rest` stands in for the samples the oracle did not score)."""
    lp = orc.token_logprob(H_rows, Wb, ids_rows)
    own = np.zeros(0, np.float32)
    if whole_rows:
        off = (np.arange(whole_rows // T + 1) * T).astype(np.int32)
        own = orc.sample_score(lp[:whole_rows], off).astype(np.float32)
    sc = np.concatenate([own, np.asarray(scores_rest, np.float32)])
    numer = orc.conformal_numer_sorted(sc, calib)
    orc.pvalue(numer, calib.size)
    orc.classify(numer, calib.size, alpha)
    return orc.calib_update(calib, sc[~np.isnan(sc)])


def oracle_conformal_steps(orc):
    """The oracle on the whole conformal-only workload: rank, p-values, three thresholds and insert, 64 steps."""
    cfg = inputs.CONFORMAL_STRESS
    steps = cfg["steps"]
    scores = inputs.lognormal_scores(inputs.BASE_SEED + 1, cfg["Nc"])
    calib = np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, cfg["n0"]))
    news = [inputs.lognormal_scores(inputs.BASE_SEED + 3 + t, cfg["k"]) for t in range(steps)]
    t0 = time.perf_counter()
    for t in range(steps):
        numer = orc.conformal_numer_sorted(scores, calib)
        orc.pvalue(numer, calib.size)
        for alpha in cfg["alphas"]:
            orc.classify(numer, calib.size, alpha)
        calib = orc.calib_update(calib, news[t])
    dt = time.perf_counter() - t0
    return {"value": cfg["Nc"] * steps / dt, "unit": "p-values/s", "cores": 1, "kind": "oracle",
            "sample": f"all {steps} steps of the conformal-only workload in {dt:.1f} s"}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import atts_oracle as orc
    c = inputs.CONFIGS[args.workload]
    N, T, d, V, n0 = c["N"], c["T"], c["d"], c["V"], c["n"]
    M = N * T
    rows = args.oracle_rows
    Wb = inputs.lm_head(inputs.BASE_SEED, V, d)
    # token rows scattered over the batch: a few rows from each of a few seeded slabs (a slab is what the input
    # generator can reproduce on its own)
    rng = np.random.default_rng(inputs.BASE_SEED + 9)
    n_slabs = -(-M // inputs.SLAB_ROWS)
    slabs = np.sort(rng.choice(n_slabs, size=min(n_slabs, max(1, rows // 16)), replace=False))
    per = -(-rows // slabs.size)
    picks, parts = [], []
    for j in slabs:
        a0, b0 = j * inputs.SLAB_ROWS, min((j + 1) * inputs.SLAB_ROWS, M)
        loc = np.sort(rng.choice(b0 - a0, size=min(per, b0 - a0), replace=False))
        parts.append(inputs.hidden(inputs.BASE_SEED + 1, M, d, a0, b0)[loc])
        picks.append(a0 + loc)
    idx = np.concatenate(picks)[:rows]
    Hb = np.concatenate(parts)[:rows]
    ids = inputs.zipf_ids(inputs.BASE_SEED + 2, M, V)[idx]
    rows = idx.size
    # the oracle cannot afford to score 4096 calibration samples or the other samples of the batch: LogNormal-shaped
    # stand-ins near the NLL scale feed the conformal steps
    calib = np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 5, n0)) + np.float32(11.0)
    rest = inputs.lognormal_scores(inputs.BASE_SEED + 6, N) + np.float32(11.0)
    for _ in range(args.warmup):
        calib = oracle_step(orc, Hb, Wb, ids, 0, T, rest, calib, ALPHA)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        calib = oracle_step(orc, Hb, Wb, ids, 0, T, rest, calib, ALPHA)
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    sample = (f"{rows} of {M} token rows per step, scattered over the batch by a seeded choice (full d and V), then "
              f"rank/classify/update on N={N} scores")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload.upper()}-target shape N={N} T={T} d={d} V={V} n={n0} alpha={ALPHA}", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def make_graph_timer(torch):
    def graph_ms(fn, reps=1, rounds=5):
        """GPU time of fn(): captured `reps` times into one CUDA graph, best of `rounds` replays (events around the
        replay), so that host launch overhead between these microsecond kernels is not what is measured."""
        fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(reps):
                fn()
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = float("inf")
        for _ in range(rounds):
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return best / reps
    return graph_ms


def update_bytes(n: int, k: int) -> float:
    """Algorithmic bytes of one merge-insert: the old buffer read and the merged buffer written once, the new
    scores read once."""
    return 8.0 * (n + k) + 4.0 * k


def conformal_stress(torch, binding, peaks):
    """Extra figures on the conformal-only workload: 2^20 candidates against a buffer growing from 65,536 by 4,096 a
    step, three alphas; kernel times by CUDA events (the working set is L2-resident)."""
    cfg = inputs.CONFORMAL_STRESS
    Nc, n0, k, steps = cfg["Nc"], cfg["n0"], cfg["k"], cfg["steps"]
    alphas = cfg["alphas"]
    dev = "cuda"
    hbm = peaks["hbm_gbs"]
    scores = torch.from_numpy(inputs.lognormal_scores(inputs.BASE_SEED + 1, Nc)).to(dev)
    calib0 = torch.from_numpy(np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, n0))).to(dev)
    news = [torch.from_numpy(inputs.lognormal_scores(inputs.BASE_SEED + 3 + t, k)).to(dev) for t in range(steps)]
    cap = n0 + k * steps
    buf = torch.empty(cap, device=dev)
    numer = torch.empty(Nc, dtype=torch.int32, device=dev)
    p = torch.empty(Nc, device=dev)
    stage = torch.empty(Nc, dtype=torch.uint8, device=dev)
    counts = torch.empty(3, dtype=torch.int32, device=dev)
    stage3 = torch.empty((len(alphas), Nc), dtype=torch.uint8, device=dev)
    counts3 = torch.empty((len(alphas), 3), dtype=torch.int32, device=dev)
    ws = torch.empty(binding.calib_workspace_bytes(cap, k), dtype=torch.uint8, device=dev)
    index = torch.empty(binding.calib_index_bytes(cap), dtype=torch.uint8, device=dev)
    side = torch.cuda.Stream()

    def sequence_plain():
        buf[:n0] = calib0
        n = n0
        for t in range(steps):
            binding.rank_classify(scores, buf, n, alphas, numer, p, stage3, counts3)
            n = binding.calib_update(buf, n, news[t], ws)
        return n

    def sequence():
        # the calibration state is the buffer and its index; every update leaves both describing the new fill
        buf[:n0] = calib0
        binding.calib_index_build(buf, n0, index)
        n = n0
        for t in range(steps):
            binding.rank_classify_indexed(scores, buf, n, index, alphas, numer, p, stage3, counts3)
            n = binding.calib_update_indexed(buf, n, news[t], index, ws)
        return n

    def sequence_two_streams():
        # the update of step t needs nothing the rank of step t writes: it runs on a second stream beside it; the
        # next rank waits for the update, the next update for this rank (it overwrites what this rank reads)
        main = torch.cuda.current_stream()
        buf[:n0] = calib0
        binding.calib_index_build(buf, n0, index)
        n = n0
        for t in range(steps):
            side.wait_stream(main)
            binding.rank_classify_indexed(scores, buf, n, index, alphas, numer, p, stage3, counts3)
            with torch.cuda.stream(side):
                n = binding.calib_update_indexed(buf, n, news[t], index, ws)
            main.wait_stream(side)
        return n

    graph_ms = make_graph_timer(torch)
    # best of 20 replays each: after the long scoring loop the clocks need some milliseconds to settle
    ms_seq_plain = graph_ms(sequence_plain, rounds=20)
    ms_seq = graph_ms(sequence, rounds=20)
    ms_seq2 = graph_ms(sequence_two_streams, rounds=20)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eager = []
    for _ in range(3):
        e0.record()
        sequence()
        e1.record()
        torch.cuda.synchronize()
        eager.append(e0.elapsed_time(e1))

    # ---- single calls at the last step's sizes.  The update is timed together with a copy that restores the buffer
    # (repeated inserts into the same buffer would drift its contents), and that copy alone is subtracted.
    n_end = cap - k
    calib_end = torch.sort(torch.cat([calib0] + news[:-1])).values.contiguous()
    assert calib_end.numel() == n_end

    def restore():
        buf[:n_end] = calib_end

    restore()
    ms_restore = graph_ms(restore, reps=20)
    ms_rank = graph_ms(lambda: binding.conformal_rank(scores, buf, n_end, numer, p), reps=20)
    ms_cls = graph_ms(lambda: binding.classify(numer, n_end, 0.1, stage, counts), reps=20)
    ms_fused = graph_ms(lambda: binding.rank_classify(scores, buf, n_end, alphas, numer, p, stage3, counts3), reps=20)

    def upd_plain():
        restore()
        binding.calib_update(buf, n_end, news[-1], ws)

    ms_upd = graph_ms(upd_plain, reps=20) - ms_restore
    restore()
    binding.calib_index_build(buf, n_end, index)
    ms_fused_ix = graph_ms(lambda: binding.rank_classify_indexed(scores, buf, n_end, index, alphas, numer, p, stage3,
                                                                 counts3), reps=20)
    # the indexed update reads the index's copy of fill n_end, which repeated calls leave as it is
    ms_upd_ix = graph_ms(lambda: binding.calib_update_indexed(buf, n_end, news[-1], index, ws), reps=20)
    # a drifted batch: every new score above the buffer's largest entry (one block owns and sorts them all)
    drift = (news[-1] + calib_end[-1]).contiguous()
    ms_upd_ix_drift = graph_ms(lambda: binding.calib_update_indexed(buf, n_end, drift, index, ws), reps=20)
    # The same calls with a cold L2: 512 MB are written between repetitions, one call is timed by events (the events'
    # own few microseconds are inside), median of 9.
    scrub = torch.empty(128 << 20, dtype=torch.float32, device=dev)

    def cold_us(fn):
        ts = []
        for _ in range(9):
            scrub.fill_(1.0)
            torch.cuda.synchronize()
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts))

    restore()
    cold = {
        "rank_classify_indexed_us": cold_us(lambda: binding.rank_classify_indexed(scores, buf, n_end, index, alphas,
                                                                              numer, p, stage3, counts3)),
        "rank_classify_us": cold_us(lambda: binding.rank_classify(scores, buf, n_end, alphas, numer, p, stage3, counts3)),
        "classify_us": cold_us(lambda: binding.classify(numer, n_end, 0.1, stage, counts)),
        "update_indexed_us": cold_us(lambda: binding.calib_update_indexed(buf, n_end, news[-1], index, ws)),
        "note": "L2 flushed by a 512 MB write before each call; one call between two events",
    }
    del scrub
    rank_bytes = 12.0 * Nc + 4.0 * n_end
    cls_bytes = 5.0 * Nc
    fused_bytes = rank_bytes + len(alphas) * Nc
    # algorithmic bytes of the whole 64-step sequence: per step the rank + three alphas in one pass and one merge-insert
    seq_bytes = sum(12.0 * Nc + len(alphas) * Nc + 4.0 * (n0 + k * t) + update_bytes(n0 + k * t, k) for t in range(steps))
    out = {
        "workload": f"conformal-only stress: Nc={Nc}, n {n0}->{cap}, k={k}, {steps} steps, alphas {list(alphas)}",
        "step": "atts_rank_classify_indexed (3 alphas, one launch) + atts_calib_update_indexed (one launch)",
        "pvalues_per_s": Nc * steps / (ms_seq * 1e-3),
        "ms_sequence": ms_seq, "us_per_step": ms_seq * 1e3 / steps, "ms_sequence_eager_launches": min(eager),
        "sequence_algorithmic_gbs": seq_bytes / (ms_seq * 1e-3) / 1e9,
        "sequence_frac_hbm": seq_bytes / (ms_seq * 1e-3) / 1e9 / hbm,
        "ms_sequence_two_streams": ms_seq2, "pvalues_per_s_two_streams": Nc * steps / (ms_seq2 * 1e-3),
        "ms_sequence_without_index": ms_seq_plain, "pvalues_per_s_without_index": Nc * steps / (ms_seq_plain * 1e-3),
        "timing": "64-step sequence captured in one CUDA graph, events around the replay, best of 20; working set "
                  "(<= 14 MB) is L2-resident, so GB/s are algorithmic bytes over time, not DRAM traffic; "
                  "two_streams: each update on a second stream beside the rank of the same fill",
        "rank_us": ms_rank * 1e3, "rank_gbs": rank_bytes / (ms_rank * 1e-3) / 1e9,
        "rank_frac_hbm": rank_bytes / (ms_rank * 1e-3) / 1e9 / hbm,
        "classify_us": ms_cls * 1e3, "classify_gbs": cls_bytes / (ms_cls * 1e-3) / 1e9,
        "update_us": ms_upd * 1e3, "update_gbs": update_bytes(n_end, k) / (ms_upd * 1e-3) / 1e9,
        "rank_classify_fused_us": ms_fused * 1e3, "rank_classify_fused_gbs": fused_bytes / (ms_fused * 1e-3) / 1e9,
        "rank_classify_indexed_us": ms_fused_ix * 1e3, "rank_classify_indexed_gbs": fused_bytes / (ms_fused_ix * 1e-3) / 1e9,
        "update_indexed_us": ms_upd_ix * 1e3, "update_indexed_gbs": update_bytes(n_end, k) / (ms_upd_ix * 1e-3) / 1e9,
        "update_indexed_drifted_batch_us": ms_upd_ix_drift * 1e3,
        "update_bytes": "8 (n + k) + 4 k per merge-insert (the old buffer read, the merged buffer written, the new scores read)",
        "cold_l2": cold,
    }
    if binding.last_device_status() != 0:
        raise RuntimeError("a conformal kernel reported a device-side error during the benchmark")
    del scores, numer, p, stage, stage3
    out.update(conformal_scaled(torch, binding, peaks, graph_ms))
    return out


def conformal_scaled(torch, binding, peaks, graph_ms):
    """The conformal kernels at sizes where HBM is the limit (extra points beside the five workload shapes)."""
    dev = "cuda"
    out = {}
    hbm = peaks["hbm_gbs"]
    k = inputs.CONFORMAL_STRESS["k"]
    counts = torch.empty(3, dtype=torch.int32, device=dev)
    new0 = torch.from_numpy(inputs.lognormal_scores(inputs.BASE_SEED + 3, k)).to(dev)
    # 2^26 candidates (805 MB of traffic per rank pass) against the model-sized buffer n = 4096 and against a
    # buffer of 2^22 entries, and a merge-insert into a 2^22-entry buffer.
    big, n_small, n_big = 1 << 26, 4096, 1 << 22
    gen = torch.Generator(device=dev)
    gen.manual_seed(inputs.BASE_SEED + 7)
    sc = torch.randn(big, device=dev, generator=gen).exp_()
    cal = torch.from_numpy(np.sort(inputs.lognormal_scores(inputs.BASE_SEED + 2, n_small))).to(dev)
    nm = torch.empty(big, dtype=torch.int32, device=dev)
    pv = torch.empty(big, device=dev)
    st = torch.empty(big, dtype=torch.uint8, device=dev)

    def point(ms, nbytes, **extra):
        d = {"us": ms * 1e3, "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_hbm": nbytes / (ms * 1e-3) / 1e9 / hbm}
        d.update(extra)
        return d

    ms = graph_ms(lambda: binding.conformal_rank(sc, cal, n_small, nm, pv), reps=2)
    out["scaled_rank"] = point(ms, 12.0 * big, Nc=big, n=n_small)
    # the same candidates against 2^22 calibration scores: with the index (three 32-byte loads per candidate from the
    # L2-resident index, bound by the rate at which an SM serves divergent loads) and without it
    bufb = torch.empty(n_big + k, device=dev)
    bufb[:n_big] = torch.sort(torch.randn(n_big, device=dev, generator=gen).exp_()).values
    calib_big = bufb[:n_big].clone()
    ixb = torch.empty(binding.calib_index_bytes(n_big + k), dtype=torch.uint8, device=dev)
    binding.calib_index_build(bufb, n_big, ixb)
    ms = graph_ms(lambda: binding.rank_classify_indexed(sc, bufb, n_big, ixb, (), nm, pv), reps=2)
    out["scaled_rank_large_buffer_indexed"] = point(ms, 12.0 * big + 4.0 * n_big, Nc=big, n=n_big)
    ms = graph_ms(lambda: binding.conformal_rank(sc, bufb, n_big, nm, pv), reps=1)
    out["scaled_rank_large_buffer_without_index"] = point(ms, 12.0 * big + 4.0 * n_big, Nc=big, n=n_big)
    binding.conformal_rank(sc, cal, n_small, nm, pv)
    ms = graph_ms(lambda: binding.classify(nm, n_small, 0.1, st, counts), reps=2)
    out["scaled_classify"] = point(ms, 5.0 * big, Nc=big)
    tau = torch.empty(1, device=dev)
    binding.threshold(cal, n_small, 0.1, tau)
    ms = graph_ms(lambda: binding.classify_threshold(sc, tau, st, counts), reps=2)
    out["scaled_classify_threshold"] = point(ms, 5.0 * big, Nc=big)
    # budget report: positions of the stage-3 samples among 2^26 (stages from the classify call above, alpha = 0.1)
    ids = torch.empty(big // 4, dtype=torch.int32, device=dev)
    cnt = torch.empty(1, dtype=torch.int32, device=dev)
    ws_ids = torch.empty(binding.takeover_ids_workspace_bytes(big), dtype=torch.uint8, device=dev)
    binding.classify(nm, n_small, 0.1, st, counts)
    ms = graph_ms(lambda: binding.takeover_ids(st, ids, cnt, ws_ids), reps=2)
    B = int(cnt.cpu().numpy().view(np.uint32)[0])
    out["scaled_takeover_ids"] = point(ms, 1.0 * big + 4.0 * B, Nc=big, B=B,
                                       note="one pass: every stage byte read once, every position written once")
    del ids, ws_ids
    # conditional coverage: 2^24 candidates, each ranked against its own input's 64 calibration scores
    ncond, G, m = 1 << 24, 1 << 16, 64
    segs = torch.sort(torch.randn(G, m, device=dev, generator=gen).exp_(), dim=1).values.reshape(-1).contiguous()
    seg_off = (torch.arange(G + 1, device=dev, dtype=torch.int64) * m).to(torch.int32)
    gid = torch.randint(0, G, (ncond,), device=dev, dtype=torch.int32, generator=gen)
    dn = torch.empty(ncond, dtype=torch.int32, device=dev)
    ms = graph_ms(lambda: binding.conformal_rank_conditional(sc[:ncond], gid, segs, seg_off, nm[:ncond], dn, pv[:ncond]), reps=2)
    cbytes = 20.0 * ncond    # score + group id in, numer + denom + p out
    out["scaled_rank_conditional"] = point(ms, cbytes, Nc=ncond, groups=G, group_size=m)
    # the same with the candidates of one input adjacent (how a batch of per-input samples arrives)
    gid_grouped = torch.sort(gid).values
    ms = graph_ms(lambda: binding.conformal_rank_conditional(sc[:ncond], gid_grouped, segs, seg_off, nm[:ncond], dn, pv[:ncond]), reps=2)
    out["scaled_rank_conditional_grouped"] = point(ms, cbytes, Nc=ncond, groups=G, group_size=m,
                                                   note="group ids non-decreasing: candidates of one input are adjacent")
    del sc, nm, pv, st, gid, gid_grouped, dn, segs
    # merge-insert of 4096 scores into 2^22: the call without an index (merge into the workspace + copy back, timed
    # with a restoring copy that is subtracted) and the indexed call (one pass, no copy back)
    wsb = torch.empty(binding.calib_workspace_bytes(n_big, k), dtype=torch.uint8, device=dev)

    def restore():
        bufb[:n_big] = calib_big

    ms_restore = graph_ms(restore, reps=4)

    def upd_plain():
        restore()
        binding.calib_update(bufb, n_big, new0, wsb)

    ms = graph_ms(upd_plain, reps=4) - ms_restore
    out["scaled_update"] = point(ms, update_bytes(n_big, k), n=n_big, k=k,
                                 note="merge into the workspace, then a copy back: the implementation moves 16 (n + k) bytes")
    restore()
    binding.calib_index_build(bufb, n_big, ixb)
    ms = graph_ms(lambda: binding.calib_update_indexed(bufb, n_big, new0, ixb, wsb), reps=4)
    out["scaled_update_indexed"] = point(ms, update_bytes(n_big, k), n=n_big, k=k,
                                         note="one pass from one half of the index into the other half and the buffer: "
                                              "the implementation moves 12 (n + k) bytes")
    out["bytes"] = "algorithmic: rank 12 Nc (+ 4 n), classify 5 Nc, budget report Nc + 4 B, merge-insert 8 (n + k) + 4 k"
    return out


def per_config_leg(torch, binding, peaks, name, dev, target_ms=1000.0):
    """One of the other workload shapes, timed like the bench line's device-resident leg: step = score + rank +
    classify at each of the shape's alphas + calibration update.  The inputs have the recipe's distributions but are
    drawn on the device (torch Philox) to keep the whole benchmark within minutes."""
    c = inputs.CONFIGS[name]
    N, T, d, V, n0, alphas = c["N"], c["T"], c["d"], c["V"], c["n"], c["alphas"]
    M = N * T
    gen = torch.Generator(device=dev)
    gen.manual_seed(inputs.BASE_SEED + 200 + sorted(inputs.CONFIGS).index(name))
    W_d = torch.empty(V, d, dtype=torch.bfloat16, device=dev)
    for r0 in range(0, V, 16384):
        r1 = min(r0 + 16384, V)
        W_d[r0:r1] = (torch.randn(r1 - r0, d, device=dev, generator=gen) * 0.02).to(torch.bfloat16)
    cdf = torch.cumsum(torch.arange(1, V + 1, device=dev, dtype=torch.float64) ** -1.1, 0)
    cdf /= cdf[-1].clone()
    off_d = torch.from_numpy(inputs.seg_offsets(N, T)).to(dev)

    def draw_batch(H):
        for r0 in range(0, M, 8192):
            x = torch.randn(min(8192, M - r0), d, device=dev, generator=gen)
            H[r0:r0 + x.shape[0]] = (x / x.pow(2).mean(1, keepdim=True).sqrt()).to(torch.bfloat16)
        u = torch.rand(M, device=dev, dtype=torch.float64, generator=gen)
        return torch.searchsorted(cdf, u, right=True).clamp_(max=V - 1).to(torch.int32)

    H_d = torch.empty(M, d, dtype=torch.bfloat16, device=dev)
    score_d = torch.empty(N, device=dev)
    numer = torch.empty(N, dtype=torch.int32, device=dev)
    pval = torch.empty(N, device=dev)
    stage = torch.empty(N, dtype=torch.uint8, device=dev)
    counts = torch.empty(3, dtype=torch.int32, device=dev)
    ws_s = torch.empty(binding.score_workspace_bytes(M, d, V, N), dtype=torch.uint8, device=dev)
    cap = n0 + N * 2100
    calib = torch.empty(cap, device=dev)
    ws_c = torch.empty(binding.calib_workspace_bytes(cap, N), dtype=torch.uint8, device=dev)
    n = 0
    for _ in range(n0 // N):       # calibration buffer: n0 scores of calibration batches through the same calls
        ids_c = draw_batch(H_d)
        binding.score_logprob(H_d, W_d, ids_c, off_d, None, score_d, ws_s)
        n = binding.calib_update(calib, n, score_d, ws_c)
    ids_d = draw_batch(H_d)
    state = {"n": n}

    def step():
        binding.score_logprob(H_d, W_d, ids_d, off_d, None, score_d, ws_s)
        binding.conformal_rank(score_d, calib, state["n"], numer, pval)
        for alpha in alphas:
            binding.classify(numer, state["n"], alpha, stage, counts)
        state["n"] = binding.calib_update(calib, state["n"], score_d, ws_c)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(3):
        step()
    e1.record()
    torch.cuda.synchronize()
    est = e0.elapsed_time(e1) / 3
    K = int(min(2000, max(10, target_ms / max(est, 1e-3))))
    binding.profile_begin(K)
    e0.record()
    for _ in range(K):
        step()
    e1.record()
    torch.cuda.synchronize()
    k1 = binding.profile_end()
    ms = e0.elapsed_time(e1) / K
    if binding.last_device_status() != 0:
        raise RuntimeError(f"device status set while timing the {name} shape")
    k1_ms = sum(k1) / len(k1)
    tflops = 2.0 * M * d * V / (k1_ms * 1e-3) / 1e12
    return {"workload": f"N={N} x T={T}, d={d}, V={V}, n={n0}, alphas {list(alphas)}", "steps": K, "ms_per_step": ms,
            "tokens_per_s": M / (ms * 1e-3), "fused_kernel_ms": k1_ms, "fused_kernel_tflops": tflops,
            "frac_of_sustained_peak": tflops / peaks["bf16_tflops_sustained"], "frac_of_burst_peak": tflops / peaks["bf16_tflops"],
            "data": "synthetic, drawn on the device with the recipe's distributions",
            "l2": "inputs larger than L2" if (V * d * 2 + M * d * 2) > (126 << 20) else
                  "inputs fit in L2 (W %.1f MB + H %.1f MB): warm-cache figure" % (V * d * 2 / 1e6, M * d * 2 / 1e6)}


def run_ours(args):
    import torch
    from paper_2509_15148_b200 import binding, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    binding.load()
    peaks, peak_kind = measured_peaks()
    if args.conformal_only or args.conformal_scaled_only:
        if rank == 0:
            res = (conformal_scaled(torch, binding, peaks, make_graph_timer(torch)) if args.conformal_scaled_only
                   else conformal_stress(torch, binding, peaks))
            print(json.dumps({"conformal_stress": res}), flush=True)
        return

    c = inputs.CONFIGS[args.workload]
    N, T, d, V, n0 = c["N"], c["T"], c["d"], c["V"], c["n"]
    M = N * T
    K, Wm = args.steps, args.warmup
    dev = torch.device("cuda", local)

    # ---- synthetic inputs (seeded) ----
    Wb = inputs.lm_head(inputs.BASE_SEED, V, d)
    W_d = torch.from_numpy(Wb.view(np.int16)).to(dev).view(torch.bfloat16)
    Hb = inputs.hidden(sharding.rank_seed(inputs.BASE_SEED, rank, 1), M, d)
    H_host = torch.from_numpy(Hb.view(np.int16)).view(torch.bfloat16).pin_memory()
    ids_host = torch.from_numpy(inputs.zipf_ids(sharding.rank_seed(inputs.BASE_SEED, rank, 2), M, V)).pin_memory()
    off_host = torch.from_numpy(inputs.seg_offsets(N, T)).pin_memory()
    H_d, ids_d, off_d = H_host.to(dev), ids_host.to(dev), off_host.to(dev)

    score_d = torch.empty(N, device=dev)
    numer = torch.empty(N, dtype=torch.int32, device=dev)
    pval = torch.empty(N, device=dev)
    stage = torch.empty(N, dtype=torch.uint8, device=dev)
    counts = torch.empty(3, dtype=torch.int32, device=dev)
    cap = n0 + N * world * (2 * K + 2 * Wm + 16)
    calib = torch.empty(cap, device=dev)
    ws_s = torch.empty(binding.score_workspace_bytes(M, d, V, N), dtype=torch.uint8, device=dev)
    ws_c = torch.empty(binding.calib_workspace_bytes(cap, N * world), dtype=torch.uint8, device=dev)
    res_host = {"stage": torch.empty(N, dtype=torch.uint8).pin_memory(), "counts": torch.empty(3, dtype=torch.int32).pin_memory(),
                "pval": torch.empty(N).pin_memory(), "score": torch.empty(N).pin_memory()}

    # ---- calibration prefill (untimed): n0 scores from calibration batches drawn on the device with the same
    # distribution (identical on every rank), scored through the same kernel and merge-inserted ----
    gen = torch.Generator(device=dev)
    gen.manual_seed(inputs.BASE_SEED + 100)
    cdf = torch.cumsum(torch.arange(1, V + 1, device=dev, dtype=torch.float64) ** -1.1, 0)
    cdf /= cdf[-1].clone()
    n = 0
    Hc = torch.empty(M, d, dtype=torch.bfloat16, device=dev)
    for _ in range(n0 // N):
        for r0 in range(0, M, 8192):
            x = torch.randn(min(8192, M - r0), d, device=dev, generator=gen)
            Hc[r0:r0 + x.shape[0]] = (x / x.pow(2).mean(1, keepdim=True).sqrt()).to(torch.bfloat16)
        u = torch.rand(M, device=dev, dtype=torch.float64, generator=gen)
        idc = torch.searchsorted(cdf, u, right=True).clamp_(max=V - 1).to(torch.int32)
        binding.score_logprob(Hc, W_d, idc, off_d, None, score_d, ws_s)
        n = binding.calib_update(calib, n, score_d, ws_c)
    del Hc, cdf
    if binding.last_device_status() != 0:
        raise RuntimeError("device status set during calibration prefill")

    state = {"n": n}

    def step(_unused: bool = False):
        binding.score_logprob(H_d, W_d, ids_d, off_d, None, score_d, ws_s)
        new = sharding.all_gather_scores(score_d, world, dist)
        binding.conformal_rank(score_d, calib, state["n"], numer, pval)
        binding.classify(numer, state["n"], ALPHA, stage, counts)
        state["n"] = binding.calib_update(calib, state["n"], new, ws_c)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if world == 1:
            return x
        t = torch.tensor([x], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    # ---- device-timed leg: inputs resident in HBM ----
    for _ in range(Wm):
        step(False)
    sampler = ClockSampler(str(torch.cuda.get_device_properties(dev).uuid) if hasattr(torch.cuda.get_device_properties(dev), "uuid") else str(local))
    if not sampler.gpu_id.startswith("GPU-"):
        sampler.gpu_id = "GPU-" + sampler.gpu_id if len(sampler.gpu_id) > 8 else str(local)
    barrier()
    if rank == 0:
        sampler.start()
    binding.profile_begin(max(K, 1))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(K):
        step(False)
    e1.record()
    barrier()
    k1_ms = binding.profile_end()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    stage_counts_last = counts.cpu().numpy().astype(np.int64).tolist()
    if binding.last_device_status() != 0:
        raise RuntimeError("device status set during the timed region")

    # ---- end-to-end leg: every step's inputs come from pinned host memory and its results go back to the host.
    # Two device input buffers: the copy of step i + 1 runs on a second stream while step i computes, and the
    # host reads step i's results while step i + 1 is in flight (nothing in the path waits for the host).
    cur = torch.cuda.current_stream()
    copy_stream = torch.cuda.Stream(device=dev)
    bufs = [(H_d, ids_d, off_d), (torch.empty_like(H_d), torch.empty_like(ids_d), torch.empty_like(off_d))]
    ready = [torch.cuda.Event(), torch.cuda.Event()]
    free = [torch.cuda.Event(), torch.cuda.Event()]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    res = [res_host, {k: torch.empty_like(v).pin_memory() for k, v in res_host.items()}]

    def e2e_steps(count: int):
        for b in (0, 1):
            free[b].record(cur)
        for i in range(count):
            b = i & 1
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(free[b])
                bufs[b][0].copy_(H_host, non_blocking=True)
                bufs[b][1].copy_(ids_host, non_blocking=True)
                bufs[b][2].copy_(off_host, non_blocking=True)
                ready[b].record(copy_stream)
            cur.wait_event(ready[b])
            binding.score_logprob(bufs[b][0], W_d, bufs[b][1], bufs[b][2], None, score_d, ws_s)
            free[b].record(cur)
            new = sharding.all_gather_scores(score_d, world, dist)
            binding.conformal_rank(score_d, calib, state["n"], numer, pval)
            binding.classify(numer, state["n"], ALPHA, stage, counts)
            state["n"] = binding.calib_update(calib, state["n"], new, ws_c)
            res[b]["stage"].copy_(stage, non_blocking=True)
            res[b]["counts"].copy_(counts, non_blocking=True)
            res[b]["pval"].copy_(pval, non_blocking=True)
            res[b]["score"].copy_(score_d, non_blocking=True)
            done[b].record(cur)
            if i >= 1:
                done[b ^ 1].synchronize()      # the host has step i - 1's stages, counts, p-values and scores
        done[(count - 1) & 1].synchronize()

    e2e_steps(min(Wm, 3))
    barrier()
    e0.record()
    e2e_steps(K)
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1))
    h2d = H_host.numel() * 2 + ids_host.numel() * 4 + off_host.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in res_host.values())

    # ---- extension entry points on the same batch (reported beside the line, not part of the step) ----
    ext = None
    if rank == 0:
        rs = torch.empty(M, device=dev)
        tau = torch.empty(1, device=dev)
        binding.rms_inv(H_d, 1e-6, rs)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(5):
            binding.rms_inv(H_d, 1e-6, rs)
        e1.record()
        torch.cuda.synchronize()
        ms_rms = e0.elapsed_time(e1) / 5
        binding.profile_begin(4)
        for _ in range(2):
            binding.score_logprob_scaled(H_d, W_d, ids_d, rs, off_d, None, score_d, ws_s)
        ms_scaled = binding.profile_end()[-1]
        binding.threshold(calib, state["n"], ALPHA, tau)
        binding.classify_threshold(score_d, tau, stage, counts)
        torch.cuda.synchronize()
        ext = {"rms_inv_ms": ms_rms, "rms_inv_gbs": (M * d * 2 + M * 4) / (ms_rms * 1e-3) / 1e9,
               "rms_inv_frac_hbm": (M * d * 2 + M * 4) / (ms_rms * 1e-3) / 1e9 / peaks["hbm_gbs"],
               "scaled_score_kernel_ms": ms_scaled,
               "note": "atts_rms_inv reads H once; atts_score_logprob_scaled folds the row factor into the epilogue"}

    # ---- the library GEMM on the same GPU in the same run (context for the roofline fraction: chips and boxes differ in
    # what the power cap lets them sustain): torch.matmul of the bench shape, which writes the M x V logits the fused
    # kernel never materialises (no softmax), and the square shape the measured peak was taken on ----
    lib_gemm = None
    if rank == 0 and world == 1 and not args.no_library_gemm:
        try:
            logits = torch.empty((M, V), dtype=torch.bfloat16, device=dev)
            for _ in range(2):
                torch.matmul(H_d, W_d.t(), out=logits)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(8):
                torch.matmul(H_d, W_d.t(), out=logits)
            e1.record()
            torch.cuda.synchronize()
            ms_same = e0.elapsed_time(e1) / 8
            # the library route to the same outputs: materialised bf16 logits, then torch's cross entropy over them
            ids64 = ids_d.long()
            torch.nn.functional.cross_entropy(logits, ids64, reduction="none")
            torch.cuda.synchronize()
            e0.record()
            for _ in range(3):
                torch.matmul(H_d, W_d.t(), out=logits)
                torch.nn.functional.cross_entropy(logits, ids64, reduction="none")
            e1.record()
            torch.cuda.synchronize()
            ms_route = e0.elapsed_time(e1) / 3
            del logits, ids64
            a = torch.randn((8192, 8192), dtype=torch.bfloat16, device=dev)
            b = torch.randn((8192, 8192), dtype=torch.bfloat16, device=dev)
            c = torch.empty((8192, 8192), dtype=torch.bfloat16, device=dev)
            for _ in range(20):
                torch.matmul(a, b, out=c)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(1500):
                torch.matmul(a, b, out=c)
            e1.record()
            torch.cuda.synchronize()
            ms_sq = e0.elapsed_time(e1) / 1500
            del a, b, c
            lib_gemm = {"same_shape_ms": ms_same, "same_shape_tflops": 2.0 * M * d * V / (ms_same * 1e-3) / 1e12,
                        "matmul_plus_cross_entropy_ms": ms_route,
                        "matmul_plus_cross_entropy_tokens_per_s": M / (ms_route * 1e-3),
                        "square_8192_tflops_sustained": 2.0 * 8192 ** 3 / (ms_sq * 1e-3) / 1e12,
                        "note": "torch.matmul (cuBLAS) on this GPU in this run: the bench shape with the M x V bf16 logits "
                                f"written to HBM ({M * V * 2 / 1e9:.1f} GB, no softmax, 8 back-to-back calls); the same followed by "
                                "torch's cross_entropy over those bf16 logits (per-token log-probs at bf16 logit precision, "
                                "not the 2e-3 contract); and 1500 back-to-back 8192^3 products"}
        except RuntimeError as exc:   # e.g. not enough free memory for the logits
            lib_gemm = {"unavailable": str(exc)[:120]}
        torch.cuda.empty_cache()

    tokens = M * world * K
    value = tokens / (ms_total * 1e-3)
    k1_avg = sum(k1_ms) / len(k1_ms)
    flops = 2.0 * M * d * V
    achieved = flops / (k1_avg * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"{args.workload.upper()}-target shape: N={N} samples x T={T} tokens per GPU, d={d}, V={V}, online calibration "
                               f"n={n0} growing by {N * world} per step, alpha={ALPHA}",
                   "step": "score_logprob + conformal_rank + classify + calib_update",
                   "l2": f"inputs larger than L2 (H {M * d * 2 / 1e6:.0f} MB, W {V * d * 2 / 1e6:.0f} MB per step), no flush needed",
                   "parallelism": f"dp{world}: samples sharded, W replicated, all-gather of {N} scores per rank"
                   if world > 1 else "single GPU"},
        "clocks": clocks,
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / K,
                "pipeline": "two input buffers: the host-to-device copy of step i+1 overlaps step i on a second stream; "
                            "the host reads step i's results while step i+1 runs"},
        "gpu_launches": KERNELS_PER_STEP * K,
        "roofline": {"bound": "tensor", "kernel": "lmhead_lse_kernel", "achieved": achieved,
                     "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": achieved / peaks["bf16_tflops_sustained"], "peak_kind": f"{peak_kind}, sustained bf16 GEMM "
                     "(kernel timed inside a long step)", "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                     "kernel_ms": k1_avg, "flops_per_launch": flops,
                     "traffic": k1_traffic_bytes() if args.workload == WORKLOAD else None,
                     "traffic_note": "stored figure: dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of "
                                     "this kernel source on this workload (mean of 3 launches), not measured in this run; "
                                     "captures on other boxes and builds ranged 45-105 GB per launch; null once the kernel source changes"},
        "stage_counts_last_step": stage_counts_last, "calib_n_end": state["n"],
    }
    # Asynchronous arithmetic intensity of the step (the paper's r = T_c / (T_m + T_s)): T_c the fused kernel's time,
    # T_m the time the step's algorithmic bytes would take at the measured copy bandwidth, T_s everything of the
    # step that is not the fused kernel (launch gaps, the six microsecond-scale kernels, the all-gather): an upper
    # bound on synchronisation.  The calls never wait for the host, so T_s stays at launch-latency scale.
    alg_bytes = V * d * 2 + M * d * 2 + M * 4 + (N + 1) * 4
    t_m = alg_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3
    t_s = max(ms_total / K - k1_avg, 0.0)
    line["async_arithmetic_intensity"] = {"T_c_ms": k1_avg, "T_m_ms": t_m, "T_s_ms_upper": t_s,
                                          "r": k1_avg / (t_m + t_s)}
    if ext is not None:
        line["extensions"] = ext
    if lib_gemm is not None:
        line["library_gemm"] = lib_gemm
        if "same_shape_tflops" in lib_gemm:
            line["roofline"]["frac_of_library_gemm_same_shape_same_gpu"] = achieved / lib_gemm["same_shape_tflops"]
    if rank == 0 and world == 1:
        if not args.no_cpu_baseline:
            from oracle import atts_oracle as orc
            # one whole draft sample plus token rows scattered over the rest of the batch
            whole = 1 if args.oracle_rows >= 256 else 0
            plan = oracle_rows_plan(M, T, whole, args.oracle_rows, inputs.BASE_SEED + 9)
            cal = calib[:state["n"]].cpu().numpy()
            ids_np = ids_host.numpy()
            rest = score_d.cpu().numpy()[whole:]        # the other samples' scores feed the conformal steps
            t0 = time.perf_counter()
            oracle_step(orc, Hb[plan], Wb, ids_np[plan], whole * T, T, rest, cal, ALPHA)
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": plan.size / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                    "sample": f"{plan.size} of {M} token rows of the same batch (full d and V) in {dt:.1f} s: "
                                              f"{whole} whole sample(s) of {T} tokens plus {plan.size - whole * T} rows scattered "
                                              f"over the rest by a seeded permutation; then rank/classify/update on N={N} scores"}
            line["cpu_baseline"]["conformal_only"] = oracle_conformal_steps(orc)
        del H_d, W_d, bufs
        torch.cuda.empty_cache()
        if not args.no_per_config and args.workload == WORKLOAD:
            line["per_config"] = {name: per_config_leg(torch, binding, peaks, name, dev)
                                  for name in ("tiny", "7b", "70b")}
            torch.cuda.empty_cache()
        if not args.no_conformal:
            line["conformal_stress"] = conformal_stress(torch, binding, peaks)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--oracle-rows", type=int, default=256, help="token rows the CPU oracle scores per step")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(inputs.CONFIGS),
                    help="shape to run (default: the bench line's workload; others are for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-conformal", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the tiny / 7B / 70B shapes beside the bench line")
    ap.add_argument("--no-library-gemm", action="store_true", help="skip the torch.matmul comparison on the same GPU")
    ap.add_argument("--conformal-scaled-only", action="store_true",
                    help="run only the HBM-scale points of the conformal kernels (for profiling)")
    ap.add_argument("--conformal-only", action="store_true",
                    help="run only the conformal-only workload section and print it (for profiling those kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2509_15148_b200 import sharding
    if sharding.needs_launch(args.gpus, os.environ):
        # started as a plain `python bench.py --gpus N`: start the N ranks (one per GPU) and hand over to them
        cmd, env = sharding.launch_command(os.path.abspath(__file__), sys.argv[1:], args.gpus, sharding.free_port(),
                                           sys.executable, os.environ)
        sys.exit(subprocess.run(cmd, env=env).returncode)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
