"""Thin Python binding of libatts (ctypes): argument marshalling only.

Every function takes torch CUDA tensors, passes their device pointers and the current
CUDA stream to the C entry point of the same name (include/atts.h), and raises
:class:`AttsError` on a non-zero status.  Nothing is computed here, and there is no
fallback: if the CUDA library cannot be loaded, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_double, c_int, c_int32, c_int64, c_size_t, c_void_p, c_char_p, POINTER, c_uint32

from . import build as _build

EXPORTS = (
    "atts_strerror", "atts_version", "atts_score_workspace_bytes", "atts_score_logprob",
    "atts_conformal_rank", "atts_classify", "atts_calib_workspace_bytes", "atts_calib_update",
    "atts_last_device_status", "atts_profile_begin", "atts_profile_end",
    "atts_calib_update_static", "atts_rank_classify", "atts_score_logprob_scaled", "atts_rms_inv",
    "atts_threshold", "atts_classify_threshold", "atts_conformal_rank_conditional", "atts_classify_conditional",
    "atts_debug_score_plan", "atts_debug_score_unit", "atts_score_slice", "atts_score_combine",
    "atts_calib_index_bytes", "atts_calib_index_build", "atts_calib_update_indexed", "atts_rank_classify_indexed",
    "atts_takeover_ids_workspace_bytes", "atts_takeover_ids", "atts_debug_set_wait", "atts_debug_score_form",
)

STAGE_DRAFT, STAGE_ACCEPTED, STAGE_TARGET = 1, 2, 3
DEV_TOKEN_ID_RANGE, DEV_WAIT_EXPIRED, DEV_GROUP_ID_RANGE, DEV_INDEX_STALE = 1, 2, 4, 8

_lib = None


class AttsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


def load(rebuild_if_stale: bool = True) -> ctypes.CDLL:
    """Load libatts.so from the package directory (building it first if the sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if rebuild_if_stale and _build.is_stale():
        # A library older than its sources is never loaded: if it cannot be rebuilt (no nvcc, or the sources no
        # longer compile) this raises, so that nothing runs on a binary that does not match the tree.
        _build.build_library()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2509_15148_b200.build`")
    lib = ctypes.CDLL(path)
    lib.atts_strerror.restype = c_char_p
    lib.atts_strerror.argtypes = [c_int]
    lib.atts_version.restype = c_int
    lib.atts_score_workspace_bytes.argtypes = [c_int64, c_int64, c_int64, c_int64, POINTER(c_size_t)]
    lib.atts_score_logprob.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int64,
                                       c_int32, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.atts_conformal_rank.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_void_p, c_void_p]
    lib.atts_classify.argtypes = [c_void_p, c_int64, c_int64, c_double, c_void_p, c_void_p, c_void_p]
    lib.atts_rank_classify.argtypes = [c_void_p, c_int64, c_void_p, c_int64, POINTER(c_double), c_int32, c_void_p, c_void_p,
                                       c_void_p, c_void_p, c_void_p]
    lib.atts_score_logprob_scaled.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64,
                                              c_int64, c_int32, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.atts_score_slice.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int64, c_void_p, c_void_p,
                                     c_size_t, c_void_p]
    lib.atts_score_combine.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_int64, c_int32, c_void_p, c_void_p, c_void_p,
                                       c_size_t, c_void_p]
    lib.atts_rms_inv.argtypes = [c_void_p, c_int64, c_int64, ctypes.c_float, c_void_p, c_void_p]
    lib.atts_threshold.argtypes = [c_void_p, c_int64, c_double, c_void_p, c_void_p]
    lib.atts_classify_threshold.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.atts_conformal_rank_conditional.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_int64,
                                                    c_void_p, c_void_p, c_void_p, c_void_p]
    lib.atts_classify_conditional.argtypes = [c_void_p, c_void_p, c_int64, c_double, c_void_p, c_void_p, c_void_p]
    lib.atts_debug_score_plan.argtypes = [c_int64, c_int64, c_int64, c_int32, c_int32, POINTER(c_int32)]
    lib.atts_debug_score_unit.argtypes = [c_int64, c_int64, c_int64, c_int32, c_int32, c_int32, POINTER(c_int32)]
    lib.atts_calib_workspace_bytes.argtypes = [c_int64, c_int64, POINTER(c_size_t)]
    lib.atts_calib_update.argtypes = [c_void_p, c_int64, c_int64, c_void_p, c_int64, POINTER(c_int64), c_void_p,
                                      c_size_t, c_void_p]
    lib.atts_last_device_status.argtypes = [c_void_p, POINTER(c_uint32)]
    lib.atts_calib_update_static.argtypes = [c_void_p, c_int64, c_int64, c_void_p, c_int64, POINTER(c_int64), c_void_p]
    lib.atts_calib_index_bytes.argtypes = [c_int64, POINTER(c_size_t)]
    lib.atts_calib_index_build.argtypes = [c_void_p, c_int64, c_void_p, c_size_t, c_void_p]
    lib.atts_calib_update_indexed.argtypes = [c_void_p, c_int64, c_int64, c_void_p, c_int64, POINTER(c_int64), c_void_p,
                                              c_size_t, c_void_p, c_size_t, c_void_p]
    lib.atts_rank_classify_indexed.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_void_p, POINTER(c_double), c_int32,
                                               c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.atts_takeover_ids_workspace_bytes.argtypes = [c_int64, POINTER(c_size_t)]
    lib.atts_takeover_ids.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.atts_debug_set_wait.argtypes = [c_int64, c_int32]
    lib.atts_debug_score_form.argtypes = [c_int64, c_int64, c_int64, POINTER(c_int32)]
    lib.atts_profile_begin.argtypes = [c_int]
    lib.atts_profile_end.argtypes = [POINTER(ctypes.c_float), c_int, POINTER(c_int)]
    for name in EXPORTS[2:]:
        getattr(lib, name).restype = c_int
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().atts_strerror(int(status)).decode()


def version() -> int:
    return load().atts_version()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise AttsError(status, where)


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def score_workspace_bytes(M: int, d: int, V: int, S: int) -> int:
    out = c_size_t(0)
    _check(load().atts_score_workspace_bytes(M, d, V, S, ctypes.byref(out)), "atts_score_workspace_bytes")
    return out.value


def score_logprob(hidden, lm_head, token_ids, seg_offsets, token_logprob, sample_score, workspace,
                  score_mode: int = 0) -> None:
    """hidden [M,d] bf16, lm_head [V,d] bf16, token_ids [M] i32, seg_offsets [S+1] i32 ->
    token_logprob [M] f32 (or None), sample_score [S] f32; workspace: uint8 tensor."""
    M, d = hidden.shape
    V = lm_head.shape[0]
    S = seg_offsets.numel() - 1
    _check(load().atts_score_logprob(_ptr(hidden), _ptr(lm_head), _ptr(token_ids), _ptr(seg_offsets), M, d, V, S,
                                     score_mode, _ptr(token_logprob), _ptr(sample_score), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream()), "atts_score_logprob")


def score_logprob_scaled(hidden, lm_head, token_ids, row_scale, seg_offsets, token_logprob, sample_score, workspace,
                         score_mode: int = 0) -> None:
    """score_logprob with logits of row i multiplied by row_scale[i] (f32 [M], finite and > 0)."""
    M, d = hidden.shape
    V = lm_head.shape[0]
    S = seg_offsets.numel() - 1
    _check(load().atts_score_logprob_scaled(_ptr(hidden), _ptr(lm_head), _ptr(token_ids), _ptr(row_scale),
                                            _ptr(seg_offsets), M, d, V, S, score_mode, _ptr(token_logprob),
                                            _ptr(sample_score), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream()),
           "atts_score_logprob_scaled")


def score_slice(hidden, lm_head_slice, token_ids, vocab_offset: int, slice_stats, workspace) -> None:
    """Per-token (max, sum exp, token logit or -inf) over one vocabulary slice: slice_stats [M, 3] f32."""
    M, d = hidden.shape
    _check(load().atts_score_slice(_ptr(hidden), _ptr(lm_head_slice), _ptr(token_ids), M, d, lm_head_slice.shape[0],
                                   int(vocab_offset), _ptr(slice_stats), _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream()), "atts_score_slice")


def score_combine(slice_stats, seg_offsets, token_logprob, sample_score, workspace, score_mode: int = 0) -> None:
    """Merge slice_stats [G, M, 3] (all ranks' blocks in rank order) into token log-probs and sample scores."""
    G, M = slice_stats.shape[0], slice_stats.shape[1]
    S = seg_offsets.numel() - 1
    _check(load().atts_score_combine(_ptr(slice_stats), G, _ptr(seg_offsets), M, S, score_mode, _ptr(token_logprob),
                                     _ptr(sample_score), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                     _stream()), "atts_score_combine")


def rms_inv(hidden, eps: float, row_scale) -> None:
    """row_scale[i] = 1 / sqrt(mean(hidden[i]^2) + eps)."""
    M, d = hidden.shape
    _check(load().atts_rms_inv(_ptr(hidden), M, d, float(eps), _ptr(row_scale), _stream()), "atts_rms_inv")


def threshold(calib_sorted, n: int, alpha: float, tau) -> None:
    """tau[0] = the floor(alpha (n + 1))-th largest of the first n calibration scores (+inf if that is 0)."""
    _check(load().atts_threshold(_ptr(calib_sorted), n, float(alpha), _ptr(tau), _stream()), "atts_threshold")


def classify_threshold(scores, tau, stage, stage_counts=None) -> None:
    """Stage per sample from s > tau[0]; stage_counts [3] or None."""
    _check(load().atts_classify_threshold(_ptr(scores), scores.numel(), _ptr(tau), _ptr(stage), _ptr(stage_counts),
                                          _stream()), "atts_classify_threshold")


def takeover_ids_workspace_bytes(Nc: int) -> int:
    out = c_size_t(0)
    _check(load().atts_takeover_ids_workspace_bytes(Nc, ctypes.byref(out)), "atts_takeover_ids_workspace_bytes")
    return out.value


def takeover_ids(stage, ids, count, workspace) -> None:
    """Positions (ascending, int32) of the samples in stage 3 into ids (as many as fit), their number into count[0]."""
    _check(load().atts_takeover_ids(_ptr(stage), stage.numel(), _ptr(ids), 0 if ids is None else ids.numel(), _ptr(count),
                                    _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream()), "atts_takeover_ids")


def conformal_rank_conditional(scores, group_ids, calib_segments, seg_offsets, numer, denom, pvalue=None) -> None:
    """Rank each score against the ascending calibration segment of its own group."""
    _check(load().atts_conformal_rank_conditional(_ptr(scores), _ptr(group_ids), scores.numel(), _ptr(calib_segments),
                                                  calib_segments.numel(), _ptr(seg_offsets), seg_offsets.numel() - 1,
                                                  _ptr(numer), _ptr(denom), _ptr(pvalue), _stream()),
           "atts_conformal_rank_conditional")


def classify_conditional(numer, denom, alpha: float, stage, stage_counts=None) -> None:
    _check(load().atts_classify_conditional(_ptr(numer), _ptr(denom), numer.numel(), float(alpha), _ptr(stage),
                                            _ptr(stage_counts), _stream()), "atts_classify_conditional")


def conformal_rank(scores, calib_sorted, n: int, numer, pvalue=None) -> None:
    """scores [Nc] f32, calib_sorted (first n entries used) -> numer [Nc] u32 (int32 storage), pvalue [Nc] f32."""
    _check(load().atts_conformal_rank(_ptr(scores), scores.numel(), _ptr(calib_sorted), n, _ptr(numer), _ptr(pvalue),
                                      _stream()), "atts_conformal_rank")


def classify(numer, n: int, alpha: float, stage, stage_counts=None) -> None:
    """numer [Nc] u32 -> stage [Nc] u8, stage_counts [3] u32 (int32 storage) or None."""
    _check(load().atts_classify(_ptr(numer), numer.numel(), n, float(alpha), _ptr(stage), _ptr(stage_counts),
                                _stream()), "atts_classify")


def rank_classify(scores, calib_sorted, n: int, alphas, numer, pvalue, stage, stage_counts=None) -> None:
    """Rank and threshold at up to four alphas in one launch: stage [len(alphas), Nc] u8, stage_counts [len(alphas), 3]."""
    arr = (c_double * len(alphas))(*[float(a) for a in alphas])
    _check(load().atts_rank_classify(_ptr(scores), scores.numel(), _ptr(calib_sorted), n, arr, len(alphas), _ptr(numer),
                                     _ptr(pvalue), _ptr(stage), _ptr(stage_counts), _stream()), "atts_rank_classify")


def calib_workspace_bytes(n: int, k: int) -> int:
    out = c_size_t(0)
    _check(load().atts_calib_workspace_bytes(n, k, ctypes.byref(out)), "atts_calib_workspace_bytes")
    return out.value


def calib_update(calib, n: int, new_scores, workspace) -> int:
    """calib: f32 buffer of capacity calib.numel() whose first n entries are sorted; inserts new_scores in place.
    Returns the new fill n + k."""
    n_out = c_int64(0)
    k = 0 if new_scores is None else new_scores.numel()
    _check(load().atts_calib_update(_ptr(calib), n, calib.numel(), _ptr(new_scores), k, ctypes.byref(n_out),
                                    _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream()), "atts_calib_update")
    return n_out.value


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def calib_index_bytes(cap: int) -> int:
    out = c_size_t(0)
    _check(load().atts_calib_index_bytes(cap, ctypes.byref(out)), "atts_calib_index_bytes")
    return out.value


def calib_index_build(calib_sorted, n: int, index) -> None:
    """Write into `index` (uint8 tensor) the search index of the first n entries of calib_sorted."""
    _check(load().atts_calib_index_build(_ptr(calib_sorted), n, _ptr(index), _nbytes(index), _stream()),
           "atts_calib_index_build")


def calib_update_indexed(calib, n: int, new_scores, index, workspace) -> int:
    """:func:`calib_update` that also leaves in `index` the search index of the updated buffer. Returns n + k."""
    n_out = c_int64(0)
    k = 0 if new_scores is None else new_scores.numel()
    _check(load().atts_calib_update_indexed(_ptr(calib), n, calib.numel(), _ptr(new_scores), k, ctypes.byref(n_out),
                                            _ptr(index), _nbytes(index), _ptr(workspace), _nbytes(workspace), _stream()),
           "atts_calib_update_indexed")
    return n_out.value


def rank_classify_indexed(scores, calib_sorted, n: int, index, alphas, numer, pvalue=None, stage=None,
                          stage_counts=None) -> None:
    """:func:`rank_classify` with the buffer's search index; alphas may be empty (ranks and p-values only)."""
    arr = (c_double * max(len(alphas), 1))(*[float(a) for a in alphas])
    _check(load().atts_rank_classify_indexed(_ptr(scores), scores.numel(), _ptr(calib_sorted), n, _ptr(index), arr,
                                             len(alphas), _ptr(numer), _ptr(pvalue), _ptr(stage), _ptr(stage_counts),
                                             _stream()), "atts_rank_classify_indexed")


STATIC_MAX_TOTAL, STATIC_MAX_NEW = 65536, 16384


def calib_update_static(calib, n: int, new_scores) -> int:
    """Same as :func:`calib_update` without a workspace, for callers that cannot allocate device memory (an engine
    plug-in left with no free HBM, a loop that must not pay cudaMalloc's device-wide synchronisation): the scratch is
    a fixed array inside the library, so n + k <= STATIC_MAX_TOTAL and k <= STATIC_MAX_NEW (status 10 otherwise).
    All calls on a device share that array: keep them on one stream or order them, overlapping calls race.
    Make the first call on a device at start-up (it looks up the array's address). Returns n + k."""
    n_out = c_int64(0)
    k = 0 if new_scores is None else new_scores.numel()
    _check(load().atts_calib_update_static(_ptr(calib), n, calib.numel(), _ptr(new_scores), k, ctypes.byref(n_out),
                                           _stream()), "atts_calib_update_static")
    return n_out.value


def last_device_status() -> int:
    """Synchronises the current stream; returns and clears the device status bits. Raises on an expired wait or a
    stale calibration index."""
    bits = c_uint32(0)
    st = load().atts_last_device_status(_stream(), ctypes.byref(bits))
    if st != 0:
        raise AttsError(st, "atts_last_device_status")
    return bits.value


def debug_set_wait(limit_cycles: int = 0, withhold_loads: bool = False) -> None:
    """Bound (SM cycles; <= 0 restores the default) of the scoring kernel's pipeline waits for later calls, and the
    diagnostic switch that makes its producer issue no loads so that the first wait for data runs out."""
    _check(load().atts_debug_set_wait(int(limit_cycles), 1 if withhold_loads else 0), "atts_debug_set_wait")


def debug_score_form(M: int, d: int, V: int) -> int:
    """1 if score_logprob runs this shape on single CTAs on the current device, 2 if on CTA pairs."""
    out = c_int32(0)
    _check(load().atts_debug_score_form(M, d, V, ctypes.byref(out)), "atts_debug_score_form")
    return out.value


def profile_begin(max_records: int = 1024) -> None:
    """Start recording CUDA-event pairs around the fused scoring kernel of every score_logprob call."""
    _check(load().atts_profile_begin(int(max_records)), "atts_profile_begin")


def profile_end(cap: int = 4096) -> list[float]:
    """Stop recording; returns the fused kernel's durations in milliseconds, one per recorded call."""
    buf = (ctypes.c_float * cap)()
    cnt = c_int(0)
    _check(load().atts_profile_end(buf, cap, ctypes.byref(cnt)), "atts_profile_end")
    return [float(buf[i]) for i in range(min(cnt.value, cap))]


def debug_score_plan(M: int, d: int, V: int, workers: int, ctas: int) -> dict:
    """The fused kernel's static schedule for a shape (no device needed)."""
    out = (c_int32 * 8)()
    _check(load().atts_debug_score_plan(M, d, V, workers, ctas, out), "atts_debug_score_plan")
    return dict(zip(("RB", "NT", "KB", "C", "Gr", "units", "M_pad", "ctas"), list(out)))


def debug_score_unit(M: int, d: int, V: int, workers: int, ctas: int, u: int) -> tuple:
    """(row block, chunk, first tile, one past the last tile) of unit u of that schedule."""
    out = (c_int32 * 4)()
    _check(load().atts_debug_score_unit(M, d, V, workers, ctas, u, out), "atts_debug_score_unit")
    return tuple(out)
