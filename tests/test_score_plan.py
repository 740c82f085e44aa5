"""Host logic of the fused kernel's static schedule (no GPU): every (row block, vocabulary tile) is covered by
exactly one unit, chunks are non-empty and contiguous, and the makespan stays close to the ideal."""
import math

import numpy as np
import pytest

from paper_2509_15148_b200 import binding, inputs

SHAPES = [(1, 64, 1), (128, 64, 256), (129, 128, 257), (300, 192, 1000), (1000, 320, 2049), (520, 1024, 12345),
          (70000, 64, 300)]
SHAPES += [(c["N"] * c["T"], c["d"], c["V"]) for c in inputs.CONFIGS.values()]


@pytest.mark.parametrize("M,d,V", SHAPES)
@pytest.mark.parametrize("workers,ctas", [(148, 1), (74, 2), (132, 1), (7, 2)])
def test_units_tile_the_problem_exactly_once(M, d, V, workers, ctas):
    p = binding.debug_score_plan(M, d, V, workers, ctas)
    rows = 128 * ctas
    assert p["RB"] == math.ceil(M / rows) and p["NT"] == math.ceil(V / 256) and p["KB"] == d // 64
    assert 1 <= p["C"] <= min(p["NT"], workers) and p["units"] == p["RB"] * p["C"]
    assert 1 <= p["Gr"] <= max(p["RB"], 1) and p["M_pad"] == p["RB"] * rows
    if p["units"] > 40000:
        pytest.skip("coverage loop too long for this shape")
    cover = np.zeros((p["RB"], p["NT"]), dtype=np.int32)
    seen = set()
    for u in range(p["units"]):
        rb, c, nt0, nt1 = binding.debug_score_unit(M, d, V, workers, ctas, u)
        assert 0 <= rb < p["RB"] and 0 <= c < p["C"] and 0 <= nt0 < nt1 <= p["NT"]
        assert (rb, c) not in seen
        seen.add((rb, c))
        cover[rb, nt0:nt1] += 1
    assert (cover == 1).all()


def test_makespan_close_to_ideal_on_the_model_shapes():
    for name, c in inputs.CONFIGS.items():
        if name == "tiny":
            continue
        M, d, V = c["N"] * c["T"], c["d"], c["V"]
        p = binding.debug_score_plan(M, d, V, 148, 1)
        waves = math.ceil(p["units"] / 148)
        span = waves * math.ceil(p["NT"] / p["C"])
        ideal = p["RB"] * p["NT"] / 148
        assert span <= 1.05 * ideal, (name, span, ideal)


def test_plan_argument_errors():
    import ctypes
    lib = binding.load()
    out = (ctypes.c_int32 * 8)()
    assert lib.atts_debug_score_plan(128, 100, 256, 148, 1, out) == 2
    assert lib.atts_debug_score_plan(128, 64, 256, 0, 1, out) == 6
    assert lib.atts_debug_score_plan(128, 64, 256, 148, 3, out) == 6
    assert lib.atts_debug_score_unit(128, 64, 256, 148, 1, 5, out) == 6
    assert lib.atts_debug_score_plan(128, 64, 256, 148, 1, None) == 1
