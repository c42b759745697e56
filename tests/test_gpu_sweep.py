"""The format search of Sec. 7.2 (Eq. 2) on the tiny configuration: a reduced grid runs end to end on the GPU, its
bookkeeping agrees with the oracle's objective, and the measured quantities behave as the format dictates."""
import pytest

import synth
from oracle import model

pytestmark = pytest.mark.gpu


def test_sweep_reduced_grid():
    from paper_2605_26558_b200 import sweep
    recs = sweep.sweep("tiny", steps=6, gamma=4, n_prompt=48, grid_p=(300, 600), grid_t=(0, 3, 4), search_kv=True)
    w = [r for r in recs if r["search"] == "weights"]
    kv = [r for r in recs if r["search"] == "kv"]
    assert len(w) == 6 and len(kv) == 4 and sum(r["best"] for r in recs) == 1
    shape = synth.TINY
    s_w = sweep._weight_values(shape)
    assert s_w == 2 * (512 * 256 + 256 * 256 + 3 * 688 * 256) + 1024 * 256
    for r in recs:
        assert r["status"] == 0 and 0.0 <= r["alpha"] <= 1.0 and r["tokens_per_s"] > 0
        assert abs(r["mean_accepted"] - 4 * r["alpha"]) < 1e-9
        ctx = 48 + 6 * 5 // 2
        s_kv = 2 * shape.n_layers * shape.n_kv_heads * shape.head_dim * ctx
        want = model.design_objective(r["alpha"], s_w, r["w_p"], r["w_t"], s_kv, r["kv_p"], r["kv_t"])
        assert abs(r["J"] - want) <= 1e-12 * max(want, 1e-30)
    by = {(r["w_p"], r["w_t"]): r for r in w}
    # content of the speculation data: 1 bitmap bit + kept * (sign + kept mantissa bits + codeword) per value
    for p in (0.3, 0.6):
        assert by[(p, 0)]["content_bits_per_weight"] > by[(p, 3)]["content_bits_per_weight"] > by[(p, 4)]["content_bits_per_weight"]
        d = by[(p, 0)]["content_bits_per_weight"] - by[(p, 4)]["content_bits_per_weight"]
        assert abs(d - 4 * (1 - p)) < 0.02                     # four mantissa bits of every kept value
    for t in (0, 3, 4):
        assert by[(0.3, t)]["content_bits_per_weight"] > by[(0.6, t)]["content_bits_per_weight"]
    best = next(r for r in recs if r["best"])
    assert best["J"] == max(r["J"] for r in recs)
