"""The synthetic workload recipe, run end to end through the oracle on the tiny configuration."""
import numpy as np

import oracle
from paper_2608_21362_b200 import synth

import oracle_glue as helpers


def test_cfg0_recipe_and_selection_finds_the_seams():
    wl = synth.workload(0)
    sh = wl.shape
    (req,) = helpers.materialize_with_oracle(wl)
    assert req.plan.T == 512 and len(req.chunks) == 4
    modes = [c.plan.mode for c in req.chunks]
    assert sorted(modes) == [0, 2, 2, 2]
    kv, fresh = helpers.bits_of(req.kv_buf), helpers.bits_of(req.fresh)
    d64, d32 = oracle.deviation(kv, fresh, helpers.dt_code(sh), wl.select.which)
    k = oracle.select_count(req.plan.T, wl.select.ratio)
    assert k == 76
    rank = oracle.topk(d32, k)
    # the seam noise sits on the first 16 tokens of each cached chunk: all 48 must be selected
    seam = {c.plan.new_pos + i for c in req.chunks if c.plan.mode != 0 for i in range(16)}
    assert seam <= set(rank.tolist())
    # fresh chunks are bit copies, so they never deviate
    for c in req.chunks:
        if c.plan.mode == 0:
            assert np.all(d64[c.plan.new_pos : c.plan.new_pos + sh.C] == 0.0)
    sel = oracle.seam_select(rank, [c.plan.new_pos for c in req.chunks], modes, req.plan.T, 16, 0)
    assert k <= len(sel) <= req.sel_capacity and np.all(np.diff(sel) > 0)


def test_workload_plans_tile_the_prompt():
    for idx in range(5):
        wl = synth.workload(idx)
        for rp in wl.requests:
            assert [c.new_pos for c in rp.chunks] == list(range(0, rp.T, wl.shape.C))
            assert all(c.mode != 0 or c.orig_pos == c.new_pos for c in rp.chunks)
    assert len(synth.workload(4).requests) == 32
    assert synth.workload(2).requests[0].chunks == synth.workload(3).requests[0].chunks
