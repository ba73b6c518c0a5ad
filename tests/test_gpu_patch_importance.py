"""Parity of the two steps next to the main path: the patch of Algorithm 2 step 4 (bit-exact row
replacement) and the chunk importance of Eq. 7 (float32 norms, 1e-5 relative)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import oracle_glue as helpers
from test_gpu_parity import prepare, run_assemble, run_select

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("idx,n_req,table", [(0, None, False), (4, 3, False), (4, 3, True)])
def test_patch_matches_oracle(idx, n_req, table):
    """table: the descriptors go through the uploaded table (the route of calls with more requests than fit
    the kernel's own argument) instead of travelling with the launch."""
    build_library()
    wl = synth.workload(idx, n_req) if n_req else synth.workload(idx)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        before = [helpers.bits_of(r.kv_buf) for r in reqs]
        if table:
            B.kvb_set_debug_option(ctx, "descriptor_copy", 1)
        B.kvb_patch(ctx, tbl, sel)
        B.kvb_last_status(ctx)
        for i, r in enumerate(reqs):
            n = int(sel.n_sel[i])
            idxs = sel.sel[i].cpu().numpy()[:n]
            want = oracle.patch(before[i], helpers.bits_of(r.fresh), idxs)
            assert np.array_equal(helpers.bits_of(r.kv_buf), want)  # selected rows replaced, all others untouched
        # after the patch the selected positions no longer deviate
        sel2, _, _ = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        for i, r in enumerate(reqs):
            n = int(sel.n_sel[i])
            idxs = torch.from_numpy(sel.sel[i].cpu().numpy()[:n].astype(np.int64)).to(DEV)
            assert float(sel2.delta[i][idxs].abs().max()) == 0.0
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("kv_dtype,Hkv,Hq", [("bf16", 1, 8), ("fp16", 8, 8), ("bf16", 4, 16)])
def test_patch_other_row_widths(kv_dtype, Hkv, Hq):
    """A token row of Hkv * 256 bytes is copied in 512-byte pieces, one warp each: half a warp for one KV
    head, four pieces for eight.  Bit-exact against the oracle's row replacement; every other row untouched;
    an out-of-range entry in the selection (a caller's stale list) is skipped."""
    build_library()
    sh = synth.Shape(L=3, Hq=Hq, Hkv=Hkv, kv_dtype=kv_dtype)
    modes = [synth.MODE_INT8, synth.MODE_FRESH, synth.MODE_INT4, synth.MODE_INT8, synth.MODE_FP16]
    wl = synth.Workload("patch", 41, sh, [synth._request(5 * sh.C, sh.C, modes, [512, 0, 128, 2048, 0]), synth._request(2 * sh.C, sh.C, modes[:2], [0, 0])],
                        synth.SelectPlan(ratio=0.3, seam_before=4, seam_after=4))
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        n0 = int(sel.n_sel[0])
        good = sel.sel[0].cpu().numpy()[:n0].copy()
        sel.sel[0][1] = reqs[0].plan.T + 5  # stale entries: beyond the prompt, negative
        sel.sel[0][2] = -3
        before = [helpers.bits_of(r.kv_buf) for r in reqs]
        B.kvb_patch(ctx, tbl, sel)
        B.kvb_last_status(ctx)
        for i, r in enumerate(reqs):
            n = int(sel.n_sel[i])
            idxs = sel.sel[i].cpu().numpy()[:n]
            if i == 0:
                idxs = np.delete(good, [1, 2])
            want = oracle.patch(before[i], helpers.bits_of(r.fresh), idxs)
            assert np.array_equal(helpers.bits_of(r.kv_buf), want)
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("kv_dtype,Hkv,Hq", [("bf16", 2, 16), ("fp16", 4, 8)])
def test_chunk_importance_matches_oracle(kv_dtype, Hkv, Hq):
    build_library()
    sh = synth.Shape(L=5, Hq=Hq, Hkv=Hkv, kv_dtype=kv_dtype)
    modes = [synth.MODE_INT8, synth.MODE_FRESH, synth.MODE_FP16, synth.MODE_INT4, synth.MODE_INT8]
    wl = synth.Workload("imp", 31, sh, [synth._request(5 * sh.C, sh.C, modes, [512, 0, 128, 2048, 0]), synth._request(2 * sh.C, sh.C, modes[:2], [0, 0])], synth.SelectPlan())
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        outs = [torch.full((len(r.chunks),), -1.0, dtype=torch.float32, device=DEV) for r in reqs]
        B.kvb_chunk_importance(ctx, tbl, outs)
        B.kvb_last_status(ctx)
        for r, o in zip(reqs, outs):
            want = oracle.importance(helpers.bits_of(r.kv_buf), sh.C, helpers.dt_code(sh))
            got = o.cpu().numpy().astype(np.float64)
            assert np.abs(got - want).max() <= 1e-5 * np.abs(want).max()
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("case", ["cfg0", "cfg1_L3", "mixed_bf16_H2", "mixed_fp16_H4", "mixed_bf16_H1"])
def test_importance_as_a_by_product_of_the_stitch(case):
    """kvb_request.importance: the stitching calls deliver Eq. 7 from the key rows they hold in
    registers.  Against the oracle's fp64 value on the buffer the same call wrote (1e-6 relative),
    identical from the one-pass call, the plain stitch and a repeated call (bit for bit: the norm sums
    are added in a fixed order), and the stitched buffer and the selection are not disturbed."""
    build_library()
    from test_gpu_parity import _mixed_workload

    if case == "cfg0":
        wl = synth.workload(0)
    elif case == "cfg1_L3":
        w1 = synth.workload(1)
        wl = synth.Workload(w1.name, w1.seed, synth.Shape(L=3), w1.requests, w1.select)
    else:
        kv_dtype, H = case.split("_")[1], int(case.split("_H")[1])
        wl = _mixed_workload(H, 8, kv_dtype)
    sh, sp = wl.shape, wl.select
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        Ts = [r.plan.T for r in reqs]
        ks = [B.kvb_select_count(T, sp.ratio) for T in Ts]
        # reference run without the importance output
        tbl0 = B.RequestTable(reqs)
        sel0 = B.SelectionTable(Ts, ks, [r.sel_capacity for r in reqs], DEV)
        B.kvb_assemble_select(ctx, tbl0, sp.ratio, -1, sp.seam_before, sp.seam_after, sp.which, sel0)
        B.kvb_last_status(ctx)
        kv0 = [r.kv_buf.view(torch.int16).clone() for r in reqs]
        got = {}
        for call in ("one_pass", "one_pass_again", "stitch_only", "keys_not_compared"):
            for r in reqs:
                r.importance = torch.full((len(r.chunks),), -1.0, dtype=torch.float32, device=DEV)
                r.kv_buf.zero_()
            tbl = B.RequestTable(reqs)
            sel = B.SelectionTable(Ts, ks, [r.sel_capacity for r in reqs], DEV)
            if call == "stitch_only":
                B.kvb_assemble(ctx, tbl)
            else:  # which = 2: the deviation looks at values only, the key norms are still wanted
                B.kvb_assemble_select(ctx, tbl, sp.ratio, -1, sp.seam_before, sp.seam_after, 2 if call == "keys_not_compared" else sp.which, sel)
            B.kvb_last_status(ctx)
            got[call] = [r.importance.clone() for r in reqs]
            for r, k0 in zip(reqs, kv0):
                assert torch.equal(r.kv_buf.view(torch.int16), k0)
            if call == "one_pass":
                for i in range(len(reqs)):
                    assert torch.equal(sel.delta[i], sel0.delta[i]) and torch.equal(sel.sel[i], sel0.sel[i]) and torch.equal(sel.rank[i], sel0.rank[i])
        for i, r in enumerate(reqs):
            want = oracle.importance(helpers.bits_of(r.kv_buf), sh.C, helpers.dt_code(sh))
            g = got["one_pass"][i].cpu().numpy().astype(np.float64)
            assert np.abs(g - want).max() <= 1e-6 * np.abs(want).max(), np.abs(g / want - 1).max()
            for other in ("one_pass_again", "stitch_only", "keys_not_compared"):
                assert torch.equal(got["one_pass"][i], got[other][i]), other
        # the stand-alone call on the stitched buffer agrees as well
        outs = [torch.zeros(len(r.chunks), dtype=torch.float32, device=DEV) for r in reqs]
        B.kvb_chunk_importance(ctx, B.RequestTable(reqs), outs)
        B.kvb_last_status(ctx)
        for i in range(len(reqs)):
            assert float((outs[i] - got["one_pass"][i]).abs().max()) <= 2e-6 * float(outs[i].abs().max())
    finally:
        B.kvb_destroy(ctx)
