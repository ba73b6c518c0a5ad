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


@pytest.mark.parametrize("idx,n_req", [(0, None), (4, 3)])
def test_patch_matches_oracle(idx, n_req):
    build_library()
    wl = synth.workload(idx, n_req) if n_req else synth.workload(idx)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        before = [helpers.bits_of(r.kv_buf) for r in reqs]
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
