"""The one-pass entry point (stitch + deviation sums in one kernel, then the selection) against the
oracle and against the two-call path."""
import numpy as np
import pytest
import torch

from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import oracle_glue as helpers
from test_gpu_parity import _mixed_workload, check_assembled, check_selection, oracle_stitch, prepare, run_assemble, run_select

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

PLANS = (
    None,  # the workload's own
    synth.SelectPlan(ratio=0.25, seam_before=0, seam_after=16, which=1),
    synth.SelectPlan(ratio=0.05, seam_before=16, seam_after=16, which=2),
)


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def run_fused(ctx, wl, reqs, sp=None, sink_tokens=0):
    sp = sp or wl.select
    tbl = B.RequestTable(reqs)
    Ts = [r.plan.T for r in reqs]
    ks = [sp.k_override if sp.k_override >= 0 else B.kvb_select_count(T, sp.ratio) for T in Ts]
    caps = [max(1, min(r.plan.T, k + sink_tokens + (len(r.chunks) - 1) * (sp.seam_before + sp.seam_after))) for r, k in zip(reqs, ks)]
    sel = B.SelectionTable(Ts, ks, caps, DEV)
    for r in reqs:
        r.kv_buf.fill_(float("nan"))  # every row must be rewritten
    B.kvb_assemble_select(ctx, tbl, sp.ratio, sp.k_override, sp.seam_before, sp.seam_after, sp.which, sel, sink_tokens=sink_tokens)
    B.kvb_last_status(ctx)
    return tbl, sel, ks


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_fused_matches_oracle_and_two_call_path(idx):
    wl = synth.workload(idx)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        stitched = [oracle_stitch(sh, r) for r in reqs]
        for sp in PLANS:
            sp = sp or wl.select
            tbl, sel, ks = run_fused(ctx, wl, reqs, sp)
            fused_bits = [r.kv_buf.view(torch.int16).clone() for r in reqs]
            for r, (kv_o, exact) in zip(reqs, stitched):
                check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
            check_selection(sh, reqs, sel, ks, sp)
            # the two-call path on the same inputs: same buffer bit for bit, delta to float32 rounding
            run_assemble(ctx, reqs)
            sel2, ks2, _ = run_select(ctx, wl, reqs, tbl, sp, use_oracle_buffer=False)
            for i, r in enumerate(reqs):
                assert torch.equal(fused_bits[i], r.kv_buf.view(torch.int16))
                assert float((sel.delta[i] - sel2.delta[i]).abs().max()) <= 1e-6
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("Hkv,Hq,kv_dtype", [(2, 16, "bf16"), (2, 16, "fp16"), (1, 8, "bf16"), (4, 8, "bf16"), (8, 8, "fp16")])
def test_fused_all_modes_head_counts_and_dtypes(Hkv, Hq, kv_dtype):
    wl = _mixed_workload(Hkv, Hq, kv_dtype)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        kv_o, exact = oracle_stitch(sh, r)
        for sp in (synth.SelectPlan(ratio=0.15, seam_before=16, seam_after=0, which=3), PLANS[1], PLANS[2]):
            tbl, sel, ks = run_fused(ctx, wl, reqs, sp)
            check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
            check_selection(sh, reqs, sel, ks, sp)
            d = sel.delta[0].cpu().numpy()
            assert np.all(d[3 * sh.C : 4 * sh.C] == 0.0)  # the FRESH chunk deviates from nothing
    finally:
        B.kvb_destroy(ctx)


def test_fused_is_repeatable_and_mixes_with_the_two_call_path():
    """The accumulator is left clean: repeated and interleaved calls give identical bits."""
    wl = synth.workload(1)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl, sel_a, ks = run_fused(ctx, wl, reqs, sink_tokens=4)
        run_assemble(ctx, reqs)
        sel_mid, _, _ = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        tbl, sel_b, _ = run_fused(ctx, wl, reqs, sink_tokens=4)
        for i in range(len(reqs)):
            assert torch.equal(sel_a.delta[i].view(torch.int32), sel_b.delta[i].view(torch.int32))
            assert torch.equal(sel_a.rank[i], sel_b.rank[i]) and torch.equal(sel_a.sel[i], sel_b.sel[i])
            n = int(sel_a.n_sel[i])
            assert {0, 1, 2, 3} <= set(sel_a.sel[i].cpu().numpy()[:n].tolist())
    finally:
        B.kvb_destroy(ctx)


def test_fused_rejects_what_either_call_rejects():
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = B.RequestTable(reqs)
        sel = B.SelectionTable([r.plan.T], [10], [r.plan.T], DEV)
        before = B.kvb_launch_count(ctx)
        assert B.kvb_assemble_select(ctx, tbl, 0.15, -1, 16, 0, 0, sel, check=False) == B.KVB_ERR_INVALID_ARG  # which = 0
        small = B.SelectionTable([r.plan.T], [10], [5], DEV)
        assert B.kvb_assemble_select(ctx, tbl, 0.0, 10, 0, 0, 3, small, check=False) == B.KVB_ERR_INVALID_ARG  # k > sel_capacity
        ck = next(c for c in r.chunks if c.plan.mode != synth.MODE_FRESH)
        keep = ck.k_codes
        ck.k_codes = None  # the stitch needs the payload
        assert B.kvb_assemble_select(ctx, B.RequestTable(reqs), 0.0, 10, 0, 0, 3, sel, check=False) == B.KVB_ERR_INVALID_ARG
        ck.k_codes = keep
        assert B.kvb_launch_count(ctx) == before
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("seed", [1, 3, 8, 13])
def test_random_ragged_batches_through_the_one_pass_path_and_attention(seed):
    """Seeded random batches: head counts, layers, dtype, request lengths, chunk modes and original
    positions (aligned, unaligned, unmoved), selection ratio (0 and 1 included), seam windows, which of
    K / V is compared and attention sinks are all drawn; stitch, selection and attention are checked
    against the oracle."""
    import math

    from test_gpu_parity import check_attention

    M = synth
    rng = np.random.default_rng(1000 + seed)
    Hkv, rep, dt = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4, 8])), str(rng.choice(["bf16", "fp16"]))
    sh = M.Shape(L=int(rng.integers(1, 4)), Hq=Hkv * rep, Hkv=Hkv, kv_dtype=dt)
    plans = []
    for _ in range(int(rng.integers(1, 5))):
        nch = int(rng.integers(1, 11))
        modes = rng.choice([M.MODE_FRESH, M.MODE_FP16, M.MODE_INT8, M.MODE_INT4], size=nch, p=[0.25, 0.25, 0.3, 0.2])
        origs = [int(rng.integers(0, (1 << 24) - 128)) if rng.random() < 0.7 else int(rng.integers(0, 64)) * 128 for _ in range(nch)]
        origs = [i * sh.C if rng.random() < 0.2 else o for i, o in enumerate(origs)]
        plans.append(M._request(nch * sh.C, sh.C, list(modes), origs))
    sp = M.SelectPlan(ratio=float(rng.choice([0.0, 0.05, 0.15, 0.5, 1.0])), seam_before=int(rng.choice([0, 4, 16, 40])),
                      seam_after=int(rng.choice([0, 8, 16])), which=int(rng.choice([1, 2, 3])))
    sinks = int(rng.choice([0, 0, 4]))
    wl = M.Workload("rand", 1000 + seed, sh, plans, sp)
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0, max_requests=len(reqs))
    try:
        tbl, sel, ks = run_fused(ctx, wl, reqs, sp, sink_tokens=sinks)
        for r in reqs:
            kv_o, exact = oracle_stitch(sh, r)
            check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
        if sinks == 0:
            check_selection(sh, reqs, sel, ks, sp)
        qs = [(torch.randn(sh.L, sel.sel[i].numel(), sh.Hq, sh.d, device=DEV, generator=torch.Generator(DEV).manual_seed(seed * 10 + i)) / math.sqrt(sh.d)).to(r.fresh.dtype)
              for i, r in enumerate(reqs)]
        outs = [torch.zeros_like(q) for q in qs]
        B.kvb_selective_attn(ctx, tbl, sel, qs, outs, 1.0 / math.sqrt(sh.d))
        B.kvb_last_status(ctx)
        for i, r in enumerate(reqs):
            n = int(sel.n_sel[i])
            r.q = qs[i]
            if n:
                check_attention(sh, r, sel.sel[i].cpu().numpy()[:n], outs[i], None, None)
            assert not outs[i][:, n:].any()
    finally:
        B.kvb_destroy(ctx)
