"""Parity of the CUDA path (called through the C ABI) against the CPU oracle, stage by stage,
on the same seeded inputs.  Tolerances:
  stitched rows   |g - y| <= 1e-3 * ref + ulp16(y)/2 + 2e-6 * M, y the oracle's un-rounded value,
                  ref = norm of the rotation pair (keys) or |y| (values), M = max |y| of the chunk-layer
                  (1e-3 relative is the stated bar; ulp16/2 is the one 16-bit rounding both sides make,
                  which alone reaches 3.9e-3 relative in bf16; 2e-6 M covers float32 arithmetic on
                  intermediates of size M, where q*scale and min cancel)
  deviation       |delta_gpu - delta_oracle| <= 1e-5 absolute, both fed the same stored buffer
  selection       rank / sel / n_sel bit-exact against the oracle run on the GPU's own delta
  attention       |o_gpu - o_oracle| <= 2e-2 absolute (bf16 / fp16 output)
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import oracle_glue as helpers

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def _ctx(sh, **kw):
    return B.create_for_shape(sh, 0, **kw)


def to_device(reqs):
    for r in reqs:
        r.fresh = r.fresh.to(DEV)
        r.kv_oracle = r.kv_buf  # the oracle's stitched buffer stays on the host
        r.kv_buf = torch.zeros_like(r.fresh)
        r.q = r.q.to(DEV)
        for ck in r.chunks:
            for name in ("k_codes", "v_codes", "k_meta", "v_meta"):
                t = getattr(ck, name)
                if t is not None:
                    setattr(ck, name, t.to(DEV).contiguous())
    return reqs


ulp16, check_assembled = helpers.ulp16, helpers.check_assembled


def oracle_stitch(sh, req):
    return helpers.oracle_assemble_np(sh, req.plan, req.chunks_host, helpers.bits_of(req.fresh_host), want_exact=True)


def prepare(wl, request_ids=None):
    """Inputs by the oracle-side recipe, a device copy for the CUDA path."""
    reqs = helpers.materialize_with_oracle(wl, "cpu", request_ids)
    for r in reqs:
        r.fresh_host = r.fresh
        r.chunks_host = [synth.Chunk(c.plan, c.k_codes, c.v_codes, c.k_meta, c.v_meta) for c in r.chunks]
    return to_device(reqs)


def run_assemble(ctx, reqs):
    tbl = B.RequestTable(reqs)
    B.kvb_assemble(ctx, tbl)
    B.kvb_last_status(ctx)
    return tbl


# ------------------------------------------------------------------------------- stitching
@pytest.mark.parametrize("idx", [0, 1])
def test_assemble_matches_oracle(idx):
    wl = synth.workload(idx)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh)
    try:
        run_assemble(ctx, reqs)
        for r in reqs:
            kv_o, exact = oracle_stitch(sh, r)
            check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
    finally:
        B.kvb_destroy(ctx)


def _mixed_workload(Hkv, Hq, kv_dtype, L=3, seed=11):
    """All four modes, zero / negative / large position shifts, unaligned original positions."""
    sh = synth.Shape(L=L, Hq=Hq, Hkv=Hkv, kv_dtype=kv_dtype)
    M = synth
    spec = [  # (mode, orig_pos)
        (M.MODE_INT8, 0), (M.MODE_INT4, 128), (M.MODE_FP16, 256), (M.MODE_FRESH, 0),
        (M.MODE_INT8, 4096 * 4 - 1), (M.MODE_INT4, 7), (M.MODE_FP16, 1 << 20), (M.MODE_INT8, 896),
        (M.MODE_FP16, 1024 + 77), (M.MODE_INT4, (1 << 24) - 128),
    ]
    chunks = []
    for i, (m, o) in enumerate(spec):
        new = i * sh.C
        o = new if m == M.MODE_FRESH else o
        chunks.append(M.ChunkPlan(new, o, m, M._match(o, new, m)))
    return M.Workload("mixed", seed, sh, [M.RequestPlan(len(spec) * sh.C, chunks)], M.SelectPlan())


@pytest.mark.parametrize("Hkv,Hq,kv_dtype", [(2, 16, "bf16"), (2, 16, "fp16"), (1, 8, "bf16"), (4, 8, "bf16"), (8, 8, "fp16")])
def test_assemble_all_modes_and_shifts(Hkv, Hq, kv_dtype):
    wl = _mixed_workload(Hkv, Hq, kv_dtype)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh)
    try:
        run_assemble(ctx, reqs)
        (r,) = reqs
        kv_o, exact = oracle_stitch(sh, r)
        g = helpers.bits_of(r.kv_buf)
        check_assembled(sh, r, g, exact, kv_o)
        # chunks 0, 1, 2 keep their position: rotation is the identity, unquantised rows are bit copies
        assert np.array_equal(g[:, :, 256:384], np.stack([helpers.bits_of(r.chunks_host[2].k_codes), helpers.bits_of(r.chunks_host[2].v_codes)], 1))
        # values are never rotated: dequantisation alone, whatever the shift.  The GPU rounds a float32
        # result (error <= 3 * 2^-24 relative) to 16 bits, the oracle rounds the exact value once: they
        # differ only when the value sits that close to a rounding boundary (spacing 2^-11 relative in
        # fp16), i.e. for at most 2 * 3 * 2^-24 / 2^-11 = 7e-4 of the values
        assert np.mean(g[:, 1] == kv_o[:, 1]) > 0.9993
    finally:
        B.kvb_destroy(ctx)


def test_assemble_long_int4_prompt():
    wl = synth.workload(2)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh)
    try:
        run_assemble(ctx, reqs)
        (r,) = reqs
        kv_o, exact = oracle_stitch(sh, r)
        check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
    finally:
        B.kvb_destroy(ctx)


def test_assemble_leaves_other_memory_alone_and_is_deterministic():
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    # canaries around the buffer: the kernel must write rows [0, T) of each plane and nothing else
    n = r.kv_buf.numel()
    big = torch.full((n + 2048,), 7.0, dtype=r.kv_buf.dtype, device=DEV)
    r.kv_buf = big[1024 : 1024 + n].view(r.fresh.shape)
    ctx = _ctx(sh)
    try:
        run_assemble(ctx, reqs)
        first = r.kv_buf.clone()
        assert torch.all(big[:1024] == 7.0) and torch.all(big[1024 + n :] == 7.0)
        run_assemble(ctx, reqs)
        assert torch.equal(first.view(torch.int16), r.kv_buf.view(torch.int16))
    finally:
        B.kvb_destroy(ctx)


# ------------------------------------------------------------------------------- deviation + selection
def run_select(ctx, wl, reqs, tbl, sp=None, use_oracle_buffer=True):
    sp = sp or wl.select
    if use_oracle_buffer:  # stage isolation: both sides see the same stored buffer
        for r in reqs:
            r.kv_buf.copy_(r.kv_oracle.to(DEV))
    Ts = [r.plan.T for r in reqs]
    ks = [sp.k_override if sp.k_override >= 0 else B.kvb_select_count(T, sp.ratio) for T in Ts]
    caps = [max(1, min(r.plan.T, k + (len(r.chunks) - 1) * (sp.seam_before + sp.seam_after))) for r, k in zip(reqs, ks)]
    sel = B.SelectionTable(Ts, ks, caps, DEV)
    B.kvb_deviation_topk(ctx, tbl, sp.ratio, sp.k_override, sp.seam_before, sp.seam_after, sp.which, sel)
    B.kvb_last_status(ctx)
    return sel, ks, caps


def check_selection(sh, reqs, sel, ks, sp):
    """delta within 1e-5 of the oracle; rank / sel bit-exact against the oracle applied to the GPU's delta;
    end to end, rank may differ from the oracle's own only inside the +-2e-5 band around its k-th value."""
    n_sel = sel.n_sel.cpu().numpy()
    for i, r in enumerate(reqs):
        kv = helpers.bits_of(r.kv_buf)
        d64, d32 = oracle.deviation(kv, helpers.bits_of(r.fresh), helpers.dt_code(sh), sp.which)
        dg = sel.delta[i].cpu().numpy()
        assert np.abs(dg.astype(np.float64) - d64).max() <= 1e-5
        k = ks[i]
        rank_g = sel.rank[i].cpu().numpy()[:k]
        assert np.array_equal(rank_g, oracle.topk(dg, k))
        modes = [c.plan.mode for c in r.chunks]
        pos = [c.plan.new_pos for c in r.chunks]
        want_sel = oracle.seam_select(rank_g, pos, modes, r.plan.T, sp.seam_before, sp.seam_after)
        assert n_sel[i] == len(want_sel)
        assert np.array_equal(sel.sel[i].cpu().numpy()[: n_sel[i]], want_sel)
        rank_o = oracle.topk(d32, k)
        diff = set(rank_g.tolist()) ^ set(rank_o.tolist())
        if diff and k > 0:
            kth = float(d32[rank_o[-1]])
            assert all(abs(float(d64[t]) - kth) <= 2e-5 for t in diff), "selection differs outside the tolerance band"


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_deviation_topk_matches_oracle(idx):
    wl = synth.workload(idx)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh)
    try:
        tbl = B.RequestTable(reqs)
        for sp in (wl.select, synth.SelectPlan(ratio=0.25, seam_before=0, seam_after=16, which=1), synth.SelectPlan(ratio=0.05, seam_before=16, seam_after=16, which=2)):
            sel, ks, caps = run_select(ctx, wl, reqs, tbl, sp)
            check_selection(sh, reqs, sel, ks, sp)
    finally:
        B.kvb_destroy(ctx)


def test_selection_ties_plateaus_and_extremes():
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    T = r.plan.T
    ctx = _ctx(sh)
    try:
        tbl = B.RequestTable(reqs)
        # duplicate whole tokens (stored and fresh rows alike) -> exactly equal deviations inside the top-k
        kvo = r.kv_oracle.clone()
        for src, dst in ((130, 5), (130, 301), (131, 17), (140, 300)):
            kvo[:, :, dst] = kvo[:, :, src]
            r.fresh[:, :, dst] = r.fresh[:, :, src]
        r.kv_oracle = kvo
        for k in (0, 1, 76, 200, T - 140, T - 1, T):  # thresholds inside the big zero plateau of the fresh chunk too
            sp = synth.SelectPlan(k_override=k, seam_before=16, seam_after=0)
            sel, ks, caps = run_select(ctx, wl, reqs, tbl, sp)
            check_selection(sh, reqs, sel, ks, sp)
            dg = sel.delta[0].cpu().numpy()
            assert dg[5] == dg[130] == dg[301] and dg[17] == dg[131]
        # all rows identical to fresh -> all deviations 0 -> the first k indices
        r.kv_oracle = r.fresh.cpu().clone()
        sp = synth.SelectPlan(k_override=33, seam_before=0, seam_after=0)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, sp)
        assert np.all(sel.delta[0].cpu().numpy() == 0.0)
        assert sel.rank[0].cpu().numpy().tolist() == list(range(33))
        assert sel.sel[0].cpu().numpy()[: int(sel.n_sel[0])].tolist() == list(range(33))
    finally:
        B.kvb_destroy(ctx)


def test_deviation_degenerate_rows():
    """Zero rows: equal zero rows count as cos 1; a zero row against a non-zero row as cos 0."""
    sh = synth.Shape(L=2, Hq=16, Hkv=2)
    wl = synth.Workload("deg", 5, sh, [synth._request(256, sh.C, [synth.MODE_FP16, synth.MODE_FP16], [0, 128])], synth.SelectPlan(seam_before=0))
    reqs = prepare(wl)
    (r,) = reqs
    kvo = r.kv_oracle.clone()
    kvo[:, :, 3] = 0
    r.fresh[:, :, 3] = 0  # both zero
    kvo[:, :, 9] = 0  # stored zero, fresh not
    r.fresh[:, :, 20] = 0  # fresh zero, stored not
    kvo[:, :, 30] = -r.fresh[:, :, 30].cpu()  # opposite
    r.kv_oracle = kvo
    ctx = _ctx(sh)
    try:
        tbl = B.RequestTable(reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl)
        check_selection(sh, reqs, sel, ks, wl.select)
        dg = sel.delta[0].cpu().numpy()
        assert dg[3] == 0.0 and dg[9] == 1.0 and dg[20] == 1.0 and abs(dg[30] - 2.0) < 1e-6
    finally:
        B.kvb_destroy(ctx)


# ------------------------------------------------------------------------------- attention
def run_attention(ctx, sh, reqs, tbl, sel):
    outs = [torch.zeros_like(r.q) for r in reqs]
    B.kvb_selective_attn(ctx, tbl, sel, [r.q for r in reqs], outs, 1.0 / math.sqrt(sh.d))
    B.kvb_last_status(ctx)
    return outs


def check_attention(sh, r, sel_idx, out, layers, rows):
    dtc = helpers.dt_code(sh)
    o_bits, exact = oracle.attention(helpers.bits_of(r.q), helpers.bits_of(r.kv_buf), sel_idx, sh.Hq, dtc, 1.0 / math.sqrt(sh.d), layers=layers, rows=rows, want_exact=True)
    g = oracle.bits_to_f64(helpers.bits_of(out), dtc)
    L = list(range(sh.L)) if layers is None else list(layers)
    R = list(range(len(sel_idx))) if rows is None else list(rows)
    err = np.abs(g[np.ix_(L, R)] - exact[np.ix_(L, R)]).max()
    assert err <= 2e-2, "attention error %.4g" % err
    return err


@pytest.mark.parametrize("idx", [0, 1])
def test_selective_attention_matches_oracle(idx):
    wl = synth.workload(idx)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh)
    try:
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        outs = run_attention(ctx, sh, reqs, tbl, sel)
        (r,) = reqs
        n = int(sel.n_sel[0])
        sel_idx = sel.sel[0].cpu().numpy()[:n]
        assert n > ks[0]  # top-k plus seam windows
        layers = None if idx == 0 else [0, 17, 35]
        check_attention(sh, r, sel_idx, outs[0], layers, None)
        assert not outs[0][:, n:].any(), "rows past n_sel must stay untouched"
    finally:
        B.kvb_destroy(ctx)


def test_selective_attention_edge_rows():
    """Position 0 (one visible key), the last position, a ragged tail tile and no GQA sharing."""
    for Hkv, Hq in ((2, 16), (2, 2), (4, 8)):
        sh = synth.Shape(L=2, Hq=Hq, Hkv=Hkv)
        wl = synth.Workload("edge", 21, sh, [synth._request(512, sh.C, [synth.MODE_INT8, synth.MODE_FRESH, synth.MODE_FP16, synth.MODE_INT4], [384, 0, 1024, 0])], synth.SelectPlan(k_override=37, seam_before=0, seam_after=0))
        reqs = prepare(wl)
        (r,) = reqs
        ctx = _ctx(sh)
        try:
            tbl = run_assemble(ctx, reqs)
            sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
            # overwrite the selection with a hand-made one: first, last, and a scattered middle
            mine = np.array(sorted({0, 1, 2, 63, 64, 65, 127, 128, 200, 255, 256, 300, 383, 384, 450, 510, 511}), np.int32)
            sel.sel[0][: len(mine)] = torch.from_numpy(mine).to(DEV)
            sel.n_sel[0] = len(mine)
            outs = run_attention(ctx, sh, reqs, tbl, sel)
            check_attention(sh, r, mine, outs[0], None, None)
            v0 = r.kv_buf[:, 1, 0]  # [L,H,d]: position 0 attends only itself -> output = V_0 of its KV head
            got = outs[0][:, 0].view(sh.L, Hkv, Hq // Hkv, sh.d)
            assert torch.equal(got, v0[:, :, None, :].expand_as(got))
        finally:
            B.kvb_destroy(ctx)


# ------------------------------------------------------------------------------- whole path, ragged batch
def test_ragged_batch_pipeline():
    wl = synth.workload(4, n_requests=5)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh)
    try:
        tbl = run_assemble(ctx, reqs)
        for r in reqs:
            kv_o, exact = oracle_stitch(sh, r)
            check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        check_selection(sh, reqs, sel, ks, wl.select)
        outs = run_attention(ctx, sh, reqs, tbl, sel)
        rng = np.random.default_rng(0)
        for i, r in enumerate(reqs):
            n = int(sel.n_sel[i])
            sel_idx = sel.sel[i].cpu().numpy()[:n]
            rows = np.sort(rng.choice(n, size=min(n, 24), replace=False)).astype(np.int32)
            rows[-1] = n - 1
            check_attention(sh, r, sel_idx, outs[i], [0, int(rng.integers(1, sh.L))], rows)
        # the whole batch goes in a fixed number of launches, whatever the number of requests: table +
        # stitch, (store) + deviation + selection, (store) + attention
        assert 5 <= B.kvb_launch_count(ctx) <= 7
    finally:
        B.kvb_destroy(ctx)


# ------------------------------------------------------------------------------- quantiser (cache-population side)
@pytest.mark.parametrize("kv_dtype", ["bf16", "fp16"])
def test_quantizer_codes_bit_exact(kv_dtype):
    sh = synth.Shape(L=3, kv_dtype=kv_dtype)
    ctx = _ctx(sh)
    try:
        g = torch.Generator().manual_seed(3)
        x = (torch.randn((sh.L, sh.C, sh.Hkv, sh.d), generator=g) * torch.exp(torch.rand((sh.L, 1, sh.Hkv, sh.d), generator=g) * 4.6 - 2.3)).to(sh.torch_dtype)
        x[0, :, 0, 5] = 1.25  # a constant channel: scale 1, codes 0
        x[1, 7, 1, :] = -3.0  # a constant token row
        qk, qv = B.quantize_fns(ctx, sh)
        for bits, group in ((8, sh.C), (4, sh.int4_group)):
            ck, mk = qk(x.to(DEV), bits, group)
            ok, om = helpers.oracle_quantize_k(x, bits, group)
            assert torch.equal(ck.cpu(), ok) and torch.equal(mk.cpu(), om)
        for bits, group in ((8, sh.d), (4, sh.int4_group)):
            cv, mv = qv(x.to(DEV), bits, group)
            ov, om = helpers.oracle_quantize_v(x, bits, group)
            assert torch.equal(cv.cpu(), ov) and torch.equal(mv.cpu(), om)
    finally:
        B.kvb_destroy(ctx)


# ------------------------------------------------------------------------------- error paths on a live context
def test_rejected_calls_launch_nothing():
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    ctx = _ctx(sh, max_requests=1, max_chunks_total=4, max_tokens_total=512)
    try:
        before = B.kvb_launch_count(ctx)
        reqs[0].chunks[1].plan.new_pos = 0
        assert B.kvb_assemble(ctx, B.RequestTable(reqs), check=False) == B.KVB_ERR_BAD_TABLE
        assert "gap or overlap" in B.kvb_last_error(ctx)
        reqs[0].chunks[1].plan.new_pos = 128
        tbl = B.RequestTable(reqs)
        sel = B.SelectionTable([512], [76], [10], DEV)  # capacity below k
        assert B.kvb_deviation_topk(ctx, tbl, 0.15, -1, 16, 0, 3, sel, check=False) == B.KVB_ERR_INVALID_ARG
        assert B.kvb_deviation_topk(ctx, tbl, 0.15, -1, 16, 0, 0, sel, check=False) == B.KVB_ERR_INVALID_ARG
        assert B.kvb_launch_count(ctx) == before
        assert B.kvb_assemble(ctx, B.RequestTable(reqs + reqs), check=False) == B.KVB_ERR_WORKSPACE
        assert B.kvb_assemble(ctx, tbl) == B.KVB_OK and B.kvb_last_status(ctx) == B.KVB_OK
    finally:
        B.kvb_destroy(ctx)
    with pytest.raises(B.KvbError):
        B.create_for_shape(synth.Shape(d=64))  # head_dim the kernels are not built for


# ------------------------------------------------------------------------------- shape corners
@pytest.mark.parametrize("Hkv,Hq,kv_dtype", [(1, 16, "bf16"), (16, 16, "fp16"), (16, 64, "bf16"), (8, 128, "bf16"), (4, 16, "fp16")])
def test_whole_path_at_the_corners_of_the_supported_shapes(Hkv, Hq, kv_dtype):
    """Stitch, deviation + selection and attention against the oracle at the ends of the supported head
    counts (1 and 16 KV heads; 1, 4 and 16 query heads per KV head), every mode in one request."""
    sh = synth.Shape(L=2, Hq=Hq, Hkv=Hkv, kv_dtype=kv_dtype)
    modes = [synth.MODE_INT8, synth.MODE_INT4, synth.MODE_FRESH, synth.MODE_FP16, synth.MODE_INT8]
    wl = synth.Workload("corner", 100 + 17 * Hkv + Hq, sh, [synth._request(640, sh.C, modes, [384, 7, 0, 1 << 18, 512])],
                        synth.SelectPlan(ratio=0.15, seam_before=8, seam_after=8))
    reqs = prepare(wl)
    (r,) = reqs
    ctx = _ctx(sh)
    try:
        tbl = run_assemble(ctx, reqs)
        kv_o, exact = oracle_stitch(sh, r)
        check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, wl.select, use_oracle_buffer=False)
        check_selection(sh, reqs, sel, ks, wl.select)
        n = int(sel.n_sel[0])
        (out,) = run_attention(ctx, sh, reqs, tbl, sel)
        check_attention(sh, r, sel.sel[0].cpu().numpy()[:n], out, None, None)
        assert not out[:, n:].any()
    finally:
        B.kvb_destroy(ctx)
