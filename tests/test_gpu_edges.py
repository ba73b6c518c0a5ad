"""Edge cases of the CUDA path: empty batches, the smallest and the largest requests the selection
kernel takes, an empty selection, overlapping and clamped seam windows."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import oracle_glue as helpers
from test_gpu_parity import check_assembled, check_attention, check_selection, oracle_stitch, prepare, run_assemble, run_attention, run_select

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def test_empty_batch_is_a_no_op():
    sh = synth.Shape(L=2)
    ctx = B.create_for_shape(sh, 0)
    try:
        empty = B.RequestTable([])
        sel = B.SelectionTable([], [], [], DEV)
        assert B.kvb_assemble(ctx, empty) == B.KVB_OK
        assert B.kvb_deviation_topk(ctx, empty, 0.15, -1, 16, 0, 3, sel) == B.KVB_OK
        assert B.kvb_selective_attn(ctx, empty, sel, [], [], 0.1) == B.KVB_OK
        assert B.kvb_patch(ctx, empty, sel) == B.KVB_OK
        assert B.kvb_launch_count(ctx) == 0 and B.kvb_last_status(ctx) == B.KVB_OK
    finally:
        B.kvb_destroy(ctx)


def test_single_fresh_chunk_request():
    """T = 128, nothing cached: the buffer is a copy of the fresh tensor, every deviation is 0, the
    selection is the first floor(0.15 * 128) = 19 positions, there is no seam."""
    sh = synth.Shape(L=2)
    wl = synth.Workload("one", 3, sh, [synth._request(128, sh.C, [synth.MODE_FRESH], [0])], synth.SelectPlan())
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        assert torch.equal(r.kv_buf.view(torch.int16), r.fresh.view(torch.int16))
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)
        assert ks == [19] and int(sel.n_sel[0]) == 19
        assert np.all(sel.delta[0].cpu().numpy() == 0.0)
        assert sel.rank[0].cpu().numpy().tolist() == list(range(19)) == sel.sel[0].cpu().numpy()[:19].tolist()
        outs = run_attention(ctx, sh, reqs, tbl, sel)
        check_attention(sh, r, np.arange(19, dtype=np.int32), outs[0], None, None)
    finally:
        B.kvb_destroy(ctx)


def test_selection_at_its_size_limits():
    """T = 32768 with k = 8192 is the largest request the selection kernel takes; one more chunk or
    one more selected position is refused before anything is launched."""
    sh = synth.Shape(L=1)
    n_chunks = 256
    rng = np.random.default_rng(8)
    modes = [synth.MODE_INT8 if rng.random() < 0.8 else synth.MODE_FRESH for _ in range(n_chunks)]
    origs = (rng.permutation(1024)[:n_chunks] * sh.C).tolist()
    sp = synth.SelectPlan(k_override=8192, seam_before=16, seam_after=0)
    wl = synth.Workload("big", 8, sh, [synth._request(n_chunks * sh.C, sh.C, modes, origs)], sp)
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0, max_requests=1, max_chunks_total=n_chunks + 1, max_tokens_total=(n_chunks + 1) * sh.C)
    try:
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, sp, use_oracle_buffer=False)
        check_selection(sh, reqs, sel, ks, sp)
        before = B.kvb_launch_count(ctx)
        sel2 = B.SelectionTable([32768], [8193], [32768], DEV)
        assert B.kvb_deviation_topk(ctx, tbl, 0.0, 8193, 0, 0, 3, sel2, check=False) == B.KVB_ERR_UNSUPPORTED
        assert B.kvb_launch_count(ctx) == before
    finally:
        B.kvb_destroy(ctx)
    # one chunk more than the kernel takes
    wl2 = synth.Workload("too_big", 9, sh, [synth._request((n_chunks + 1) * sh.C, sh.C, [synth.MODE_FRESH] * (n_chunks + 1), [0] * (n_chunks + 1))], sp)
    plan = wl2.requests[0]

    class R:
        pass

    r = R()
    r.plan, r.chunks = plan, [synth.Chunk(c) for c in plan.chunks]
    r.kv_buf = torch.zeros((1, 2, plan.T, sh.Hkv, sh.d), dtype=torch.bfloat16, device=DEV)
    r.fresh = torch.zeros_like(r.kv_buf)
    ctx = B.create_for_shape(sh, 0, max_requests=1, max_chunks_total=n_chunks + 1, max_tokens_total=plan.T)
    try:
        sel3 = B.SelectionTable([plan.T], [10], [plan.T], DEV)
        assert B.kvb_deviation_topk(ctx, B.RequestTable([r]), 0.0, 10, 0, 0, 3, sel3, check=False) == B.KVB_ERR_UNSUPPORTED
        assert "limits" in B.kvb_last_error(ctx)
    finally:
        B.kvb_destroy(ctx)


def test_attention_sink_tokens_join_the_selection():
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        k = B.kvb_select_count(r.plan.T, 0.15)
        sel = B.SelectionTable([r.plan.T], [k], [r.plan.T], DEV)
        B.kvb_deviation_topk(ctx, tbl, 0.15, -1, 16, 0, 3, sel, sink_tokens=4)
        B.kvb_last_status(ctx)
        rank = sel.rank[0].cpu().numpy()[:k]
        want = oracle.seam_select(rank, [c.plan.new_pos for c in r.chunks], [c.plan.mode for c in r.chunks], r.plan.T, 16, 0, sinks=4)
        n = int(sel.n_sel[0])
        assert np.array_equal(sel.sel[0].cpu().numpy()[:n], want) and {0, 1, 2, 3} <= set(want.tolist())
        assert B.kvb_deviation_topk(ctx, tbl, 0.15, -1, 16, 0, 3, sel, check=False, sink_tokens=-1) == B.KVB_ERR_INVALID_ARG
    finally:
        B.kvb_destroy(ctx)


def test_descriptor_upload_paths_agree():
    """Small calls send their tables as a kernel argument (and fill the rotation table in the same
    launch); the context's "descriptor_copy" option forces the pinned-buffer copy and the separate table
    kernel, "dependent_launch" = 0 launches the chain without programmatic dependent launch.  Same bits."""
    wl = synth.workload(0)
    sh = wl.shape
    got = {}
    for mode in ("kernel", "copy", "no_pdl"):
        reqs = prepare(wl)
        (r,) = reqs
        ctx = B.create_for_shape(sh, 0)
        try:
            if mode == "copy":
                B.kvb_set_debug_option(ctx, "descriptor_copy", 1)
            if mode == "no_pdl":
                B.kvb_set_debug_option(ctx, "dependent_launch", 0)
            assert B.kvb_set_debug_option(ctx, "no_such_option", 1, check=False) == B.KVB_ERR_INVALID_ARG
            assert B.kvb_set_debug_option(ctx, "descriptor_copy", 2, check=False) == B.KVB_ERR_INVALID_ARG
            before = B.kvb_launch_count(ctx)
            tbl = B.RequestTable(reqs)
            k = B.kvb_select_count(r.plan.T, 0.15)
            sel = B.SelectionTable([r.plan.T], [k], [r.sel_capacity], DEV)
            B.kvb_assemble_select(ctx, tbl, 0.15, -1, 16, 0, 3, sel)
            out = torch.zeros_like(r.q)
            B.kvb_selective_attn(ctx, tbl, sel, [r.q], [out], 0.1)
            B.kvb_last_status(ctx)
            # kernel path: store+table, stitch, selection; store, attention.  copy path: table, stitch, selection; attention
            assert B.kvb_launch_count(ctx) - before == (4 if mode == "copy" else 5)
            got[mode] = (r.kv_buf.view(torch.int16).clone(), sel.delta[0].clone(), sel.sel[0].clone(), out.view(torch.int16).clone())
        finally:
            B.kvb_destroy(ctx)
    for other in ("copy", "no_pdl"):
        for a, b in zip(got["kernel"], got[other]):
            assert torch.equal(a, b)


def test_selection_overflow_is_reported_once_and_cut_cleanly():
    """sel_capacity = k passes the host check, but the seam windows add positions: the kernel keeps
    the first sel_capacity entries of the ascending union, sets the status word, and the next
    report is clean again (no trap, the context stays usable)."""
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        k = B.kvb_select_count(r.plan.T, 0.15)
        sel = B.SelectionTable([r.plan.T], [k], [k], DEV)  # room for the top-k only
        guard = torch.full((k + 64,), -7, dtype=torch.int32, device=DEV)
        sel.sel[0] = guard[:k]
        sel.array[0].sel = guard.data_ptr()
        B.kvb_deviation_topk(ctx, tbl, 0.15, -1, 16, 0, 3, sel)
        assert B.kvb_last_status(ctx, check=False) == B.KVB_ERR_DEVICE_STATUS
        assert "0x4" in B.kvb_last_error(ctx) and "sel_capacity" in B.kvb_last_error(ctx)
        assert int(sel.n_sel[0]) == k
        rank = sel.rank[0].cpu().numpy()[:k]
        want = oracle.seam_select(rank, [c.plan.new_pos for c in r.chunks], [c.plan.mode for c in r.chunks], r.plan.T, 16, 0)
        assert len(want) > k
        assert np.array_equal(guard[:k].cpu().numpy(), want[:k])
        assert torch.all(guard[k:] == -7), "nothing may be written past sel_capacity"
        assert B.kvb_last_status(ctx, check=False) == B.KVB_OK  # reported once
        sel2, ks, caps = run_select(ctx, wl, reqs, tbl, use_oracle_buffer=False)  # a correct call afterwards
        check_selection(sh, reqs, sel2, ks, wl.select)
    finally:
        B.kvb_destroy(ctx)


def test_attention_persistent_and_one_tile_ctas_agree():
    """The attention kernel runs as persistent CTAs drawing tiles from a counter; the context's
    "attention_one_tile_per_cta" option runs one tile per CTA instead.  Both must give the same bits, on
    a batch whose tiles are short, ragged and partly empty (sel_capacity = T > n_sel)."""
    sh = synth.Shape(L=3, Hq=16, Hkv=2)
    plans = [synth._request(T, sh.C, [synth.MODE_INT8] * (T // sh.C), [((5 * i) % (T // sh.C)) * sh.C for i in range(T // sh.C)]) for T in (128, 640, 1152, 256)]
    wl = synth.Workload("modes", 31, sh, plans, synth.SelectPlan(ratio=0.2, seam_before=8, seam_after=8))
    reqs = prepare(wl)
    outs = {}
    for mode in ("persistent", "onetile"):
        ctx = B.create_for_shape(sh, 0, max_requests=len(reqs))
        try:
            B.kvb_set_debug_option(ctx, "attention_one_tile_per_cta", int(mode == "onetile"))
            tbl = run_assemble(ctx, reqs)
            Ts = [r.plan.T for r in reqs]
            ks = [B.kvb_select_count(T, 0.2) for T in Ts]
            sel = B.SelectionTable(Ts, ks, Ts, DEV)  # capacity T: many tiles past n_sel have no rows
            for r in reqs:
                r.sel_capacity = r.plan.T
            B.kvb_deviation_topk(ctx, tbl, 0.2, -1, 8, 8, 3, sel)
            qs = [torch.randn(sh.L, T, sh.Hq, sh.d, device=DEV, generator=torch.Generator(DEV).manual_seed(T)).to(r.fresh.dtype) for T, r in zip(Ts, reqs)]
            out = [torch.zeros_like(q) for q in qs]
            for _ in range(2):  # a second call reuses the context's tile counter slot
                B.kvb_selective_attn(ctx, tbl, sel, qs, out, 1.0 / math.sqrt(sh.d))
            B.kvb_last_status(ctx)
            outs[mode] = out
            if mode == "persistent":
                for i, r in enumerate(reqs):
                    n = int(sel.n_sel[i])
                    r.q = qs[i]
                    check_attention(sh, r, sel.sel[i].cpu().numpy()[:n], out[i], None, None)
                    assert not out[i][:, n:].any()
        finally:
            B.kvb_destroy(ctx)
    for a, b in zip(outs["persistent"], outs["onetile"]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_empty_selection_and_wide_overlapping_seam_windows():
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        # nothing selected: k = 0 and no windows -> n_sel = 0, attention and patch touch nothing
        sp0 = synth.SelectPlan(k_override=0, seam_before=0, seam_after=0)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, sp0, use_oracle_buffer=False)
        assert int(sel.n_sel[0]) == 0
        sel_for_attn = B.SelectionTable([r.plan.T], [0], [r.sel_capacity], DEV)  # capacity of the Q tensor, n_sel = 0
        out = torch.full_like(r.q, 3.0)
        B.kvb_selective_attn(ctx, tbl, sel_for_attn, [r.q], [out], 0.1)
        before = r.kv_buf.clone()
        B.kvb_patch(ctx, tbl, sel_for_attn)
        B.kvb_last_status(ctx)
        assert torch.all(out == 3.0) and torch.equal(before.view(torch.int16), r.kv_buf.view(torch.int16))
        # windows wider than a chunk: they overlap each other and are clamped at 0 and T
        sp = synth.SelectPlan(ratio=0.05, seam_before=200, seam_after=150)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, sp, use_oracle_buffer=False)
        check_selection(sh, reqs, sel, ks, sp)
        assert int(sel.n_sel[0]) == r.plan.T  # three seams x 350 positions cover all 512
    finally:
        B.kvb_destroy(ctx)


def test_attention_rejects_an_output_that_is_not_32_byte_aligned():
    """Output rows leave the attention kernel as 32-byte stores; the call checks the base pointer on the
    host and launches nothing when it is off (q only needs 16 bytes)."""
    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, wl.select, use_oracle_buffer=False)
        flat = torch.zeros(r.q.numel() + 8, dtype=r.q.dtype, device=DEV)
        off = flat[8:].view(r.q.shape)  # 16 bytes past a 32-byte boundary
        assert off.data_ptr() % 32 == 16
        before = B.lib().kvb_launch_count(ctx)
        st = B.kvb_selective_attn(ctx, tbl, sel, [r.q], [off], 0.1, check=False)
        assert st == B.KVB_ERR_BAD_TABLE and B.lib().kvb_launch_count(ctx) == before
        assert not flat.any()
        q_off = torch.zeros(r.q.numel() + 8, dtype=r.q.dtype, device=DEV)[8:].view(r.q.shape)  # a 16-byte aligned q is fine
        q_off.copy_(r.q)
        out = torch.zeros_like(r.q)
        B.kvb_selective_attn(ctx, tbl, sel, [q_off], [out], 1.0 / math.sqrt(sh.d))
        B.kvb_last_status(ctx)
        ref = torch.zeros_like(r.q)
        B.kvb_selective_attn(ctx, tbl, sel, [r.q], [ref], 1.0 / math.sqrt(sh.d))
        B.kvb_last_status(ctx)
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    finally:
        B.kvb_destroy(ctx)


def test_a_barrier_wait_that_cannot_complete_gives_up_and_is_reported():
    """The attention kernel's waits are bounded by wall time.  The library's self-test runs that wait on
    a barrier nothing arrives at: the kernel must return after the limit, raise status bit 0x1, and
    leave the context fit for the next call."""
    import time

    wl = synth.workload(0)
    sh = wl.shape
    reqs = prepare(wl)
    (r,) = reqs
    ctx = B.create_for_shape(sh, 0)
    try:
        assert B.kvb_selftest_wait_timeout(ctx, 0, check=False) == B.KVB_ERR_INVALID_ARG
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        B.kvb_selftest_wait_timeout(ctx, 30)
        with pytest.raises(B.KvbError) as ei:
            B.kvb_last_status(ctx)  # synchronises
        dt = time.perf_counter() - t0
        assert ei.value.status == B.KVB_ERR_DEVICE_STATUS and "0x1" in str(ei.value) and "wait" in str(ei.value)
        assert 0.03 <= dt < 1.0, dt
        assert B.kvb_last_status(ctx) == B.KVB_OK  # reported once
        # the context still works
        tbl = run_assemble(ctx, reqs)
        sel, ks, caps = run_select(ctx, wl, reqs, tbl, wl.select, use_oracle_buffer=False)
        out = torch.zeros_like(r.q)
        B.kvb_selective_attn(ctx, tbl, sel, [r.q], [out], 1.0 / math.sqrt(sh.d))
        assert B.kvb_last_status(ctx) == B.KVB_OK
        n = int(sel.n_sel[0])
        check_attention(sh, r, sel.sel[0].cpu().numpy()[:n], out, None, None)
    finally:
        B.kvb_destroy(ctx)


def test_selection_cluster_path_plateaus_windows_and_extremes():
    """Prompts beyond 2048 positions are selected by a thread-block cluster, every CTA owning a slice:
    thresholds that fall on plateaus of equal deviations spanning slice boundaries (taken lowest index
    first), k = 0 / 1 / T - 1 / T, windows that straddle slices, a slice count that does not divide the
    prompt, and a batch that mixes short and long prompts.  rank / sel / n_sel must equal the oracle's
    selection of the GPU's own delta, bit for bit."""
    sh = synth.Shape(L=2, Hq=16, Hkv=2)
    Ts = (4224, 16384, 640, 8192 + 128)  # 3, 8, (8), 5 slices of unequal fill; the short prompt shares the launch
    rng = np.random.default_rng(11)

    class R:
        pass

    reqs = []
    for T in Ts:
        r = R()
        modes = [synth.MODE_FP16 if (i % 5) else synth.MODE_FRESH for i in range(T // sh.C)]
        r.plan = synth._request(T, sh.C, modes, [i * sh.C for i in range(T // sh.C)])
        r.chunks = [synth.Chunk(cp) for cp in r.plan.chunks]
        g = torch.Generator(device=DEV).manual_seed(T)
        r.kv_buf = torch.randn((sh.L, 2, T, sh.Hkv, sh.d), generator=g, device=DEV).to(torch.bfloat16)
        noise = 0.02 * torch.randn(r.kv_buf.shape, generator=g, device=DEV)
        r.fresh = (r.kv_buf.float() + noise).to(torch.bfloat16)
        # plateaus: long runs of exact copies (delta 0), and groups of positions that repeat one (stored, fresh) pair
        r.fresh[:, :, T // 3 : T // 3 + T // 4] = r.kv_buf[:, :, T // 3 : T // 3 + T // 4]
        src = int(rng.integers(0, T // 3))
        for dst in rng.choice(np.arange(T // 3 + T // 4, T), size=T // 16, replace=False):
            r.kv_buf[:, :, dst] = r.kv_buf[:, :, src]
            r.fresh[:, :, dst] = r.fresh[:, :, src]
        reqs.append(r)
    ctx = B.create_for_shape(sh, 0, max_requests=len(reqs), max_chunks_total=sum(T // sh.C for T in Ts), max_tokens_total=sum(Ts))
    try:
        # the whole batch (k up to the kernel's limit of 8192), then the 4224-token prompt alone with k = T - 1 and k = T
        cases = [(reqs, Ts, c) for c in ((0.15, -1, 16, 0, 0), (0.45, -1, 40, 40, 100), (0.0, 0, 0, 0, 0), (0.0, 1, 0, 0, 0), (0.5, -1, 0, 0, 4000))]
        cases += [(reqs[:1], Ts[:1], c) for c in ((1.0, -1, 0, 0, 0), (0.9999, -1, 3, 3, 0))]
        for rs, ts, (ratio, k_over, before, after, sinks) in cases:
            tbl = B.RequestTable(rs)
            ks = [k_over if k_over >= 0 else B.kvb_select_count(T, ratio) for T in ts]
            sel = B.SelectionTable(ts, ks, ts, DEV)
            B.kvb_deviation_topk(ctx, tbl, ratio, k_over, before, after, 3, sel, sink_tokens=sinks)
            B.kvb_last_status(ctx)
            for i, (r, T, k) in enumerate(zip(rs, ts, ks)):
                dg = sel.delta[i].cpu().numpy()
                want_rank = oracle.topk(dg, k)
                assert np.array_equal(sel.rank[i].cpu().numpy()[:k], want_rank), (T, k)
                want = oracle.seam_select(want_rank, [c.plan.new_pos for c in r.chunks], [c.plan.mode for c in r.chunks], T, before, after, sinks)
                n = int(sel.n_sel[i])
                assert n == len(want) and np.array_equal(sel.sel[i].cpu().numpy()[:n], want), (T, k)
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("option", ["attention_cta_pairs", "attention_two_tiles"])
def test_attention_cta_pair_form_matches_oracle(option):
    """(attention_two_tiles: two neighbouring tiles per CTA sharing K/V, one CTA per SM -- same check.)
    The paired form of the attention kernel (two neighbouring tiles on two SMs per MMA, the context's
    "attention_cta_pairs" option; the single-CTA kernel is the default because it measures faster) computes
    the same attention: against the oracle at 2e-2 on a batch whose tiles are short, ragged, odd in number
    per plane and partly empty, with rows past n_sel left untouched.  Its bits may differ from the
    single-CTA kernel's: keys go by sub-blocks of 128 instead of 64, so the lazy reference maximum moves at
    other places and the float32 sums are taken in another order."""
    sh = synth.Shape(L=3, Hq=16, Hkv=2)
    plans = [synth._request(T, sh.C, [synth.MODE_INT8] * (T // sh.C), [((5 * i) % (T // sh.C)) * sh.C for i in range(T // sh.C)]) for T in (128, 640, 1152, 256, 2176)]
    wl = synth.Workload("pairs", 37, sh, plans, synth.SelectPlan(ratio=0.2, seam_before=8, seam_after=8))
    reqs = prepare(wl)
    ctx = B.create_for_shape(sh, 0, max_requests=len(reqs))
    try:
        B.kvb_set_debug_option(ctx, option, 1)
        tbl = run_assemble(ctx, reqs)
        Ts = [r.plan.T for r in reqs]
        ks = [B.kvb_select_count(T, 0.2) for T in Ts]
        sel = B.SelectionTable(Ts, ks, Ts, DEV)  # capacity T: many tiles past n_sel have no rows
        for r in reqs:
            r.sel_capacity = r.plan.T
        B.kvb_deviation_topk(ctx, tbl, 0.2, -1, 8, 8, 3, sel)
        # queries by the workloads' recipe, N(0, 1 / d), for every row of the capacity
        qs = [(torch.randn(sh.L, T, sh.Hq, sh.d, device=DEV, generator=torch.Generator(DEV).manual_seed(T)) / math.sqrt(sh.d)).to(r.fresh.dtype)
              for T, r in zip(Ts, reqs)]
        out = [torch.zeros_like(q) for q in qs]
        for _ in range(2):
            B.kvb_selective_attn(ctx, tbl, sel, qs, out, 1.0 / math.sqrt(sh.d))
        B.kvb_last_status(ctx)
        for i, r in enumerate(reqs):
            n = int(sel.n_sel[i])
            r.q = qs[i]
            check_attention(sh, r, sel.sel[i].cpu().numpy()[:n], out[i], None, None)
            assert not out[i][:, n:].any()
    finally:
        B.kvb_destroy(ctx)
