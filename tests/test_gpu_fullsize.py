"""Full-size parity, in the launch configuration bench.py times (its Replica objects: inputs drawn on
the GPU, chunks quantised by the CUDA quantiser, one call per stage for the whole batch).  The oracle
cannot redo 300k tokens x 36 layers, so it recomputes sampled outputs one by one:
  stitching   sampled (request, chunk, layer) blocks from the chunk's own codes and metadata
  deviation   sampled positions over all layers, from the stored buffer and the fresh tensor
  selection   the whole rank / sel lists (cheap) against the oracle run on the GPU's delta
  attention   sampled selected rows on sampled layers, from the stored buffer
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import bench
import oracle_glue as helpers
from test_gpu_parity import ulp16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_path(wl):
    sh, sp = wl.shape, wl.select
    ctx = B.create_for_shape(sh, 0, max_requests=len(wl.requests), max_chunks_total=sum(len(r.chunks) for r in wl.requests),
                             max_tokens_total=sum(r.T for r in wl.requests))
    rep = bench.Replica(B, ctx, wl, DEV, 0)
    bench.step(B, ctx, rep, sp, 1.0 / math.sqrt(sh.d))
    B.kvb_last_status(ctx)
    torch.cuda.synchronize()
    return ctx, rep


def _check_chunk_layer(sh, r, ck, l):
    """One chunk, one layer: oracle dequantise + rotate from the chunk's codes vs the rows the GPU wrote."""
    dtc = helpers.dt_code(sh)
    sl = slice(ck.plan.new_pos, ck.plan.new_pos + sh.C)
    got = helpers.bits_of(r.kv_buf[l, :, sl])  # [2,C,H,d]
    if ck.plan.mode == synth.MODE_FRESH:
        assert np.array_equal(got, helpers.bits_of(r.fresh[l, :, sl]))
        return
    if ck.plan.mode == synth.MODE_FP16:
        k = oracle.bits_to_f64(helpers.bits_of(ck.k_codes[l]), dtc)
        v = oracle.bits_to_f64(helpers.bits_of(ck.v_codes[l]), dtc)
    else:
        bits = 8 if ck.plan.mode == synth.MODE_INT8 else 4
        gk, gv = (sh.C, sh.d) if bits == 8 else (sh.int4_group, sh.int4_group)
        k = oracle.dequant_k(ck.k_codes[l].cpu().numpy(), ck.k_meta[l].cpu().numpy(), sh.d, bits, gk)
        v = oracle.dequant_v(ck.v_codes[l].cpu().numpy(), ck.v_meta[l].cpu().numpy(), sh.d, bits, gv)
    k = oracle.rope_rotate(k, sh.theta, float(ck.plan.new_pos - ck.plan.orig_pos))
    y = np.stack([k, v])
    half = sh.d // 2
    ref = np.abs(y).copy()
    pair = np.sqrt(y[0, ..., :half] ** 2 + y[0, ..., half:] ** 2)
    ref[0, ..., :half] = pair
    ref[0, ..., half:] = pair
    M = np.abs(y).max(axis=(1, 2, 3), keepdims=True)
    bound = 1e-3 * ref + 0.5 * ulp16(y, sh.kv_dtype) + 2e-6 * M
    err = np.abs(oracle.bits_to_f64(got, dtc) - y)
    assert float((err / bound).max()) <= 1.0
    assert np.mean(got == oracle.round_to_bits(y, dtc)) > 0.999


def _check_request(sh, sp, rep, i, rng, n_chunk_samples, n_tok_samples, attn_layers, n_attn_rows):
    r = rep.reqs[i]
    dtc = helpers.dt_code(sh)
    T = r.plan.T
    # stitching
    for _ in range(n_chunk_samples):
        _check_chunk_layer(sh, r, r.chunks[int(rng.integers(len(r.chunks)))], int(rng.integers(sh.L)))
    # deviation on sampled positions (all layers)
    ts = np.unique(np.concatenate([rng.integers(0, T, n_tok_samples), [0, T - 1]]))
    tsd = torch.from_numpy(ts).to(DEV)
    kv_s = helpers.bits_of(r.kv_buf[:, :, tsd])
    fr_s = helpers.bits_of(r.fresh[:, :, tsd])
    d64, _ = oracle.deviation(kv_s, fr_s, dtc, sp.which)
    dg = rep.sel.delta[i].cpu().numpy()
    assert np.abs(dg[ts].astype(np.float64) - d64).max() <= 1e-5
    # selection, whole lists
    k = rep.ks[i]
    rank_g = rep.sel.rank[i].cpu().numpy()[:k]
    assert np.array_equal(rank_g, oracle.topk(dg, k))
    n = int(rep.sel.n_sel[i])
    want = oracle.seam_select(rank_g, [c.plan.new_pos for c in r.chunks], [c.plan.mode for c in r.chunks], T, sp.seam_before, sp.seam_after)
    sel_idx = rep.sel.sel[i].cpu().numpy()[:n]
    assert np.array_equal(sel_idx, want)
    # attention on sampled rows
    if attn_layers:
        rows = np.unique(np.concatenate([rng.integers(0, n, n_attn_rows), [0, n - 1]])).astype(np.int32)
        kv_host = helpers.bits_of(r.kv_buf)
        _, exact = oracle.attention(helpers.bits_of(r.q), kv_host, sel_idx, sh.Hq, dtc, 1.0 / math.sqrt(sh.d), layers=attn_layers, rows=rows, want_exact=True)
        og = oracle.bits_to_f64(helpers.bits_of(rep.out[i]), dtc)
        err = np.abs(og[np.ix_(attn_layers, rows)] - exact[np.ix_(attn_layers, rows)]).max()
        assert err <= 2e-2, "attention error %.4g" % err


def test_cfg3_selective_attention_full_size():
    build_library()
    wl = synth.workload(3)  # 8192-token int4 prompt, k = 1229, no seam windows
    ctx, rep = _run_path(wl)
    try:
        assert int(rep.sel.n_sel[0]) == 1229
        rng = np.random.default_rng(3)
        _check_request(wl.shape, wl.select, rep, 0, rng, 6, 256, [0, 13, 35], 40)
        # every selected row on one layer
        r = rep.reqs[0]
        dtc = helpers.dt_code(wl.shape)
        sel_idx = rep.sel.sel[0].cpu().numpy()[:1229]
        _, exact = oracle.attention(helpers.bits_of(r.q), helpers.bits_of(r.kv_buf), sel_idx, wl.shape.Hq, dtc, 1.0 / math.sqrt(128), layers=[21], want_exact=True)
        og = oracle.bits_to_f64(helpers.bits_of(rep.out[0][21]), dtc)
        assert np.abs(og[:1229] - exact[21, :1229]).max() <= 2e-2
    finally:
        B.kvb_destroy(ctx)


def test_cfg4_ragged_batch_full_size():
    build_library()
    wl = synth.workload(4)  # 32 requests, ~300k tokens, fp16 / int8 / int4 / fresh chunks mixed
    ctx, rep = _run_path(wl)
    try:
        rng = np.random.default_rng(4)
        order = np.argsort([r.plan.T for r in rep.reqs])
        attn_on = {int(order[0]), int(order[-1]), int(order[len(order) // 2])}  # shortest, longest, median
        for i in range(len(rep.reqs)):
            _check_request(wl.shape, wl.select, rep, i, rng, 3, 96, [int(rng.integers(wl.shape.L))] if i in attn_on else None, 10)
        # every mode was exercised
        assert {c.plan.mode for r in rep.reqs for c in r.chunks} == {0, 1, 2, 3}
    finally:
        B.kvb_destroy(ctx)
