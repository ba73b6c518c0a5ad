"""Compact metadata: (scale, min) pairs stored as binary16 (kvb_chunk.meta_fp16 = 1), written by
kvb_quantize_chunk_ex and read by the stitching kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import oracle_glue as helpers
from test_gpu_parity import check_assembled, check_selection

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def _tensor(sh, seed, spread=3.0):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn((sh.L, sh.C, sh.Hkv, sh.d), generator=g) * torch.exp(torch.rand((sh.L, 1, sh.Hkv, sh.d), generator=g) * spread - spread / 2)
    return x.to(sh.torch_dtype)


def _gpu_quantize(ctx, sh, x, is_value, bits, meta16, unrotate_from=-1):
    L, Cn, H, d = x.shape
    codes = torch.empty((L, Cn, H, d * bits // 8), dtype=torch.uint8, device=DEV)
    if is_value:
        shape = (L, Cn, H, 1 if bits == 8 else d // sh.int4_group, 2)
    else:
        shape = (L, 1 if bits == 8 else Cn // sh.int4_group, H, d, 2)
    meta = torch.empty(shape, dtype=torch.float16 if meta16 else torch.float32, device=DEV)
    B.kvb_quantize_chunk_ex(ctx, x.to(DEV), is_value, bits, unrotate_from, meta16, codes, meta)
    B.kvb_last_status(ctx)
    return codes, meta


def _oracle_quantize(sh, x, is_value, bits, meta16):
    xs = helpers.f64_of(x)
    group = (sh.d if bits == 8 else sh.int4_group) if is_value else (sh.C if bits == 8 else sh.int4_group)
    fn = oracle.quantize_v if is_value else oracle.quantize_k
    codes, metas = zip(*[fn(xs[l], bits, group, meta16=meta16) for l in range(xs.shape[0])])
    return np.stack(codes), np.stack(metas)


@pytest.mark.parametrize("kv_dtype", ["bf16", "fp16"])
def test_compact_quantiser_bit_exact(kv_dtype):
    sh = synth.Shape(L=2, kv_dtype=kv_dtype)
    ctx = B.create_for_shape(sh, 0)
    try:
        x = _tensor(sh, 21)
        x[0, :, 0, 7] = 0.3333  # a constant channel / a constant row still round outward
        x[1, 5, 1, :] = -2.5
        for is_value in (False, True):
            for bits in (8, 4):
                codes, meta = _gpu_quantize(ctx, sh, x, is_value, bits, True)
                oc, om = _oracle_quantize(sh, x, is_value, bits, True)
                assert np.array_equal(codes.cpu().numpy(), oc), (is_value, bits)
                assert np.array_equal(meta.float().cpu().numpy(), om), (is_value, bits)
        # with the rotation back to position 0 as well
        codes, meta = _gpu_quantize(ctx, sh, x, False, 8, True, unrotate_from=4096 + 128)
        dtc = helpers.dt_code(sh)
        for l in range(sh.L):
            u = oracle.unrotate_keys(helpers.bits_of(x)[l], dtc, sh.theta, 4096 + 128)
            oc, om = oracle.quantize_k(u, 8, sh.C, meta16=True)
            assert np.array_equal(codes[l].cpu().numpy(), oc) and np.array_equal(meta[l].float().cpu().numpy(), om)
        c8, m8 = _gpu_quantize(ctx, sh, x, True, 8, False)
        assert B.kvb_quantize_chunk_ex(ctx, x.to(DEV), True, 8, 128, False, c8, m8, check=False) == B.KVB_ERR_INVALID_ARG  # values never rotate
        assert B.kvb_quantize_chunk_ex(ctx, x.to(DEV), False, 8, -1, 2, c8, m8, check=False) == B.KVB_ERR_INVALID_ARG
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("Hkv,Hq,kv_dtype", [(2, 16, "bf16"), (1, 8, "fp16"), (8, 8, "bf16")])
def test_stitch_and_one_pass_with_compact_metadata(Hkv, Hq, kv_dtype):
    """A request mixing compact and float32 metadata, int8 and int4, moved and unmoved chunks."""
    sh = synth.Shape(L=2, Hq=Hq, Hkv=Hkv, kv_dtype=kv_dtype)
    M = synth
    spec = [  # (mode, orig_pos, compact)
        (M.MODE_INT8, 0, True), (M.MODE_INT4, 128, True), (M.MODE_INT8, 4096 * 3, True), (M.MODE_FRESH, 0, False),
        (M.MODE_INT4, 7, True), (M.MODE_INT8, 896, False), (M.MODE_INT4, (1 << 20) + 5, False), (M.MODE_FP16, 256, False),
    ]
    T = len(spec) * sh.C
    plans = []
    for i, (m, o, _) in enumerate(spec):
        new = i * sh.C
        o = new if m == M.MODE_FRESH else o
        plans.append(M.ChunkPlan(new, o, m, M._match(o, new, m)))
    plan = M.RequestPlan(T, plans)
    g = torch.Generator().manual_seed(4)
    fresh = (torch.randn((sh.L, 2, T, sh.Hkv, sh.d), generator=g) * 1.5).to(sh.torch_dtype)
    chunks_host = []
    for i, (m, o, compact) in enumerate(spec):
        if m == M.MODE_FRESH:
            chunks_host.append(M.Chunk(plans[i]))
            continue
        # payload = the fresh rows plus a perturbation, so that deviations are small but not zero
        sl = slice(i * sh.C, (i + 1) * sh.C)
        xk = (fresh[:, 0, sl].float() + 0.05 * _tensor(sh, 100 + i).float()).to(sh.torch_dtype)
        xv = (fresh[:, 1, sl].float() + 0.05 * _tensor(sh, 200 + i).float()).to(sh.torch_dtype)
        if m == M.MODE_FP16:
            chunks_host.append(M.Chunk(plans[i], xk.clone(), xv.clone()))
            continue
        bits = 8 if m == M.MODE_INT8 else 4
        kc, km = _oracle_quantize(sh, xk, False, bits, compact)
        vc, vm = _oracle_quantize(sh, xv, True, bits, compact)
        mt = torch.float16 if compact else torch.float32
        chunks_host.append(M.Chunk(plans[i], torch.from_numpy(kc), torch.from_numpy(vc), torch.from_numpy(km).to(mt),
                                   torch.from_numpy(vm).to(mt), meta_fp16=int(compact)))

    class R:
        pass

    r = R()
    r.plan = plan
    r.chunks = [M.Chunk(c.plan, *(None if t is None else t.to(DEV).contiguous() for t in (c.k_codes, c.v_codes, c.k_meta, c.v_meta)), meta_fp16=c.meta_fp16)
                for c in chunks_host]
    r.fresh = fresh.to(DEV)
    r.kv_buf = torch.zeros_like(r.fresh)
    kv_o, exact = helpers.oracle_assemble_np(sh, plan, chunks_host, helpers.bits_of(fresh), want_exact=True)
    ctx = B.create_for_shape(sh, 0)
    try:
        tbl = B.RequestTable([r])
        B.kvb_assemble(ctx, tbl)
        B.kvb_last_status(ctx)
        check_assembled(sh, r, helpers.bits_of(r.kv_buf), exact, kv_o)
        two_call = r.kv_buf.view(torch.int16).clone()
        r.kv_buf.zero_()
        sp = synth.SelectPlan(ratio=0.1, seam_before=8, seam_after=0)
        k = B.kvb_select_count(T, sp.ratio)
        sel = B.SelectionTable([T], [k], [T], DEV)
        B.kvb_assemble_select(ctx, tbl, sp.ratio, -1, sp.seam_before, sp.seam_after, 3, sel)
        B.kvb_last_status(ctx)
        assert torch.equal(two_call, r.kv_buf.view(torch.int16))
        check_selection(sh, [r], sel, [k], sp)
        bad = M.Chunk(r.chunks[0].plan, r.chunks[0].k_codes, r.chunks[0].v_codes, r.chunks[0].k_meta, r.chunks[0].v_meta, meta_fp16=3)
        r.chunks[0] = bad
        assert B.kvb_assemble(ctx, B.RequestTable([r]), check=False) == B.KVB_ERR_INVALID_ARG
    finally:
        B.kvb_destroy(ctx)
