"""Position-free cache population (kvb_quantize_keys_at): keys rotated back by their original position
before Eq. 6, so that a cached chunk is listed with orig_pos = 0 and re-used with one rotation."""
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


def _keys(sh, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn((sh.L, sh.C, sh.Hkv, sh.d), generator=g) * torch.exp(torch.rand((sh.L, 1, sh.Hkv, sh.d), generator=g) * 3.0 - 1.5)
    return x.to(sh.torch_dtype)


def _quantize_at(ctx, sh, x_dev, pos, bits):
    L, Cn, H, d = x_dev.shape
    codes = torch.empty((L, Cn, H, d * bits // 8), dtype=torch.uint8, device=DEV)
    meta = torch.empty((L, 1 if bits == 8 else Cn // sh.int4_group, H, d, 2), dtype=torch.float32, device=DEV)
    B.kvb_quantize_keys_at(ctx, x_dev, pos, bits, codes, meta)
    B.kvb_last_status(ctx)
    return codes, meta


@pytest.mark.parametrize("kv_dtype", ["bf16", "fp16"])
def test_codes_and_metadata_bit_exact(kv_dtype):
    sh = synth.Shape(L=2, kv_dtype=kv_dtype)
    dtc = helpers.dt_code(sh)
    ctx = B.create_for_shape(sh, 0)
    try:
        x = _keys(sh, 5)
        xb = helpers.bits_of(x)
        for pos in (0, 128, 4096 * 3 + 128, (1 << 24) - 128):
            for bits, group in ((8, sh.C), (4, sh.int4_group)):
                codes, meta = _quantize_at(ctx, sh, x.to(DEV), pos, bits)
                for l in range(sh.L):
                    u = oracle.unrotate_keys(xb[l], dtc, sh.theta, pos)
                    oc, om = oracle.quantize_k(u, bits, group)
                    assert np.array_equal(codes[l].cpu().numpy(), oc), "codes, pos %d bits %d" % (pos, bits)
                    assert np.array_equal(meta[l].cpu().numpy(), om), "metadata, pos %d bits %d" % (pos, bits)
        # position 0 is the plain quantiser
        qk, _ = B.quantize_fns(ctx, sh)
        c0, m0 = _quantize_at(ctx, sh, x.to(DEV), 0, 8)
        c1, m1 = qk(x.to(DEV), 8, sh.C)
        assert torch.equal(c0, c1) and torch.equal(m0, m1)
        assert B.kvb_quantize_keys_at(ctx, x.to(DEV), -1, 8, c0, m0, check=False) == B.KVB_ERR_INVALID_ARG
        assert B.kvb_quantize_keys_at(ctx, x.to(DEV), 0, 5, c0, m0, check=False) == B.KVB_ERR_INVALID_ARG
    finally:
        B.kvb_destroy(ctx)


def test_reuse_at_another_position_is_one_rotation():
    """Keys encoded at position 896, stored position-free, re-used at position 256: the stitched rows are
    the original keys rotated by 256 - 896, up to the quantisation step (Eq. 6: half a step per channel,
    a rotation mixes two channels)."""
    sh = synth.Shape(L=2)
    dtc = helpers.dt_code(sh)
    orig, new, T = 896, 256, 512
    ctx = B.create_for_shape(sh, 0)
    try:
        x = _keys(sh, 9)
        vals = _keys(sh, 10)
        codes, meta = _quantize_at(ctx, sh, x.to(DEV), orig, 8)
        qk, qv = B.quantize_fns(ctx, sh)
        vcodes, vmeta = qv(vals.to(DEV), 8, sh.d)
        plan = synth._request(T, sh.C, [synth.MODE_FRESH, synth.MODE_FRESH, synth.MODE_INT8, synth.MODE_FRESH], [0, 0, 0, 0])
        assert plan.chunks[2].new_pos == new and plan.chunks[2].orig_pos == 0

        class R:
            pass

        r = R()
        r.plan = plan
        r.chunks = [synth.Chunk(c) for c in plan.chunks]
        r.chunks[2] = synth.Chunk(plan.chunks[2], codes, vcodes, meta, vmeta)
        r.fresh = torch.zeros((sh.L, 2, T, sh.Hkv, sh.d), dtype=sh.torch_dtype, device=DEV)
        r.kv_buf = torch.zeros_like(r.fresh)
        B.kvb_assemble(ctx, B.RequestTable([r]))
        B.kvb_last_status(ctx)
        got = oracle.bits_to_f64(helpers.bits_of(r.kv_buf[:, 0, new : new + sh.C]), dtc)  # [L,C,H,d]
        x64 = oracle.bits_to_f64(helpers.bits_of(x), dtc)
        half = sh.d // 2
        for l in range(sh.L):
            want = oracle.rope_rotate(x64[l], sh.theta, float(new - orig))
            scale = meta[l, 0].cpu().numpy()[..., 0].astype(np.float64)  # [H,d] step of each stored channel
            step_pair = np.sqrt(scale[:, :half] ** 2 + scale[:, half:] ** 2)
            bound = 0.5 * np.concatenate([step_pair, step_pair], -1)[None] * 1.01 + 2.0**-8 * np.abs(want) + 1e-6
            assert np.all(np.abs(got[l] - want) <= bound)
    finally:
        B.kvb_destroy(ctx)


@pytest.mark.parametrize("kv_dtype,Hkv", [("bf16", 2), ("fp16", 1), ("bf16", 4), ("fp16", 8)])
def test_batched_quantiser_codes_bit_exact(kv_dtype, Hkv):
    """kvb_quantize_chunks: one launch for a batch of chunks with mixed widths, keys only / values only
    / both, keys rotated back or not, compact or float32 metadata.  Codes and metadata equal the
    oracle's bit for bit (Eq. 6 forward: float32 subtract, divide, round-half-even on both sides),
    including groups with tiny and with zero range, where the fast reciprocal must not decide."""
    sh = synth.Shape(L=3, Hq=8, Hkv=Hkv, kv_dtype=kv_dtype)
    dtc = helpers.dt_code(sh)
    ctx = B.create_for_shape(sh, 0, max_chunks_total=16)
    try:
        specs = [  # (bits, keys?, values?, unrotate_from, meta_fp16)
            (8, True, True, -1, False), (4, True, True, -1, False), (8, True, False, 4096 + 128, False), (4, True, True, 77, False),
            (8, False, True, -1, False), (4, True, True, -1, True), (8, True, True, (1 << 24) - 128, True), (8, True, True, -1, False),
            (8, True, True, -1, False), (4, True, True, -1, True),  # 8, 9: every other quotient an exact tie (below)
        ]
        jobs, xs = [], []
        for i, (bits, has_k, has_v, pos, m16) in enumerate(specs):
            k = _keys(sh, 100 + i)
            v = _keys(sh, 200 + i)
            if i == 7:  # degenerate groups: a constant channel, a constant row, a range of a few float32 ulps, a huge range
                k[:, :, :, 3] = 1.25
                v[:, 5] = -0.5
                k[:, :, :, 9] = 1.0
                k[:, 64:, :, 9] = 1.0 + 2.0 ** -7
                v[:, 7, :, ::2] = 3.0e4 if kv_dtype == "fp16" else 1.0e30
            if i >= 8:  # integers in [0, 2 * levels] with both ends in every group: scale 2, the odd ones tie, far
                # more of them than the kernel's list of places to redo with the IEEE division holds
                top = 2 * ((1 << bits) - 1)
                g = torch.Generator().manual_seed(300 + i)
                k = torch.randint(0, top // 2 + 1, (sh.L, sh.C, Hkv, sh.d), generator=g).float()
                v = torch.randint(0, top // 2 + 1, (sh.L, sh.C, Hkv, sh.d), generator=g).float()
                k[:, 0::32], k[:, 1::32] = 0.0, float(top)              # keys: groups run over tokens
                v[:, :, :, 0::32], v[:, :, :, 1::32] = 0.0, float(top)  # values: over channels
                k, v = k.to(sh.torch_dtype), v.to(sh.torch_dtype)
            mt = torch.float16 if m16 else torch.float32
            j = dict(bits=bits, unrotate_from=pos, meta_fp16=m16)
            if has_k:
                j.update(k=k.to(DEV), k_codes=torch.zeros((sh.L, sh.C, Hkv, sh.d * bits // 8), dtype=torch.uint8, device=DEV),
                         k_meta=torch.zeros((sh.L, 1 if bits == 8 else sh.C // sh.int4_group, Hkv, sh.d, 2), dtype=mt, device=DEV))
            if has_v:
                j.update(v=v.to(DEV), v_codes=torch.zeros((sh.L, sh.C, Hkv, sh.d * bits // 8), dtype=torch.uint8, device=DEV),
                         v_meta=torch.zeros((sh.L, sh.C, Hkv, 1 if bits == 8 else sh.d // sh.int4_group, 2), dtype=mt, device=DEV))
            jobs.append(j)
            xs.append((k, v))
        B.kvb_quantize_chunks(ctx, jobs)
        B.kvb_last_status(ctx)
        for (bits, has_k, has_v, pos, m16), j, (k, v) in zip(specs, jobs, xs):
            gk, gv = (sh.C, sh.d) if bits == 8 else (sh.int4_group, sh.int4_group)
            for l in range(sh.L):
                if has_k:
                    u = oracle.unrotate_keys(helpers.bits_of(k)[l], dtc, sh.theta, pos) if pos >= 0 else helpers.f64_of(k)[l]
                    oc, om = oracle.quantize_k(u, bits, gk, meta16=m16)
                    assert np.array_equal(j["k_codes"][l].cpu().numpy(), oc), ("key codes", bits, pos, m16)
                    assert np.array_equal(j["k_meta"][l].float().cpu().numpy(), om.astype(np.float32)), ("key metadata", bits, pos, m16)
                if has_v:
                    oc, om = oracle.quantize_v(helpers.f64_of(v)[l], bits, gv, meta16=m16)
                    assert np.array_equal(j["v_codes"][l].cpu().numpy(), oc), ("value codes", bits, m16)
                    assert np.array_equal(j["v_meta"][l].float().cpu().numpy(), om.astype(np.float32)), ("value metadata", bits, m16)
        # the one-chunk entry points are the same kernel with one job
        c1 = torch.zeros_like(jobs[0]["k_codes"])
        m1 = torch.zeros_like(jobs[0]["k_meta"])
        B.kvb_quantize_chunk(ctx, jobs[0]["k"], False, 8, c1, m1)
        B.kvb_last_status(ctx)
        assert torch.equal(c1, jobs[0]["k_codes"]) and torch.equal(m1, jobs[0]["k_meta"])
        # rejected: no side wanted, a missing output, too many jobs for the context
        assert B.kvb_quantize_chunks(ctx, [dict(bits=8)], check=False) == B.KVB_ERR_INVALID_ARG
        assert B.kvb_quantize_chunks(ctx, [dict(bits=8, k=jobs[0]["k"], k_codes=c1)], check=False) == B.KVB_ERR_INVALID_ARG
        assert B.kvb_quantize_chunks(ctx, [jobs[0]] * 4096, check=False) == B.KVB_ERR_WORKSPACE
        assert B.kvb_quantize_chunks(ctx, []) == B.KVB_OK
    finally:
        B.kvb_destroy(ctx)
