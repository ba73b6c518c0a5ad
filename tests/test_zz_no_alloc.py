"""kvb_deviation_static: the deviation step for hosts that may not allocate GPU memory (a server
whose block pool already owns the whole device, a thread that cannot afford cudaMalloc's implicit
device synchronisation).  It works out of a static device array instead of a context's scratch, so
it must give the same deviations as kvb_deviation_topk, call after call, although every call
reuses the same array and finds the previous call's sums in it.

Collected last on purpose: a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest
import torch

from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

import oracle
import oracle_glue as glue

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(sh, T, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    kv = torch.randn((sh.L, 2, T, sh.Hkv, sh.d), generator=g, device=DEV).to(sh.torch_dtype)
    noise = torch.randn(kv.shape, generator=g, device=DEV) * 0.05
    fresh = (kv.float() + noise).to(sh.torch_dtype)
    fresh[:, :, T // 3] = kv[:, :, T // 3]  # an exactly unchanged position
    return kv, fresh


def _with_context(sh, kv, fresh, T, which):
    """The existing entry point on the same buffers (chunk table: all positions FRESH, no seams)."""

    class R:
        pass

    r = R()
    r.plan = synth.RequestPlan(T, [])
    r.chunks = [synth.Chunk(synth.ChunkPlan(i * sh.C, i * sh.C, synth.MODE_FRESH, synth.MATCH_MISS)) for i in range(T // sh.C)]
    r.kv_buf, r.fresh = kv, fresh
    ctx = B.create_for_shape(sh, 0, max_requests=1, max_chunks_total=T // sh.C, max_tokens_total=T)
    try:
        sel = B.SelectionTable([T], [0], [1], DEV)
        B.kvb_deviation_topk(ctx, B.RequestTable([r]), 0.0, 0, 0, 0, which, sel)
        B.kvb_last_status(ctx)
        return sel.delta[0].clone()
    finally:
        B.kvb_destroy(ctx)


def test_static_scratch_deviation_matches_context_path_twice_in_a_row():
    build_library()
    sh = synth.Shape(L=5, Hq=16, Hkv=2)
    model = B.kvb_model_desc(sh.L, sh.Hq, sh.Hkv, sh.d, sh.C, B.KVB_DT_BF16, sh.int4_group, 0, sh.theta)
    # second call is shorter and uses other data: leftovers of the first call must not leak into it
    free_after_first = None
    for T, which, seed in ((1152, 3, 1), (640, 1, 2), (1152, 3, 1)):
        kv, fresh = _case(sh, T, seed)
        want = _with_context(sh, kv, fresh, T, which)
        got = torch.full((T,), -1.0, dtype=torch.float32, device=DEV)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        assert B.kvb_deviation_static(0, model, kv, fresh, T, which, got) == B.KVB_OK
        torch.cuda.synchronize()
        # the point of the entry point: no device memory is taken by the call (the first call on a device may
        # make the runtime load the static array's module; from the second call on nothing may move)
        if free_after_first is not None:
            assert torch.cuda.mem_get_info()[0] == free_before
        free_after_first = torch.cuda.mem_get_info()[0]
        assert float((got - want).abs().max()) <= 1e-5
        assert torch.equal(got, want)  # same kernel, same exact integer sums
        assert float(got[T // 3]) == 0.0 and float(got.max()) > 1e-4
        # and against the oracle's fp64 deviation of the same buffers, at the deviation tolerance
        d64, _ = oracle.deviation(glue.bits_of(kv), glue.bits_of(fresh), oracle.DT_BF16, which)
        assert np.abs(got.cpu().numpy().astype(np.float64) - d64).max() <= 1e-5


@pytest.mark.parametrize("kv_dtype,Hkv,T", [("fp16", 1, 100), ("bf16", 1, 1), ("fp16", 4, 192), ("bf16", 2, 16384)])
def test_static_scratch_other_shapes(kv_dtype, Hkv, T):
    """One KV head (rows not paired), float16, prompts that end inside a tile, and the largest size."""
    build_library()
    sh = synth.Shape(L=2, Hq=8, Hkv=Hkv, kv_dtype=kv_dtype)
    dt = B.KVB_DT_BF16 if kv_dtype == "bf16" else B.KVB_DT_F16
    model = B.kvb_model_desc(sh.L, sh.Hq, sh.Hkv, sh.d, sh.C, dt, sh.int4_group, 0, sh.theta)
    kv, fresh = _case(sh, T, 7)
    got = torch.full((T,), -1.0, dtype=torch.float32, device=DEV)
    for _ in range(2):
        assert B.kvb_deviation_static(0, model, kv, fresh, T, 3, got) == B.KVB_OK
    torch.cuda.synchronize()
    d64, _ = oracle.deviation(glue.bits_of(kv), glue.bits_of(fresh), glue.dt_code(sh), 3)
    assert np.abs(got.cpu().numpy().astype(np.float64) - d64).max() <= 1e-5
    assert float(got[T // 3]) == 0.0


def test_static_scratch_rejects_what_it_cannot_hold():
    build_library()
    sh = synth.Shape(L=1)
    model = B.kvb_model_desc(sh.L, sh.Hq, sh.Hkv, sh.d, sh.C, B.KVB_DT_BF16, sh.int4_group, 0, sh.theta)
    kv, fresh = _case(sh, 128, 3)
    out = torch.zeros(128, dtype=torch.float32, device=DEV)
    assert B.kvb_deviation_static(0, model, kv, fresh, 16384 + 128, 3, out) == B.KVB_ERR_WORKSPACE
    assert B.kvb_deviation_static(0, model, kv, fresh, 0, 3, out) == B.KVB_ERR_INVALID_ARG
    assert B.kvb_deviation_static(0, model, kv, fresh, 128, 0, out) == B.KVB_ERR_INVALID_ARG
    bad = B.kvb_model_desc(sh.L, sh.Hq, sh.Hkv, 64, sh.C, B.KVB_DT_BF16, sh.int4_group, 0, sh.theta)
    assert B.kvb_deviation_static(0, bad, kv, fresh, 128, 3, out) == B.KVB_ERR_UNSUPPORTED
    assert not out.any()
