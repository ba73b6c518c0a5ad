"""Seeded synthetic workloads (input generators only).

This module draws random numbers and lays them out; it holds none of the
method's arithmetic.  Quantising a chunk and stitching the stale buffer are
done by callables the caller passes in: the tests pass the CPU oracle's, the
benchmark passes the CUDA library's.  Neither of those two ever imports the
other; this file imports neither.

The five workloads mirror the shapes the paper evaluates on (Qwen2.5-3B KV
shape: 36 layers, 16 query / 2 KV heads, head_dim 128, 128-token chunks, RoPE
base 1e6, recompute ratio 0.15, seam window 16) and stand in for its
bug-localisation benchmark, which is not reproduced here.

Value recipe: cached keys are N(0,1) * c with a per-(layer, head, channel)
factor c log-uniform in [0.1, 10]; values are N(0,1); both rounded to the KV
dtype.  The "fresh" projection of a cached token is the stitched (stale) value
plus N(0, sigma=0.01), plus N(0, sigma=0.3) on the first 16 tokens of each
cached chunk (the seam).  Fresh chunks carry their own data in the fresh
tensor.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, List, Optional

import numpy as np
import torch

MODE_FRESH, MODE_FP16, MODE_INT8, MODE_INT4 = 0, 1, 2, 3
MATCH_MISS, MATCH_EXACT, MATCH_APPROX = 0, 1, 2


@dataclasses.dataclass
class Shape:
    L: int = 36
    Hq: int = 16
    Hkv: int = 2
    d: int = 128
    C: int = 128
    theta: float = 1.0e6
    kv_dtype: str = "bf16"  # "bf16" | "fp16"
    int4_group: int = 32

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.kv_dtype == "bf16" else torch.float16


@dataclasses.dataclass
class ChunkPlan:
    new_pos: int
    orig_pos: int
    mode: int
    match: int


@dataclasses.dataclass
class RequestPlan:
    T: int
    chunks: List[ChunkPlan]


@dataclasses.dataclass
class SelectPlan:
    ratio: float = 0.15
    k_override: int = -1
    seam_before: int = 16
    seam_after: int = 0
    which: int = 3  # bit 0 keys, bit 1 values


@dataclasses.dataclass
class Workload:
    name: str
    seed: int
    shape: Shape
    requests: List[RequestPlan]
    select: SelectPlan
    sigma_bulk: float = 0.01
    sigma_seam: float = 0.3
    seam_tokens: int = 16


def _match(orig: int, new: int, mode: int) -> int:
    if mode == MODE_FRESH:
        return MATCH_MISS
    return MATCH_EXACT if orig == new else MATCH_APPROX


def _request(T, C, modes, origs) -> RequestPlan:
    chunks = []
    for i, (m, o) in enumerate(zip(modes, origs)):
        new = i * C
        o = new if m == MODE_FRESH else int(o)
        chunks.append(ChunkPlan(new, o, int(m), _match(o, new, int(m))))
    return RequestPlan(T, chunks)


def workload(idx: int, n_requests: Optional[int] = None) -> Workload:
    """The five named configurations (index = seed)."""
    rng = np.random.Generator(np.random.Philox(idx))
    if idx == 0:
        sh = Shape(L=1, Hq=16, Hkv=2, kv_dtype="fp16")
        modes = np.array([MODE_INT8] * 3 + [MODE_FRESH])
        rng.shuffle(modes)
        origs = rng.integers(0, 4096 - sh.C + 1, size=4)  # any integer position, not chunk aligned
        return Workload("cfg0_tiny", 0, sh, [_request(512, sh.C, modes, origs)], SelectPlan())
    if idx == 1:
        sh = Shape()
        modes = np.array([MODE_INT8] * 12 + [MODE_FRESH] * 4)
        rng.shuffle(modes)
        origs = rng.permutation(32768 // sh.C)[:16] * sh.C
        return Workload("cfg1_qwen3b_2k_int8", 1, sh, [_request(2048, sh.C, modes, origs)], SelectPlan())
    if idx in (2, 3):
        sh = Shape()
        rng = np.random.Generator(np.random.Philox(2))  # cfg3 attends to cfg2's buffer
        modes = np.array([MODE_INT4] * 56 + [MODE_FRESH] * 8)
        rng.shuffle(modes)
        origs = rng.permutation(64) * sh.C
        sel = SelectPlan(seam_before=0, seam_after=0) if idx == 2 else SelectPlan(k_override=1229, seam_before=0, seam_after=0)
        name = "cfg2_long_int4_8k" if idx == 2 else "cfg3_selective_attn_8k"
        return Workload(name, 2, sh, [_request(8192, sh.C, modes, origs)], sel)
    if idx == 4:
        sh = Shape()
        n = 32 if n_requests is None else n_requests
        reqs = []
        for _ in range(n):
            nch = int(rng.integers(4, 129))
            hit = rng.uniform(0.5, 0.95)
            n_hit = int(round(hit * nch))
            modes = np.array([MODE_FRESH] * nch)
            cached = rng.choice(nch, size=n_hit, replace=False)
            modes[cached] = rng.choice([MODE_FP16, MODE_INT8, MODE_INT4], size=n_hit, p=[0.4, 0.4, 0.2])
            origs = rng.permutation(32768 // sh.C)[:nch] * sh.C
            reqs.append(_request(nch * sh.C, sh.C, modes, origs))
        return Workload("cfg4_ragged_batch", 4, sh, reqs, SelectPlan())
    raise ValueError("workload index must be 0..4")


# ----------------------------------------------------------------------------------------
# tensors
# ----------------------------------------------------------------------------------------


@dataclasses.dataclass
class Chunk:
    plan: ChunkPlan
    k_codes: Optional[torch.Tensor] = None  # u8 [L,C,H,d] | u8 [L,C,H,d/2] | kv dtype [L,C,H,d]
    v_codes: Optional[torch.Tensor] = None
    k_meta: Optional[torch.Tensor] = None  # f32 [L,G_k,H,d,2]
    v_meta: Optional[torch.Tensor] = None  # f32 [L,C,H,G_v,2]
    meta_fp16: int = 0  # 1: the two metadata tensors hold binary16 pairs (torch.float16) instead


@dataclasses.dataclass
class Request:
    plan: RequestPlan
    chunks: List[Chunk]
    fresh: torch.Tensor  # kv dtype [L,2,T,H,d]
    kv_buf: torch.Tensor  # kv dtype [L,2,T,H,d] -- the stale stitched buffer the fresh tensor was built from
    q: torch.Tensor  # kv dtype [L,cap,Hq,d]
    sel_capacity: int


def sel_capacity(plan: RequestPlan, sp: SelectPlan) -> int:
    """Upper bound on the number of selected rows: k plus every seam window."""
    k = sp.k_override if sp.k_override >= 0 else int(math.floor(sp.ratio * plan.T))
    return min(plan.T, k + (len(plan.chunks) - 1) * (sp.seam_before + sp.seam_after))


def materialize(
    wl: Workload,
    device,
    quantize_k: Callable,
    quantize_v: Callable,
    assemble: Callable,
    request_ids=None,
) -> List[Request]:
    """Draw the tensors of a workload.

    quantize_k(x [L,C,H,d] kv-dtype tensor, bits, group_tokens) -> (codes u8, meta f32)
    quantize_v(x, bits, group_channels) -> (codes u8, meta f32)
    assemble(shape, plan, chunks, fresh) -> kv_buf tensor [L,2,T,H,d] (kv dtype)
    """
    sh = wl.shape
    dt = sh.torch_dtype
    out = []
    ids = range(len(wl.requests)) if request_ids is None else request_ids
    for r in ids:
        plan = wl.requests[r]
        g = torch.Generator(device=device)
        g.manual_seed(wl.seed * 1000003 + r)
        L, H, d, Cn, T = sh.L, sh.Hkv, sh.d, sh.C, plan.T
        # per-(layer, head, channel) key magnitude, log-uniform in [0.1, 10]
        u = torch.rand((L, 1, H, d), generator=g, device=device, dtype=torch.float32)
        c_ch = torch.exp(math.log(0.1) + u * (math.log(10.0) - math.log(0.1)))
        fresh = torch.zeros((L, 2, T, H, d), device=device, dtype=dt)
        chunks = []
        for cp in plan.chunks:
            k = (torch.randn((L, Cn, H, d), generator=g, device=device, dtype=torch.float32) * c_ch).to(dt)
            v = torch.randn((L, Cn, H, d), generator=g, device=device, dtype=torch.float32).to(dt)
            ck = Chunk(cp)
            if cp.mode == MODE_FRESH:
                fresh[:, 0, cp.new_pos : cp.new_pos + Cn] = k
                fresh[:, 1, cp.new_pos : cp.new_pos + Cn] = v
            elif cp.mode == MODE_FP16:
                ck.k_codes, ck.v_codes = k.contiguous(), v.contiguous()
            else:
                bits = 8 if cp.mode == MODE_INT8 else 4
                ck.k_codes, ck.k_meta = quantize_k(k, bits, Cn if bits == 8 else sh.int4_group)
                ck.v_codes, ck.v_meta = quantize_v(v, bits, d if bits == 8 else sh.int4_group)
            chunks.append(ck)
        kv_buf = assemble(sh, plan, chunks, fresh)
        for cp in plan.chunks:
            if cp.mode == MODE_FRESH:
                continue
            sl = slice(cp.new_pos, cp.new_pos + Cn)
            noise = torch.randn((L, 2, Cn, H, d), generator=g, device=device, dtype=torch.float32) * wl.sigma_bulk
            noise[:, :, : wl.seam_tokens] += (
                torch.randn((L, 2, wl.seam_tokens, H, d), generator=g, device=device, dtype=torch.float32) * wl.sigma_seam
            )
            fresh[:, :, sl] = (kv_buf[:, :, sl].float() + noise).to(dt)
        cap = sel_capacity(plan, wl.select)
        q = (torch.randn((L, cap, sh.Hq, d), generator=g, device=device, dtype=torch.float32) / math.sqrt(d)).to(dt)
        out.append(Request(plan, chunks, fresh, kv_buf, q, cap))
    return out


# ----------------------------------------------------------------------------------------
# closed-form byte / flop counts used by the benchmark's roofline lines
# ----------------------------------------------------------------------------------------


def assemble_bytes(sh: Shape, plan: RequestPlan, pair_bytes: int = 8) -> int:
    """Bytes the stitching step must move: packed codes + metadata read, buffer rows written.
    pair_bytes: size of one (scale, min) pair -- 8 (float32) or 4 (compact binary16 metadata)."""
    E = sh.Hkv * sh.d
    pb = pair_bytes
    total = 0
    for cp in plan.chunks:
        out_b = 2 * sh.C * E * 2  # K and V rows, 16-bit
        if cp.mode in (MODE_FRESH, MODE_FP16):
            in_b = out_b
        elif cp.mode == MODE_INT8:
            in_b = 2 * sh.C * E + E * pb + sh.C * sh.Hkv * pb
        else:
            g = sh.int4_group
            in_b = sh.C * E + (sh.C // g) * E * pb + sh.C * sh.Hkv * (sh.d // g) * pb
        total += sh.L * (in_b + out_b)
    return total


def deviation_bytes(sh: Shape, plan: RequestPlan, which: int) -> int:
    nw = (which & 1) + ((which >> 1) & 1)
    return sh.L * nw * plan.T * sh.Hkv * sh.d * 2 * 2  # stored + fresh rows, 16-bit


def one_pass_bytes(sh: Shape, plan: RequestPlan, which: int, pair_bytes: int = 8) -> int:
    """Bytes of the stitch with the deviation sums taken in the same pass: the stitch's own traffic
    plus one read of the fresh rows of every cached chunk (the stored rows are never read back, a
    FRESH chunk's rows are a copy and deviate by nothing)."""
    nw = (which & 1) + ((which >> 1) & 1)
    cached = sum(1 for cp in plan.chunks if cp.mode != MODE_FRESH)
    return assemble_bytes(sh, plan, pair_bytes) + sh.L * nw * cached * sh.C * sh.Hkv * sh.d * 2


def attention_flops(sh: Shape, sel) -> int:
    """Causal-useful flops only: 4*d per (query head, key) pair, keys 0..t."""
    s = int(np.sum(np.asarray(sel, dtype=np.int64) + 1))
    return sh.L * sh.Hq * 4 * sh.d * s
