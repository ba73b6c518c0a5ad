"""Oracle-side glue for the tests, the smoke check and the benchmark's CPU legs: torch <-> numpy views and
oracle adapters for synth.materialize.  Imports the oracle and the input recipe; neither imports this."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2608_21362_b200 import synth


def dt_code(sh) -> int:
    return oracle.DT_BF16 if sh.kv_dtype == "bf16" else oracle.DT_F16


def bits_of(t: torch.Tensor) -> np.ndarray:
    """16-bit float tensor -> uint16 numpy bit patterns (host copy)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, dtype, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(dtype).to(device)


def f64_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def oracle_quantize_k(x: torch.Tensor, bits: int, group_tokens: int):
    xs = f64_of(x)
    codes, metas = zip(*[oracle.quantize_k(xs[l], bits, group_tokens) for l in range(xs.shape[0])])
    return (torch.from_numpy(np.stack(codes)).to(x.device), torch.from_numpy(np.stack(metas)).to(x.device))


def oracle_quantize_v(x: torch.Tensor, bits: int, group_ch: int):
    xs = f64_of(x)
    codes, metas = zip(*[oracle.quantize_v(xs[l], bits, group_ch) for l in range(xs.shape[0])])
    return (torch.from_numpy(np.stack(codes)).to(x.device), torch.from_numpy(np.stack(metas)).to(x.device))


def oracle_chunk_dicts(chunks):
    out = []
    for ck in chunks:
        d = dict(orig_pos=ck.plan.orig_pos, new_pos=ck.plan.new_pos, mode=ck.plan.mode)
        d["n_tokens"] = None
        for name in ("k_codes", "v_codes", "k_meta", "v_meta"):
            t = getattr(ck, name)
            if t is None:
                d[name] = None
            elif name.endswith("_meta"):  # compact (binary16) pairs reach the oracle as the float32 values they hold
                d[name] = t.detach().cpu().float().numpy()
            elif t.dtype in (torch.bfloat16, torch.float16):
                d[name] = bits_of(t)
            else:
                d[name] = t.detach().cpu().numpy()
        out.append(d)
    return out


def oracle_assemble_np(sh, plan, chunks, fresh_bits, want_exact=False):
    dicts = oracle_chunk_dicts(chunks)
    for d in dicts:
        d["n_tokens"] = sh.C
    return oracle.assemble(dicts, sh.L, sh.Hkv, sh.d, plan.T, sh.theta, dt_code(sh), sh.int4_group, fresh_bits, want_exact)


def oracle_assemble(sh, plan, chunks, fresh: torch.Tensor) -> torch.Tensor:
    kv = oracle_assemble_np(sh, plan, chunks, bits_of(fresh))
    return from_bits(kv, sh.torch_dtype, fresh.device)


def materialize_with_oracle(wl, device="cpu", request_ids=None):
    """Inputs for a workload, with every method step of the input recipe taken by the oracle."""
    return synth.materialize(wl, device, oracle_quantize_k, oracle_quantize_v, oracle_assemble, request_ids)


# ---- the stitched-row tolerance (tests and the smoke check share it)


def ulp16(y, kv_dtype):
    a = np.abs(y)
    e = np.floor(np.log2(np.maximum(a, 1e-300)))
    if kv_dtype == "bf16":
        return np.exp2(np.maximum(e, -126) - 7)
    return np.exp2(np.maximum(e, -14) - 10)


def check_assembled(sh, req, kv_gpu_bits, exact, kv_oracle_bits):
    """Element-wise tolerance check of a stitched buffer plus a bit-agreement count."""
    dtc = dt_code(sh)
    g = oracle.bits_to_f64(kv_gpu_bits, dtc)
    half = sh.d // 2
    pre_worst = 0.0
    for ck in req.chunks:
        sl = slice(ck.plan.new_pos, ck.plan.new_pos + sh.C)
        if ck.plan.mode == synth.MODE_FRESH:
            assert np.array_equal(kv_gpu_bits[:, :, sl], kv_oracle_bits[:, :, sl]), "fresh rows must be bit copies"
            continue
        y = exact[:, :, sl]  # [L,2,C,H,d]
        M = np.abs(y).max(axis=(2, 3, 4), keepdims=True)
        ref = np.abs(y).copy()
        pair = np.sqrt(y[:, 0, ..., :half] ** 2 + y[:, 0, ..., half:] ** 2)
        ref[:, 0, ..., :half] = pair
        ref[:, 0, ..., half:] = pair
        bound = 1e-3 * ref + 0.5 * ulp16(y, sh.kv_dtype) + 2e-6 * M
        err = np.abs(g[:, :, sl] - y)
        worst = float((err / bound).max())
        assert worst <= 1.0, "chunk at %d (mode %d): error %.3g x bound" % (ck.plan.new_pos, ck.plan.mode, worst)
        # The same bar without the rounding allowance, where the data can show it: at an element whose
        # stored bits differ from the oracle's rounding, the GPU's value before its 16-bit store lay on the
        # other side of the midpoint between the two 16-bit neighbours, so it was at least |y - midpoint|
        # away from y.  That inferred float32 error must itself be within 1e-3 relative (+ the float32
        # term): the whole difference is then the rounding both sides make, not the arithmetic.
        o = oracle.bits_to_f64(kv_oracle_bits[:, :, sl], dtc)
        differ = kv_gpu_bits[:, :, sl] != kv_oracle_bits[:, :, sl]
        if differ.any():
            pre = np.abs(y - 0.5 * (g[:, :, sl] + o))[differ]
            lim = (1e-3 * ref + 2e-6 * M)[differ]
            pre_worst = max(pre_worst, float((pre / lim).max()))
            assert pre_worst <= 1.0, "chunk at %d: float32 error before the store at least %.3g x (1e-3 relative)" % (ck.plan.new_pos, pre_worst)
    # Beyond the tolerance: how often the two 16-bit roundings coincide.  The GPU rounds a float32 result
    # whose error e is a few 2^-24 of the chunk's magnitude M, the oracle rounds the exact value; they
    # differ when y lies within e of a rounding boundary, i.e. with probability ~ 2e / ulp16(y)
    # = c * 2^-23 * (M/|y|) / 2^-p (p = 8 bits for bf16, 11 for fp16; c ~ 2..3, mean M/|y| ~ 3):
    # about 3e-4 in bf16 and 2e-3 in fp16 (measured: up to 2.2e-3 on int4 keys in fp16).
    agree = float(np.mean(kv_gpu_bits == kv_oracle_bits))
    floor = 0.999 if sh.kv_dtype == "bf16" else 0.995
    assert agree > floor, "only %.5f of stored values equal the oracle's rounding bit for bit" % agree
    print("stitched rows: %.5f bit-equal to the oracle's rounding; inferred pre-store error at most %.3g of the 1e-3 relative bar" % (agree, pre_worst))
    return agree
