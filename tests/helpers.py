"""Glue used by the tests only: torch <-> numpy views and oracle adapters for synth.materialize."""
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
