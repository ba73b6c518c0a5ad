"""CPU oracle for the KV-chunk stitching path (test infrastructure, not product).

Thin numpy/ctypes marshalling around ``kvb_oracle.c``; every step of the
arithmetic lives in that C file, written from the paper (KV Quantization Eq. 6,
Rotary Positional Embeddings Eq. 3, Prompt Assembly, Algorithms 1 and 2,
attention Eq. 2).  Nothing here imports the CUDA package, and the CUDA package
never imports this.  Only ``tests/``, ``__graft_entry__.smoke()`` and the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py`` may use it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvb_oracle.c")
_LIB = os.path.join(_HERE, "libkvb_oracle.so")

MODE_FRESH, MODE_FP16, MODE_INT8, MODE_INT4 = 0, 1, 2, 3
DT_F16, DT_BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 (+OpenMP); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Chunk(C.Structure):
    _fields_ = [
        ("orig_pos", C.c_int32),
        ("new_pos", C.c_int32),
        ("n_tokens", C.c_int32),
        ("mode", C.c_int32),
        ("k_codes", C.c_void_p),
        ("v_codes", C.c_void_p),
        ("k_meta", C.c_void_p),
        ("v_meta", C.c_void_p),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.kvo_bf16_to_f64.restype = C.c_double
        _lib.kvo_f16_to_f64.restype = C.c_double
        _lib.kvo_f64_to_bf16.restype = C.c_uint16
        _lib.kvo_f64_to_f16.restype = C.c_uint16
        _lib.kvo_f64_to_bf16.argtypes = [C.c_double]
        _lib.kvo_f64_to_f16.argtypes = [C.c_double]
        _lib.kvo_select_count.argtypes = [C.c_int, C.c_double]
        _lib.kvo_select_count.restype = C.c_int
        _lib.kvo_seam_select.restype = C.c_int
        _lib.kvo_max_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def max_threads() -> int:
    return int(lib().kvo_max_threads())


def set_threads(n: int) -> None:
    """Threads the oracle's parallel loops use from now on (for one-core vs all-core timings)."""
    lib().kvo_set_threads(int(n))


# ---------------------------------------------------------------- 16-bit formats
def round_to_bits(x, dtype: int) -> np.ndarray:
    """float64 array -> uint16 bit patterns of bf16 / fp16 (nearest-even, one rounding)."""
    x = _c(x, np.float64)
    out = np.empty(x.shape, np.uint16)
    lib().kvo_round_array(_p(x), C.c_int64(x.size), C.c_int(dtype), _p(out))
    return out


def bits_to_f64(b, dtype: int) -> np.ndarray:
    b = _c(b, np.uint16)
    out = np.empty(b.shape, np.float64)
    lib().kvo_decode_array(_p(b), C.c_int64(b.size), C.c_int(dtype), _p(out))
    return out


# ---------------------------------------------------------------- Eq. 6
def quantize_k(x, bits: int, group_tokens: int, meta16: bool = False):
    """x [C,H,d] float64 -> (codes u8 [C,H,d] or [C,H,d/2], meta f32 [C/group,H,d,2]).
    meta16: compact metadata (min rounded down, scale rounded up to binary16; returned as float32)."""
    x = _c(x, np.float64)
    Cn, H, d = x.shape
    codes = np.zeros((Cn, H, d * bits // 8), np.uint8)
    meta = np.zeros((Cn // group_tokens, H, d, 2), np.float32)
    lib().kvo_quantize_k_ex(_p(x), Cn, H, d, bits, group_tokens, int(meta16), _p(codes), _p(meta))
    return codes, meta


def quantize_v(x, bits: int, group_ch: int, meta16: bool = False):
    """x [C,H,d] float64 -> (codes, meta f32 [C,H,d/group,2])."""
    x = _c(x, np.float64)
    Cn, H, d = x.shape
    codes = np.zeros((Cn, H, d * bits // 8), np.uint8)
    meta = np.zeros((Cn, H, d // group_ch, 2), np.float32)
    lib().kvo_quantize_v_ex(_p(x), Cn, H, d, bits, group_ch, int(meta16), _p(codes), _p(meta))
    return codes, meta


def dequant_k(codes, meta, d: int, bits: int, group_tokens: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    meta = _c(meta, np.float32)
    Cn, H = codes.shape[0], codes.shape[1]
    out = np.empty((Cn, H, d), np.float64)
    lib().kvo_dequant_k(_p(codes), _p(meta), Cn, H, d, bits, group_tokens, _p(out))
    return out


def dequant_v(codes, meta, d: int, bits: int, group_ch: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    meta = _c(meta, np.float32)
    Cn, H = codes.shape[0], codes.shape[1]
    out = np.empty((Cn, H, d), np.float64)
    lib().kvo_dequant_v(_p(codes), _p(meta), Cn, H, d, bits, group_ch, _p(out))
    return out


# ---------------------------------------------------------------- Eq. 3
def rope_rotate(rows, theta: float, delta: float) -> np.ndarray:
    """rows [n,H,d] float64 -> R_theta^{delta} applied to every row (copy)."""
    r = np.array(rows, dtype=np.float64, order="C", copy=True)
    n, H, d = r.shape
    lib().kvo_rope_rotate(_p(r), C.c_int64(n), H, d, C.c_double(theta), C.c_double(delta))
    return r


def unrotate_keys(rows_bits, dtype: int, theta: float, orig_pos: int) -> np.ndarray:
    """rows_bits [n,H,d] uint16 -> float64 array of the float32 values R_theta^{-orig_pos} x (the keys of
    a position-free cache entry, before Eq. 6 is applied)."""
    r = _c(rows_bits, np.uint16)
    n, H, d = r.shape
    out = np.zeros((n, H, d), np.float64)
    lib().kvo_unrotate_keys_f32(_p(r), C.c_int64(n), H, d, dtype, C.c_double(theta), int(orig_pos), _p(out))
    return out


# ---------------------------------------------------------------- assembly
def assemble(chunks, L, H, d, T, theta, dtype, int4_group, fresh, want_exact=False):
    """chunks: list of dicts {orig_pos,new_pos,n_tokens,mode,k_codes,v_codes,k_meta,v_meta}
    (numpy arrays, layouts of the C file).  fresh: uint16 [L,2,T,H,d].
    Returns kv_buf uint16 [L,2,T,H,d] (rows no chunk covers stay 0) and, if asked,
    the un-rounded float64 tensor."""
    fresh = _c(fresh, np.uint16)
    arr = (_Chunk * max(1, len(chunks)))()
    keep = []
    for i, ck in enumerate(chunks):
        arr[i].orig_pos, arr[i].new_pos = int(ck["orig_pos"]), int(ck["new_pos"])
        arr[i].n_tokens, arr[i].mode = int(ck["n_tokens"]), int(ck["mode"])
        for name, dt in (("k_codes", None), ("v_codes", None), ("k_meta", np.float32), ("v_meta", np.float32)):
            a = ck.get(name)
            if a is not None:
                a = np.ascontiguousarray(a) if dt is None else _c(a, dt)
                keep.append(a)
                setattr(arr[i], name, a.ctypes.data)
    kv = np.zeros((L, 2, T, H, d), np.uint16)
    exact = np.zeros((L, 2, T, H, d), np.float64) if want_exact else None
    lib().kvo_assemble(arr, len(chunks), L, H, d, T, C.c_double(theta), dtype, int4_group, _p(fresh), _p(kv), _p(exact))
    return (kv, exact) if want_exact else kv


# ---------------------------------------------------------------- Algorithm 2 / 1
def deviation(kv_buf, fresh, dtype: int, which: int = 3):
    kv_buf = _c(kv_buf, np.uint16)
    fresh = _c(fresh, np.uint16)
    L, _, T, H, d = kv_buf.shape
    d64 = np.empty(T, np.float64)
    d32 = np.empty(T, np.float32)
    lib().kvo_deviation(_p(kv_buf), _p(fresh), L, H, d, T, dtype, which, _p(d64), _p(d32))
    return d64, d32


def select_count(T: int, ratio: float) -> int:
    return int(lib().kvo_select_count(T, ratio))


def topk(delta32, k: int) -> np.ndarray:
    delta32 = _c(delta32, np.float32)
    rank = np.empty(max(k, 0), np.int32)
    lib().kvo_topk(_p(delta32), int(delta32.size), int(k), _p(rank))
    return rank


def seam_select(rank, chunk_new_pos, chunk_mode, T: int, before: int, after: int, sinks: int = 0) -> np.ndarray:
    rank = _c(rank, np.int32)
    pos = _c(chunk_new_pos, np.int32)
    mode = _c(chunk_mode, np.int32)
    sel = np.empty(max(T, 1), np.int32)
    n = lib().kvo_seam_select(_p(rank), int(rank.size), _p(pos), _p(mode), int(pos.size), T, before, after, int(sinks), _p(sel))
    return sel[:n].copy()


# ---------------------------------------------------------------- Eq. 2
def attention(q, kv_buf, sel, Hq: int, dtype: int, scale: float, layers=None, rows=None, want_exact=False):
    """q uint16 [L,cap,Hq,d]; kv_buf uint16 [L,2,T,Hkv,d]; sel int32 [n_sel].
    Returns out uint16 [L,cap,Hq,d] (only the requested layers/rows are written)."""
    q = _c(q, np.uint16)
    kv_buf = _c(kv_buf, np.uint16)
    sel = _c(sel, np.int32)
    L, _, T, Hkv, d = kv_buf.shape
    cap = q.shape[1]
    layers = _c(np.arange(L) if layers is None else layers, np.int32)
    rows_a = None if rows is None else _c(rows, np.int32)
    out = np.zeros(q.shape, np.uint16)
    exact = np.zeros(q.shape, np.float64) if want_exact else None
    lib().kvo_attention(
        _p(q), _p(kv_buf), _p(sel), int(sel.size), cap, L, Hq, Hkv, d, T, dtype, C.c_double(scale),
        _p(layers), int(layers.size), _p(rows_a), 0 if rows_a is None else int(rows_a.size), _p(out), _p(exact),
    )
    return (out, exact) if want_exact else out


# ---------------------------------------------------------------- Algorithm 2 step 4; Eq. 7
def patch(kv_buf, fresh, sel) -> np.ndarray:
    """Copy of kv_buf with the rows of the selected positions replaced by the fresh ones."""
    kv = np.array(kv_buf, dtype=np.uint16, order="C", copy=True)
    fresh = _c(fresh, np.uint16)
    sel = _c(sel, np.int32)
    L, _, T, H, d = kv.shape
    lib().kvo_patch(_p(kv), _p(fresh), _p(sel), int(sel.size), L, T, H, d)
    return kv


def importance(kv_buf, C_tokens: int, dtype: int) -> np.ndarray:
    """Mean key norm of every chunk of a stitched buffer (Eq. 7)."""
    kv = _c(kv_buf, np.uint16)
    L, _, T, H, d = kv.shape
    out = np.empty(T // C_tokens, np.float64)
    lib().kvo_importance(_p(kv), L, T, H, d, C_tokens, dtype, _p(out))
    return out
