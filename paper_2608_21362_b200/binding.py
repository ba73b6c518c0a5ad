"""ctypes binding of libkvb: same entry-point names as include/kvb.h, argument marshalling only.

Tensors are torch CUDA tensors (torch provides device memory and streams); every step of the
path runs in the library's kernels.  There is no fallback: if the shared library is missing or
fails to load, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libkvb.so")

KVB_OK = 0
(KVB_ERR_INVALID_ARG, KVB_ERR_BAD_TABLE, KVB_ERR_UNSUPPORTED, KVB_ERR_WORKSPACE, KVB_ERR_CUDA,
 KVB_ERR_DEVICE_STATUS, KVB_ERR_NO_DEVICE) = range(1, 8)
KVB_MODE_FRESH, KVB_MODE_FP16, KVB_MODE_INT8, KVB_MODE_INT4 = 0, 1, 2, 3
KVB_MATCH_MISS, KVB_MATCH_EXACT, KVB_MATCH_APPROX = 0, 1, 2
KVB_DT_F16, KVB_DT_BF16 = 0, 1


class kvb_chunk(C.Structure):
    _fields_ = [
        ("content_hash", C.c_uint8 * 32),
        ("prefix_hash", C.c_uint8 * 32),
        ("orig_pos", C.c_int32),
        ("new_pos", C.c_int32),
        ("n_tokens", C.c_int32),
        ("mode", C.c_int32),
        ("match", C.c_int32),
        ("meta_fp16", C.c_int32),
        ("k_codes", C.c_void_p),
        ("v_codes", C.c_void_p),
        ("k_meta", C.c_void_p),
        ("v_meta", C.c_void_p),
    ]


class kvb_request(C.Structure):
    _fields_ = [
        ("T", C.c_int32),
        ("n_chunks", C.c_int32),
        ("chunks", C.POINTER(kvb_chunk)),
        ("kv_buf", C.c_void_p),
        ("fresh", C.c_void_p),
        ("importance", C.c_void_p),
    ]


class kvb_model_desc(C.Structure):
    _fields_ = [
        ("L", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
        ("chunk_tokens", C.c_int32), ("kv_dtype", C.c_int32), ("int4_group", C.c_int32), ("reserved", C.c_int32),
        ("rope_theta", C.c_double),
    ]


class kvb_limits(C.Structure):
    _fields_ = [("max_requests", C.c_int32), ("max_chunks_total", C.c_int32), ("max_tokens_total", C.c_int64)]


class kvb_select_params(C.Structure):
    _fields_ = [
        ("ratio", C.c_double), ("k_override", C.c_int32), ("seam_before", C.c_int32),
        ("seam_after", C.c_int32), ("which", C.c_int32), ("sink_tokens", C.c_int32), ("reserved", C.c_int32),
    ]


class kvb_selection(C.Structure):
    _fields_ = [
        ("delta", C.c_void_p), ("rank", C.c_void_p), ("sel", C.c_void_p), ("n_sel", C.c_void_p),
        ("sel_capacity", C.c_int32), ("reserved", C.c_int32),
    ]


class kvb_quantize_job(C.Structure):
    _fields_ = [
        ("k", C.c_void_p), ("v", C.c_void_p), ("k_codes", C.c_void_p), ("v_codes", C.c_void_p),
        ("k_meta", C.c_void_p), ("v_meta", C.c_void_p),
        ("bits", C.c_int32), ("unrotate_from", C.c_int32), ("meta_fp16", C.c_int32), ("reserved", C.c_int32),
    ]


class KvbError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("kvb status %d (%s): %s" % (status, kvb_status_string(status), message))
        self.status = status


_lib = None


def lib():
    """Loads libkvb.so (built by paper_2608_21362_b200.build); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("libkvb.so is not built: run `python -m paper_2608_21362_b200.build` (needs nvcc); there is no CPU fallback")
        L = C.CDLL(_LIB_PATH)
        vp = C.c_void_p
        L.kvb_create.argtypes = [C.POINTER(vp), C.c_int, C.POINTER(kvb_model_desc), C.POINTER(kvb_limits)]
        L.kvb_destroy.argtypes = [vp]
        L.kvb_assemble.argtypes = [vp, C.POINTER(kvb_request), C.c_int, vp]
        L.kvb_deviation_topk.argtypes = [vp, C.POINTER(kvb_request), C.c_int, C.POINTER(kvb_select_params), C.POINTER(kvb_selection), vp]
        L.kvb_assemble_select.argtypes = L.kvb_deviation_topk.argtypes
        L.kvb_selective_attn.argtypes = [vp, C.POINTER(kvb_request), C.c_int, C.POINTER(kvb_selection), C.POINTER(vp), C.POINTER(vp), C.c_float, vp]
        L.kvb_quantize_chunk.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp, vp]
        L.kvb_quantize_keys_at.argtypes = [vp, vp, C.c_int, C.c_int, vp, vp, vp]
        L.kvb_quantize_chunk_ex.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp]
        L.kvb_select_count.argtypes = [C.c_int, C.c_double]
        L.kvb_validate.argtypes = [C.POINTER(kvb_model_desc), C.POINTER(kvb_limits), C.POINTER(kvb_request), C.c_int, C.c_int, C.c_char_p, C.c_size_t]
        L.kvb_last_status.argtypes = [vp]
        L.kvb_last_error.argtypes = [vp]
        L.kvb_last_error.restype = C.c_char_p
        L.kvb_status_string.argtypes = [C.c_int]
        L.kvb_status_string.restype = C.c_char_p
        L.kvb_launch_count.argtypes = [vp]
        L.kvb_launch_count.restype = C.c_int64
        _lib = L
    return _lib


# ------------------------------------------------------------------ marshalled tables
class RequestTable:
    """Host-side kvb_request array built once from tensors and reusable across calls."""

    def __init__(self, requests: Sequence, chunk_tokens: int = 128):
        """requests: objects with .plan.T, .chunks (each .plan.{orig_pos,new_pos,mode,match} and the
        four tensors or None), .kv_buf, .fresh, optionally .importance -- e.g. synth.Request."""
        self._keep = []
        n = len(requests)
        self.n = n
        self.array = (kvb_request * max(n, 1))()
        for r, rq in enumerate(requests):
            chunks = (kvb_chunk * max(len(rq.chunks), 1))()
            self._keep.append(chunks)
            for i, ck in enumerate(rq.chunks):
                p = ck.plan
                chunks[i].orig_pos, chunks[i].new_pos = p.orig_pos, p.new_pos
                chunks[i].n_tokens = chunk_tokens
                chunks[i].mode, chunks[i].match = p.mode, p.match
                chunks[i].meta_fp16 = int(getattr(ck, "meta_fp16", 0))
                for name in ("k_codes", "v_codes", "k_meta", "v_meta"):
                    t = getattr(ck, name)
                    if t is not None:
                        self._keep.append(t)
                        setattr(chunks[i], name, t.data_ptr())
            self.array[r].T = rq.plan.T
            self.array[r].n_chunks = len(rq.chunks)
            self.array[r].chunks = chunks
            self.array[r].kv_buf = rq.kv_buf.data_ptr()
            self.array[r].fresh = rq.fresh.data_ptr()
            self._keep += [rq.kv_buf, rq.fresh]
            imp = getattr(rq, "importance", None)  # optional [n_chunks] float32 tensor: Eq. 7 from the stitch
            if imp is not None:
                self.array[r].importance = imp.data_ptr()
                self._keep.append(imp)


class SelectionTable:
    """Per-request selection outputs (device tensors) plus the marshalled kvb_selection array."""

    def __init__(self, Ts: Sequence[int], ks: Sequence[int], capacities: Sequence[int], device):
        self.n = len(Ts)
        self.delta = [torch.zeros(T, dtype=torch.float32, device=device) for T in Ts]
        self.rank = [torch.full((max(k, 1),), -1, dtype=torch.int32, device=device) for k in ks]
        self.sel = [torch.full((cap,), -1, dtype=torch.int32, device=device) for cap in capacities]
        self.n_sel = torch.zeros(max(self.n, 1), dtype=torch.int32, device=device)
        self.array = (kvb_selection * max(self.n, 1))()
        for r in range(self.n):
            a = self.array[r]
            a.delta, a.rank, a.sel = self.delta[r].data_ptr(), self.rank[r].data_ptr(), self.sel[r].data_ptr()
            a.n_sel = self.n_sel.data_ptr() + 4 * r
            a.sel_capacity = capacities[r]


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(ctx, st: int):
    if st != KVB_OK:
        raise KvbError(st, kvb_last_error(ctx) if ctx else "")
    return st


# ------------------------------------------------------------------ entry points (names of include/kvb.h)
def kvb_status_string(status: int) -> str:
    return lib().kvb_status_string(status).decode()


def kvb_last_error(ctx) -> str:
    return lib().kvb_last_error(ctx).decode()


def kvb_select_count(T: int, ratio: float) -> int:
    return int(lib().kvb_select_count(T, ratio))


def kvb_validate(model: kvb_model_desc, limits: kvb_limits, table, need_payload: bool = True):
    """Host-only table check; returns (status, message)."""
    buf = C.create_string_buffer(512)
    arr = table.array if table is not None else None
    n = table.n if table is not None else 0
    st = lib().kvb_validate(C.byref(model), C.byref(limits), arr, n, int(need_payload), buf, 512)
    return int(st), buf.value.decode()


def kvb_create(device: int, L: int, Hq: int, Hkv: int, d: int, chunk_tokens: int, rope_theta: float, kv_dtype: int,
               int4_group: int, max_requests: int, max_chunks_total: int, max_tokens_total: int, check: bool = True):
    m = kvb_model_desc(L, Hq, Hkv, d, chunk_tokens, kv_dtype, int4_group, 0, rope_theta)
    lim = kvb_limits(max_requests, max_chunks_total, max_tokens_total)
    ctx = C.c_void_p()
    st = lib().kvb_create(C.byref(ctx), device, C.byref(m), C.byref(lim))
    if st != KVB_OK:
        msg = kvb_last_error(ctx) if ctx else ""
        if ctx:
            lib().kvb_destroy(ctx)
        if check:
            raise KvbError(st, msg)
        return None, st
    return ctx if check else (ctx, st)


def kvb_destroy(ctx) -> int:
    return int(lib().kvb_destroy(ctx))


def kvb_assemble(ctx, table: RequestTable, stream=None, check: bool = True) -> int:
    st = lib().kvb_assemble(ctx, table.array, table.n, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_deviation_topk(ctx, table: RequestTable, ratio: float, k_override: int, seam_before: int, seam_after: int,
                       which: int, out: SelectionTable, stream=None, check: bool = True, sink_tokens: int = 0) -> int:
    p = kvb_select_params(ratio, k_override, seam_before, seam_after, which, sink_tokens, 0)
    st = lib().kvb_deviation_topk(ctx, table.array, table.n, C.byref(p), out.array, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_assemble_select(ctx, table: RequestTable, ratio: float, k_override: int, seam_before: int, seam_after: int,
                        which: int, out: SelectionTable, stream=None, check: bool = True, sink_tokens: int = 0) -> int:
    p = kvb_select_params(ratio, k_override, seam_before, seam_after, which, sink_tokens, 0)
    st = lib().kvb_assemble_select(ctx, table.array, table.n, C.byref(p), out.array, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_selective_attn(ctx, table: RequestTable, sel: SelectionTable, q: List[torch.Tensor], out: List[torch.Tensor],
                       softmax_scale: float, stream=None, check: bool = True) -> int:
    n = table.n
    qp = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in q])
    op = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in out])
    st = lib().kvb_selective_attn(ctx, table.array, n, sel.array, qp, op, softmax_scale, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_patch(ctx, table: RequestTable, sel: SelectionTable, stream=None, check: bool = True) -> int:
    L = lib()
    L.kvb_patch.argtypes = [C.c_void_p, C.POINTER(kvb_request), C.c_int, C.POINTER(kvb_selection), C.c_void_p]
    st = L.kvb_patch(ctx, table.array, table.n, sel.array, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_chunk_importance(ctx, table: RequestTable, importance: List[torch.Tensor], stream=None, check: bool = True) -> int:
    L = lib()
    L.kvb_chunk_importance.argtypes = [C.c_void_p, C.POINTER(kvb_request), C.c_int, C.POINTER(C.c_void_p), C.c_void_p]
    ptrs = (C.c_void_p * max(table.n, 1))(*[t.data_ptr() for t in importance])
    st = L.kvb_chunk_importance(ctx, table.array, table.n, ptrs, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_quantize_chunk(ctx, x: torch.Tensor, is_value: bool, bits: int, codes: torch.Tensor, meta: torch.Tensor,
                       stream=None, check: bool = True) -> int:
    st = lib().kvb_quantize_chunk(ctx, x.data_ptr(), int(is_value), bits, codes.data_ptr(), meta.data_ptr(), _stream(stream))
    return _check(ctx, st) if check else st


def kvb_quantize_keys_at(ctx, x: torch.Tensor, orig_pos: int, bits: int, codes: torch.Tensor, meta: torch.Tensor,
                         stream=None, check: bool = True) -> int:
    st = lib().kvb_quantize_keys_at(ctx, x.data_ptr(), int(orig_pos), bits, codes.data_ptr(), meta.data_ptr(), _stream(stream))
    return _check(ctx, st) if check else st


def kvb_quantize_chunk_ex(ctx, x: torch.Tensor, is_value: bool, bits: int, unrotate_from: int, meta_fp16: bool,
                          codes: torch.Tensor, meta: torch.Tensor, stream=None, check: bool = True) -> int:
    st = lib().kvb_quantize_chunk_ex(ctx, x.data_ptr(), int(is_value), bits, int(unrotate_from), int(meta_fp16),
                                     codes.data_ptr(), meta.data_ptr(), _stream(stream))
    return _check(ctx, st) if check else st


class QuantizeTable:
    """Host-side kvb_quantize_job array built once from tensors and reusable across calls.
    jobs: dicts with k / v (tensors or None), k_codes, v_codes, k_meta, v_meta (tensors), bits, and
    optionally unrotate_from (default -1) and meta_fp16 (default False)."""

    def __init__(self, jobs: Sequence[dict]):
        self.n = len(jobs)
        self._keep = list(jobs)
        self.array = (kvb_quantize_job * max(self.n, 1))()
        for a, j in zip(self.array, jobs):
            for name in ("k", "v", "k_codes", "v_codes", "k_meta", "v_meta"):
                t = j.get(name)
                if t is not None:
                    setattr(a, name, t.data_ptr())
            a.bits, a.unrotate_from, a.meta_fp16 = int(j["bits"]), int(j.get("unrotate_from", -1)), int(j.get("meta_fp16", False))


def kvb_quantize_chunks(ctx, jobs, stream=None, check: bool = True) -> int:
    """jobs: a QuantizeTable, or a list of job dicts (marshalled on the spot)."""
    L = lib()
    L.kvb_quantize_chunks.argtypes = [C.c_void_p, C.POINTER(kvb_quantize_job), C.c_int, C.c_void_p]
    tbl = jobs if isinstance(jobs, QuantizeTable) else QuantizeTable(jobs)
    st = L.kvb_quantize_chunks(ctx, tbl.array, tbl.n, _stream(stream))
    return _check(ctx, st) if check else st


def kvb_deviation_static(device: int, model: kvb_model_desc, kv_buf: torch.Tensor, fresh: torch.Tensor, T: int,
                         which: int, delta: torch.Tensor, stream=None) -> int:
    """Deviation of one request without a context and without any allocation (static device scratch,
    T <= 16384).  Returns the status code; the caller owns kv_buf, fresh and delta."""
    L = lib()
    L.kvb_deviation_static.argtypes = [C.c_int, C.POINTER(kvb_model_desc), C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    return int(L.kvb_deviation_static(device, C.byref(model), kv_buf.data_ptr(), fresh.data_ptr(), T, which, delta.data_ptr(), _stream(stream)))


def kvb_last_status(ctx, check: bool = True) -> int:
    st = lib().kvb_last_status(ctx)
    return _check(ctx, st) if check else st


def kvb_launch_count(ctx) -> int:
    return int(lib().kvb_launch_count(ctx))


def kvb_set_debug_option(ctx, key: str, value: int, check: bool = True) -> int:
    L = lib()
    L.kvb_set_debug_option.argtypes = [C.c_void_p, C.c_char_p, C.c_int]
    st = L.kvb_set_debug_option(ctx, key.encode(), int(value))
    return _check(ctx, st) if check else st


def kvb_selftest_wait_timeout(ctx, limit_ms: int, stream=None, check: bool = True) -> int:
    L = lib()
    L.kvb_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
    st = L.kvb_selftest_wait_timeout(ctx, limit_ms, _stream(stream))
    return _check(ctx, st) if check else st


# ------------------------------------------------------------------ small conveniences over the entry points
def create_for_shape(sh, device: int = 0, max_requests: int = 64, max_chunks_total: int = 8192,
                     max_tokens_total: int = 1 << 20):
    """Context for a synth.Shape-like object (fields L, Hq, Hkv, d, C, theta, kv_dtype, int4_group)."""
    dt = KVB_DT_BF16 if sh.kv_dtype == "bf16" else KVB_DT_F16
    return kvb_create(device, sh.L, sh.Hq, sh.Hkv, sh.d, sh.C, sh.theta, dt, sh.int4_group, max_requests,
                      max_chunks_total, max_tokens_total)


def quantize_fns(ctx, sh, meta_fp16: bool = False):
    """(quantize_k, quantize_v) callables in the form synth.materialize expects, running the CUDA quantiser.
    meta_fp16: compact metadata (torch.float16 pairs; mark the chunk with meta_fp16 = 1)."""
    mt = torch.float16 if meta_fp16 else torch.float32

    def _q(x: torch.Tensor, bits: int, is_value: bool):
        L, Cn, H, d = x.shape
        x = x.contiguous()
        codes = torch.empty((L, Cn, H, d * bits // 8), dtype=torch.uint8, device=x.device)
        if is_value:
            meta = torch.empty((L, Cn, H, 1 if bits == 8 else d // sh.int4_group, 2), dtype=mt, device=x.device)
        else:
            meta = torch.empty((L, 1 if bits == 8 else Cn // sh.int4_group, H, d, 2), dtype=mt, device=x.device)
        kvb_quantize_chunk_ex(ctx, x, is_value, bits, -1, meta_fp16, codes, meta)
        return codes, meta

    return (lambda x, bits, group: _q(x, bits, False)), (lambda x, bits, group: _q(x, bits, True))


class BatchedQuantizer:
    """quantize_k / quantize_v / assemble callables in the form synth.materialize expects, with the
    chunks of a request quantised by ONE kvb_quantize_chunks call: the quantise callables only allot
    the outputs and note the job, the assemble callable (which materialize calls once per request,
    after all its chunks) runs the batch before it stitches."""

    def __init__(self, ctx, sh, meta_fp16: bool = False):
        self.ctx, self.sh, self.meta_fp16, self.jobs = ctx, sh, meta_fp16, []
        self._stitch = assemble_fn(ctx)

    def _note(self, x: torch.Tensor, bits: int, is_value: bool):
        sh = self.sh
        mt = torch.float16 if self.meta_fp16 else torch.float32
        L, Cn, H, d = x.shape
        x = x.contiguous()
        codes = torch.empty((L, Cn, H, d * bits // 8), dtype=torch.uint8, device=x.device)
        if is_value:
            meta = torch.empty((L, Cn, H, 1 if bits == 8 else d // sh.int4_group, 2), dtype=mt, device=x.device)
            job = dict(v=x, v_codes=codes, v_meta=meta)
            if self.jobs and "v" not in self.jobs[-1] and self.jobs[-1]["bits"] == bits:
                self.jobs[-1].update(job)  # the values of the chunk whose keys were just noted: one job
            else:
                self.jobs.append(dict(job, bits=bits, meta_fp16=self.meta_fp16))
        else:
            meta = torch.empty((L, 1 if bits == 8 else Cn // sh.int4_group, H, d, 2), dtype=mt, device=x.device)
            self.jobs.append(dict(k=x, k_codes=codes, k_meta=meta, bits=bits, meta_fp16=self.meta_fp16))
        return codes, meta

    def quantize_k(self, x, bits, group):
        return self._note(x, bits, False)

    def quantize_v(self, x, bits, group):
        return self._note(x, bits, True)

    def flush(self):
        if self.jobs:
            kvb_quantize_chunks(self.ctx, self.jobs)
            kvb_last_status(self.ctx)
            self.jobs = []

    def assemble(self, sh, plan, chunks, fresh):
        self.flush()
        return self._stitch(sh, plan, chunks, fresh)


def assemble_fn(ctx):
    """assemble callable in the form synth.materialize expects, running the CUDA stitching kernel."""

    def _a(sh, plan, chunks, fresh):
        class _R:
            pass

        r = _R()
        r.plan, r.chunks, r.fresh = plan, chunks, fresh
        r.kv_buf = torch.zeros_like(fresh)
        kvb_assemble(ctx, RequestTable([r]))
        kvb_last_status(ctx)
        return r.kv_buf

    return _a
