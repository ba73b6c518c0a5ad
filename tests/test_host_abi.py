"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host-side table validation rejects malformed chunk tables before any launch."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2608_21362_b200 import binding as B
from paper_2608_21362_b200 import synth
from paper_2608_21362_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "kvb.h")).read()
    names = sorted(set(re.findall(r"^(?:int|int64_t|const char\*)\s+(kvb_[a-z_0-9]+)\(", hdr, re.M)))
    assert {"kvb_create", "kvb_destroy", "kvb_assemble", "kvb_deviation_topk", "kvb_selective_attn"} <= set(names)
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), n
        assert hasattr(B, n), "python binding lacks %s" % n


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(B.kvb_chunk) == 64 + 6 * 4 + 4 * 8
    assert C.sizeof(B.kvb_request) == 8 + 4 * 8
    assert C.sizeof(B.kvb_model_desc) == 8 * 4 + 8
    assert C.sizeof(B.kvb_selection) == 4 * 8 + 8


def test_select_count_and_status_strings():
    assert [B.kvb_select_count(T, 0.15) for T in (512, 2048, 8192, 16384)] == [76, 307, 1228, 2457]
    assert B.kvb_select_count(100, 1.0) == 100 and B.kvb_select_count(100, 0.0) == 0 and B.kvb_select_count(0, 0.5) == 0
    assert B.kvb_status_string(B.KVB_OK) == "ok" and "table" in B.kvb_status_string(B.KVB_ERR_BAD_TABLE)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU error path")
def test_create_without_gpu_fails_loudly():
    ctx, st = B.kvb_create(0, 36, 16, 2, 128, 128, 1e6, B.KVB_DT_BF16, 32, 4, 64, 8192, check=False)
    assert ctx is None and st == B.KVB_ERR_NO_DEVICE
    with pytest.raises(B.KvbError):
        B.kvb_create(0, 36, 16, 2, 128, 128, 1e6, B.KVB_DT_BF16, 32, 4, 64, 8192)


# ---------------------------------------------------------------- host-side fault injection on tables
class _FakeTensor:
    def __init__(self, ptr):
        self._p = ptr

    def data_ptr(self):
        return self._p


def _table(n_chunks=4, modes=None, mutate=None):
    modes = modes or [B.KVB_MODE_INT8] * n_chunks

    class R:
        pass

    r = R()
    r.plan = synth.RequestPlan(n_chunks * 128, [])
    r.chunks = []
    for i, m in enumerate(modes):
        ck = synth.Chunk(synth.ChunkPlan(i * 128, 4096 + i * 128, m, B.KVB_MATCH_APPROX if m else B.KVB_MATCH_MISS))
        if m != B.KVB_MODE_FRESH:
            ck.k_codes, ck.v_codes = _FakeTensor(0x10000 + 0x100 * i), _FakeTensor(0x20000 + 0x100 * i)
            if m != B.KVB_MODE_FP16:
                ck.k_meta, ck.v_meta = _FakeTensor(0x30000 + 0x100 * i), _FakeTensor(0x40000 + 0x100 * i)
        r.chunks.append(ck)
    r.kv_buf, r.fresh = _FakeTensor(0x100000), _FakeTensor(0x200000)
    if mutate:
        mutate(r)
    return B.RequestTable([r])


MODEL = B.kvb_model_desc(36, 16, 2, 128, 128, B.KVB_DT_BF16, 32, 0, 1e6)
LIMITS = B.kvb_limits(4, 64, 8192)


def _st(table, need_payload=True, limits=LIMITS):
    return B.kvb_validate(MODEL, limits, table, need_payload)


def test_valid_tables_pass():
    assert _st(_table())[0] == B.KVB_OK
    assert _st(_table(modes=[0, 1, 2, 3]))[0] == B.KVB_OK
    assert _st(None)[0] == B.KVB_OK  # empty batch


def test_gap_overlap_and_order_are_rejected():
    def gap(r):
        r.chunks[2].plan.new_pos = 3 * 128

    def overlap(r):
        r.chunks[1].plan.new_pos = 0

    def swapped(r):
        r.chunks[0], r.chunks[1] = r.chunks[1], r.chunks[0]

    for mut in (gap, overlap, swapped):
        st, msg = _st(_table(mutate=mut))
        assert st == B.KVB_ERR_BAD_TABLE and "gap or overlap" in msg

    def short(r):
        r.plan.T = 3 * 128

    assert _st(_table(mutate=short))[0] == B.KVB_ERR_BAD_TABLE


def test_bad_enums_positions_and_pointers_are_rejected():
    def bad_mode(r):
        r.chunks[1].plan.mode = 7

    def bad_match(r):
        r.chunks[1].plan.match = -1

    assert _st(_table(mutate=bad_mode))[0] == B.KVB_ERR_INVALID_ARG
    assert _st(_table(mutate=bad_match))[0] == B.KVB_ERR_INVALID_ARG

    def neg_pos(r):
        r.chunks[1].plan.orig_pos = -5

    def huge_pos(r):
        r.chunks[1].plan.orig_pos = 1 << 24

    def exact_moved(r):
        r.chunks[1].plan.match = B.KVB_MATCH_EXACT

    for mut in (neg_pos, huge_pos, exact_moved):
        assert _st(_table(mutate=mut))[0] == B.KVB_ERR_BAD_TABLE

    def exact_in_place(r):
        r.chunks[1].plan.match = B.KVB_MATCH_EXACT
        r.chunks[1].plan.orig_pos = r.chunks[1].plan.new_pos

    assert _st(_table(mutate=exact_in_place))[0] == B.KVB_OK

    def misaligned(r):
        r.chunks[2].k_codes = _FakeTensor(0x10008)

    def misaligned_buf(r):
        r.kv_buf = _FakeTensor(0x100004)

    def null_meta(r):
        r.chunks[2].v_meta = None

    assert _st(_table(mutate=misaligned))[0] == B.KVB_ERR_BAD_TABLE
    assert _st(_table(mutate=misaligned_buf))[0] == B.KVB_ERR_BAD_TABLE
    assert _st(_table(mutate=null_meta))[0] == B.KVB_ERR_INVALID_ARG
    assert _st(_table(mutate=null_meta), need_payload=False)[0] == B.KVB_OK  # selection calls do not need payloads


def test_limits_are_enforced():
    assert _st(_table(), limits=B.kvb_limits(4, 3, 8192))[0] == B.KVB_ERR_WORKSPACE
    assert _st(_table(), limits=B.kvb_limits(4, 64, 511))[0] == B.KVB_ERR_WORKSPACE
    assert _st(_table(), limits=B.kvb_limits(0, 64, 8192))[0] == B.KVB_ERR_WORKSPACE


def test_wrong_chunk_size_is_rejected():
    t = _table()
    t.array[0].chunks[1].n_tokens = 64
    assert _st(t)[0] == B.KVB_ERR_BAD_TABLE


# ---------------------------------------------------------------- property: the validator against a restatement of its rules
def _expected_status(T, chunks, kv_ptr, fresh_ptr, need_payload):
    """The header's table rules, written out again: first failing rule wins, in the order the library checks."""
    C_ = 128
    if T <= 0 or len(chunks) == 0:
        return B.KVB_ERR_INVALID_ARG
    if T % C_ != 0 or len(chunks) != T // C_:
        return B.KVB_ERR_BAD_TABLE
    if kv_ptr == 0 or fresh_ptr == 0:
        return B.KVB_ERR_INVALID_ARG
    if kv_ptr % 16 or fresh_ptr % 16:
        return B.KVB_ERR_BAD_TABLE
    for i, c in enumerate(chunks):
        if c["n_tokens"] != C_ or c["new_pos"] != i * C_:
            return B.KVB_ERR_BAD_TABLE
        if not 0 <= c["mode"] <= 3:
            return B.KVB_ERR_INVALID_ARG
        if c["meta_fp16"] not in (0, 1):
            return B.KVB_ERR_INVALID_ARG
        if not 0 <= c["match"] <= 2:
            return B.KVB_ERR_INVALID_ARG
        if c["mode"] == 0:
            continue
        if c["orig_pos"] < 0 or c["orig_pos"] >= 1 << 24 or c["new_pos"] >= 1 << 24:
            return B.KVB_ERR_BAD_TABLE
        if c["match"] == 1 and c["orig_pos"] != c["new_pos"]:
            return B.KVB_ERR_BAD_TABLE
        if not need_payload:
            continue
        if c["k_codes"] == 0 or c["v_codes"] == 0:
            return B.KVB_ERR_INVALID_ARG
        if c["k_codes"] % 16 or c["v_codes"] % 16:
            return B.KVB_ERR_BAD_TABLE
        if c["mode"] != 1:
            if c["k_meta"] == 0 or c["v_meta"] == 0:
                return B.KVB_ERR_INVALID_ARG
            if c["k_meta"] % 16 or c["v_meta"] % 16:
                return B.KVB_ERR_BAD_TABLE
    return B.KVB_OK


def test_validator_agrees_with_the_stated_rules_on_random_tables():
    hypothesis = pytest.importorskip("hypothesis")
    from hypothesis import given, settings
    from hypothesis import strategies as st

    ptr = st.sampled_from([0, 0x1000, 0x1008, 0x2010, 0x7F00])
    chunk = st.fixed_dictionaries({
        "mode": st.sampled_from([0, 1, 2, 3, 3, 2, 4, -1]),
        "match": st.sampled_from([0, 1, 2, 2, 2, 3]),
        "meta_fp16": st.sampled_from([0, 0, 0, 1, 2]),
        "n_tokens": st.sampled_from([128, 128, 128, 128, 64]),
        "orig_pos": st.sampled_from([0, 128, 4096, (1 << 24) - 128, 1 << 24, -5]),
        "pos_fault": st.sampled_from([0, 0, 0, 0, 0, 128, -128]),
        "k_codes": ptr, "v_codes": ptr, "k_meta": ptr, "v_meta": ptr,
    })

    @settings(max_examples=300, deadline=None)
    @given(st.lists(chunk, min_size=0, max_size=5), st.sampled_from([0, 0, 0, 128, -128, 64]), ptr, ptr, st.booleans())
    def run(chunks, t_fault, kv_ptr, fresh_ptr, need_payload):
        for i, c in enumerate(chunks):
            c["new_pos"] = i * 128 + c["pos_fault"]
        T = len(chunks) * 128 + t_fault
        arr = (B.kvb_chunk * max(1, len(chunks)))()
        for i, c in enumerate(chunks):
            for name in ("orig_pos", "new_pos", "n_tokens", "mode", "match", "meta_fp16"):
                setattr(arr[i], name, c[name])
            for name in ("k_codes", "v_codes", "k_meta", "v_meta"):
                setattr(arr[i], name, c[name] or None)
        req = (B.kvb_request * 1)()
        req[0].T, req[0].n_chunks, req[0].chunks = T, len(chunks), arr
        req[0].kv_buf, req[0].fresh = kv_ptr or None, fresh_ptr or None
        buf = C.create_string_buffer(512)
        got = B.lib().kvb_validate(C.byref(MODEL), C.byref(LIMITS), req, 1, int(need_payload), buf, 512)
        assert got == _expected_status(T, chunks, kv_ptr, fresh_ptr, need_payload), (buf.value, T, chunks)

    run()
