"""Pins for the CPU oracle: each check ties an oracle function to something other than
itself -- a closed form, an invariant the paper states, brute force in pure Python, or a
library routine (numpy / torch CPU) -- chosen so a dropped term, wrong sign, wrong index
or transposed operand fails at least one of them."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ------------------------------------------------------------------ storage formats
def test_fp16_rounding_matches_numpy():
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.uniform(-9, 5, 20000), [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e-8, 2.98e-8, 2.9802322e-8]])
    got = oracle.round_to_bits(x, oracle.DT_F16)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)  # numpy rounds float64 -> float16 directly, ties to even
    assert np.array_equal(got, want)
    back = oracle.bits_to_f64(got, oracle.DT_F16)
    assert np.array_equal(back[np.isfinite(back)], want.view(np.float16).astype(np.float64)[np.isfinite(back)])


def test_bf16_rounding_matches_torch_on_float32_inputs():
    # from float32 inputs there is a single rounding on both sides
    x = (rng.standard_normal(50000) * 10.0 ** rng.uniform(-30, 30, 50000)).astype(np.float32)
    got = oracle.round_to_bits(x.astype(np.float64), oracle.DT_BF16)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    back = oracle.bits_to_f64(got, oracle.DT_BF16)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy())


def test_bf16_ties_to_even_and_single_rounding():
    one = 1.0
    ulp = 2.0**-7
    assert oracle.bits_to_f64(oracle.round_to_bits([one + ulp / 2], 1), 1)[0] == one  # tie -> even (1.0)
    assert oracle.bits_to_f64(oracle.round_to_bits([one + 3 * ulp / 2], 1), 1)[0] == one + 2 * ulp  # tie -> even
    # just above a tie: a float32 detour would first round down onto the tie, then to even (wrong)
    x = one + ulp / 2 + 2.0**-40
    assert oracle.bits_to_f64(oracle.round_to_bits([x], 1), 1)[0] == one + ulp


# ------------------------------------------------------------------ Eq. 6
@pytest.mark.parametrize("bits,gk,gv", [(8, 128, 128), (4, 32, 32)])
def test_quant_roundtrip_within_half_step(bits, gk, gv):
    C, H, d = 128, 2, 128
    c = np.exp(rng.uniform(math.log(0.1), math.log(10), (1, H, d)))
    k = oracle.bits_to_f64(oracle.round_to_bits(rng.standard_normal((C, H, d)) * c, 1), 1)
    v = oracle.bits_to_f64(oracle.round_to_bits(rng.standard_normal((C, H, d)), 1), 1)
    kc, km = oracle.quantize_k(k, bits, gk)
    vc, vm = oracle.quantize_v(v, bits, gv)
    assert kc.shape == (C, H, d * bits // 8) and km.shape == (C // gk, H, d, 2)
    assert vc.shape == (C, H, d * bits // 8) and vm.shape == (C, H, d // gv, 2)
    kd = oracle.dequant_k(kc, km, d, bits, gk)
    vd = oracle.dequant_v(vc, vm, d, bits, gv)
    ks = np.repeat(km[..., 0], gk, axis=0).astype(np.float64)  # [C,H,d] step of each element's group
    vs = np.repeat(vm[..., 0], gv, axis=2).astype(np.float64)
    assert np.all(np.abs(kd - k) <= 0.5 * ks * (1 + 1e-4) + 1e-30)
    assert np.all(np.abs(vd - v) <= 0.5 * vs * (1 + 1e-4) + 1e-30)
    # the step is (max-min)/(2^b-1) of the group, min is the group's minimum
    kg = k.reshape(C // gk, gk, H, d)
    assert np.allclose(km[..., 1], kg.min(1), rtol=0, atol=0)
    assert np.allclose(km[..., 0], (kg.max(1) - kg.min(1)) / (2**bits - 1), rtol=1e-6)
    vg = v.reshape(C, H, d // gv, gv)
    assert np.array_equal(vm[..., 1], vg.min(-1).astype(np.float32))
    assert np.allclose(vm[..., 0], (vg.max(-1) - vg.min(-1)) / (2**bits - 1), rtol=1e-6)
    # group extremes hit the end codes exactly
    assert kd.reshape(kg.shape).min(1) == pytest.approx(kg.min(1), abs=0)


def test_quant_bruteforce_tiny_and_nibble_order():
    # pure-Python restatement of Eq. 6 on a 4-token, 1-head, 4-channel chunk, int4, one group
    x = np.array([[[0.0, 1.0, -2.0, 5.0]], [[1.4, 1.0, 2.0, 5.0]], [[3.0, 1.0, 0.1, 5.0]], [[0.35, 1.0, 1.0, 5.0]]])
    codes, meta = oracle.quantize_k(x, 4, 4)
    want = np.zeros((4, 4), int)
    for j in range(4):
        col = [x[t, 0, j] for t in range(4)]
        mn, mx = min(col), max(col)
        s = (mx - mn) / 15 if mx > mn else 1.0
        assert meta[0, 0, j, 1] == np.float32(mn)
        assert meta[0, 0, j, 0] == pytest.approx(s, rel=1e-6)
        for t in range(4):
            want[t, j] = min(15, max(0, round((col[t] - mn) / s)))
    # values chosen away from rounding ties
    for t in range(4):
        assert codes[t, 0, 0] == (want[t, 0] | (want[t, 1] << 4))  # even channel -> low nibble
        assert codes[t, 0, 1] == (want[t, 2] | (want[t, 3] << 4))
    # constant channels (max == min): scale 1, code 0, dequantises to the constant exactly
    assert meta[0, 0, 1, 0] == 1.0 and meta[0, 0, 3, 0] == 1.0
    d = oracle.dequant_k(codes, meta, 4, 4, 4)
    assert np.all(d[:, 0, 1] == 1.0) and np.all(d[:, 0, 3] == 5.0)


def test_quant_payload_sizes():
    # "int8 ~ 2x, int4 ~ 4x" smaller than 16-bit storage: exact for the code payload
    x = rng.standard_normal((128, 2, 128))
    fp16_bytes = x.size * 2
    assert oracle.quantize_k(x, 8, 128)[0].nbytes * 2 == fp16_bytes
    assert oracle.quantize_k(x, 4, 32)[0].nbytes * 4 == fp16_bytes
    assert oracle.quantize_v(x, 8, 128)[0].nbytes * 2 == fp16_bytes
    assert oracle.quantize_v(x, 4, 32)[0].nbytes * 4 == fp16_bytes


def test_dequant_is_affine_in_code():
    # hand-made codes and metadata: x^ = q*s + m, keys per channel, values per token
    C, H, d = 2, 1, 4
    codes = np.array([[[0, 255, 10, 3]], [[1, 2, 3, 4]]], np.uint8)
    km = np.zeros((1, H, d, 2), np.float32)
    km[0, 0, :, 0] = [0.5, 0.25, 2.0, 1.0]
    km[0, 0, :, 1] = [-1.0, 0.0, 3.0, -4.0]
    out = oracle.dequant_k(codes, km, d, 8, 2)
    assert np.array_equal(out[0, 0], [-1.0, 63.75, 23.0, -1.0])
    assert np.array_equal(out[1, 0], [-0.5, 0.5, 9.0, 0.0])
    vm = np.zeros((C, H, 1, 2), np.float32)
    vm[0, 0, 0] = [2.0, 1.0]
    vm[1, 0, 0] = [0.5, -1.0]
    out = oracle.dequant_v(codes, vm, d, 8, 4)
    assert np.array_equal(out[0, 0], [1.0, 511.0, 21.0, 7.0])
    assert np.array_equal(out[1, 0], [-0.5, 0.0, 0.5, 1.0])


# ------------------------------------------------------------------ Eq. 3
def _rot_matrix(d, theta, delta):
    """Textbook block rotation: plane (j, j+d/2) turned by delta*theta^(-2j/d)."""
    R = np.zeros((d, d))
    for j in range(d // 2):
        a = delta * theta ** (-2.0 * j / d)
        R[j, j] = math.cos(a)
        R[j, j + d // 2] = -math.sin(a)
        R[j + d // 2, j] = math.sin(a)
        R[j + d // 2, j + d // 2] = math.cos(a)
    return R


def test_rope_matches_rotation_matrix_and_hf_formula():
    d, theta = 128, 1e6
    x = rng.standard_normal((5, 2, d))
    for delta in (1.0, -37.0, 4095.0):
        got = oracle.rope_rotate(x, theta, delta)
        want = x @ _rot_matrix(d, theta, delta).T
        assert np.allclose(got, want, rtol=0, atol=1e-12)
        # the x*cos + rotate_half(x)*sin form used by HF-style implementations
        inv = theta ** (-np.arange(0, d, 2) / d)
        ang = np.concatenate([delta * inv, delta * inv])
        rh = np.concatenate([-x[..., d // 2 :], x[..., : d // 2]], -1)
        assert np.allclose(got, x * np.cos(ang) + rh * np.sin(ang), rtol=0, atol=1e-12)


def test_rope_one_plane_known_values():
    # d = 2: one plane with frequency 1, so delta is the angle in radians
    got = oracle.rope_rotate(np.array([[[1.0, 0.0]]]), 10000.0, math.pi / 2)
    assert np.allclose(got, [[[0.0, 1.0]]], atol=1e-15)
    got = oracle.rope_rotate(np.array([[[0.0, 1.0]]]), 10000.0, math.pi / 2)
    assert np.allclose(got, [[[-1.0, 0.0]]], atol=1e-15)
    got = oracle.rope_rotate(np.array([[[2.0, 3.0]]]), 10000.0, 1.0)
    assert np.allclose(got, [[[2 * math.cos(1) - 3 * math.sin(1), 3 * math.cos(1) + 2 * math.sin(1)]]], atol=1e-15)


def test_rope_group_property_and_rerotation():
    d, theta = 128, 1e6
    raw = rng.standard_normal((3, 2, d))
    for a, b in [(50, 1000), (32767, -32767), (123, 4096 - 123), (1050, -1000)]:
        ab = oracle.rope_rotate(oracle.rope_rotate(raw, theta, a), theta, b)
        assert np.allclose(ab, oracle.rope_rotate(raw, theta, a + b), rtol=0, atol=2e-11)
    # a key cached at p and corrected by q - p equals the raw key rotated at q
    p, q = 50, 1050
    assert np.allclose(oracle.rope_rotate(oracle.rope_rotate(raw, theta, p), theta, q - p), oracle.rope_rotate(raw, theta, q), atol=2e-11)
    # delta = 0 is the identity, bit for bit; rotation preserves each head's norm
    assert np.array_equal(oracle.rope_rotate(raw, theta, 0), raw)
    assert np.allclose(np.linalg.norm(oracle.rope_rotate(raw, theta, 777), axis=-1), np.linalg.norm(raw, axis=-1), rtol=1e-13)


def test_rope_inner_product_depends_on_offset_only():
    d, theta = 128, 1e6
    qv = rng.standard_normal((1, 1, d))
    kv = rng.standard_normal((1, 1, d))

    def dot(s, t):
        return float(np.sum(oracle.rope_rotate(qv, theta, s) * oracle.rope_rotate(kv, theta, t)))

    assert dot(1000, 50) == pytest.approx(dot(1000 + 4321, 50 + 4321), abs=1e-10)
    # q_s . k_t = q^T R^{t-s} k
    assert dot(7, 19) == pytest.approx(float(np.sum(qv * oracle.rope_rotate(kv, theta, 12))), abs=1e-10)
    assert abs(dot(7, 19) - dot(7, 20)) > 1e-3  # and it does depend on the offset


# ------------------------------------------------------------------ prompt assembly
def _tiny_assemble_case(dtype=oracle.DT_BF16):
    L, H, d, C, T, theta = 2, 2, 8, 4, 12, 1e4
    r = np.random.default_rng(5)
    fresh = oracle.round_to_bits(r.standard_normal((L, 2, T, H, d)), dtype)
    chunks = []
    kraw = oracle.bits_to_f64(oracle.round_to_bits(r.standard_normal((L, C, H, d)) * 3, dtype), dtype)
    vraw = oracle.bits_to_f64(oracle.round_to_bits(r.standard_normal((L, C, H, d)), dtype), dtype)
    kq = [oracle.quantize_k(kraw[l], 8, C) for l in range(L)]
    vq = [oracle.quantize_v(vraw[l], 8, d) for l in range(L)]
    chunks.append(dict(orig_pos=40, new_pos=8, n_tokens=C, mode=oracle.MODE_INT8, k_codes=np.stack([a for a, _ in kq]), k_meta=np.stack([b for _, b in kq]), v_codes=np.stack([a for a, _ in vq]), v_meta=np.stack([b for _, b in vq])))
    chunks.append(dict(orig_pos=0, new_pos=0, n_tokens=C, mode=oracle.MODE_FRESH))
    chunks.append(dict(orig_pos=3, new_pos=4, n_tokens=C, mode=oracle.MODE_FP16, k_codes=oracle.round_to_bits(kraw, dtype), v_codes=oracle.round_to_bits(vraw, dtype)))
    return L, H, d, C, T, theta, fresh, chunks, kraw, vraw, kq, vq


@pytest.mark.parametrize("dtype", [oracle.DT_BF16, oracle.DT_F16])
def test_assemble_rows_land_in_prompt_order(dtype):
    L, H, d, C, T, theta, fresh, chunks, kraw, vraw, kq, vq = _tiny_assemble_case(dtype)
    kv, exact = oracle.assemble(chunks, L, H, d, T, theta, dtype, 2, fresh, want_exact=True)
    # FRESH rows are bit copies of the caller's fresh rows
    assert np.array_equal(kv[:, :, 0:4], fresh[:, :, 0:4])
    for l in range(L):
        # values: dequantised only (never rotated), written at rows new_pos..
        vd = oracle.dequant_v(vq[l][0], vq[l][1], d, 8, d)
        assert np.array_equal(exact[l, 1, 8:12], vd)
        assert np.array_equal(kv[l, 1, 8:12], oracle.round_to_bits(vd, dtype))
        # keys: dequantised, then turned by new_pos - orig_pos = -32
        kd = oracle.dequant_k(kq[l][0], kq[l][1], d, 8, C)
        assert np.allclose(exact[l, 0, 8:12], kd @ _rot_matrix(d, theta, -32.0).T, atol=1e-12)
        # unquantised cached chunk: keys turned by +1, values copied
        assert np.array_equal(kv[l, 1, 4:8], oracle.round_to_bits(vraw[l], dtype))
        assert np.allclose(exact[l, 0, 4:8], kraw[l] @ _rot_matrix(d, theta, 1.0).T, atol=1e-12)
    assert np.array_equal(kv, oracle.round_to_bits(exact, dtype))


def test_assemble_exact_match_is_pure_dequant_and_uncovered_rows_untouched():
    L, H, d, C, T, theta, fresh, chunks, kraw, vraw, kq, vq = _tiny_assemble_case()
    only = [dict(chunks[0], orig_pos=8, new_pos=8)]  # same position: rotation is the identity
    kv, exact = oracle.assemble(only, L, H, d, T, theta, oracle.DT_BF16, 2, fresh, want_exact=True)
    for l in range(L):
        assert np.array_equal(exact[l, 0, 8:12], oracle.dequant_k(kq[l][0], kq[l][1], d, 8, C))
    assert not kv[:, :, 0:8].any()


# ------------------------------------------------------------------ Algorithm 2 step 2
def _rand_bits(shape, dtype, scale=1.0, r=rng):
    return oracle.round_to_bits(r.standard_normal(shape) * scale, dtype)


def test_deviation_matches_library_cosine():
    L, T, H, d = 3, 17, 2, 16
    a = _rand_bits((L, 2, T, H, d), 1)
    b = _rand_bits((L, 2, T, H, d), 1)
    A = torch.from_numpy(oracle.bits_to_f64(a, 1))
    B = torch.from_numpy(oracle.bits_to_f64(b, 1))
    cos = torch.nn.functional.cosine_similarity(A, B, dim=-1, eps=0.0)  # [L,2,T,H]
    for which, sl in ((1, slice(0, 1)), (2, slice(1, 2)), (3, slice(0, 2))):
        d64, d32 = oracle.deviation(a, b, 1, which)
        want = 1.0 - cos[:, sl].mean(dim=(0, 1, 3)).numpy()
        assert np.allclose(d64, want, rtol=0, atol=1e-14)
        assert np.array_equal(d32, d64.astype(np.float32))


def test_deviation_invariants():
    L, T, H, d = 2, 9, 2, 32
    a = _rand_bits((L, 2, T, H, d), 1)
    assert np.all(oracle.deviation(a, a, 1, 3)[0] == 0.0)  # identical K/V -> exactly 0
    # scale invariance (powers of two are exact in bf16)
    b = _rand_bits((L, 2, T, H, d), 1)
    a4 = oracle.round_to_bits(oracle.bits_to_f64(a, 1) * 4.0, 1)
    b8 = oracle.round_to_bits(oracle.bits_to_f64(b, 1) * 0.125, 1)
    assert np.allclose(oracle.deviation(a4, b8, 1, 1)[0], oracle.deviation(a, b, 1, 1)[0], atol=1e-15)
    # opposite vectors -> 2, range [0, 2]
    neg = oracle.round_to_bits(-oracle.bits_to_f64(a, 1), 1)
    assert np.allclose(oracle.deviation(a, neg, 1, 3)[0], 2.0, atol=1e-15)
    # K+V with identical V is half the K-only deviation
    mixed = b.copy()
    mixed[:, 1] = a[:, 1]
    assert np.allclose(oracle.deviation(a, mixed, 1, 3)[0], 0.5 * oracle.deviation(a, b, 1, 1)[0], atol=1e-15)


def test_deviation_orthogonal_and_degenerate_vectors():
    L, T, H, d = 1, 3, 1, 4
    a = np.zeros((L, 2, T, H, d))
    b = np.zeros((L, 2, T, H, d))
    a[0, 0, 0, 0] = [1, 0, 0, 0]
    b[0, 0, 0, 0] = [0, 2, 0, 0]  # orthogonal -> cos 0 -> delta 1
    a[0, 0, 1, 0] = [0, 0, 0, 0]
    b[0, 0, 1, 0] = [0, 0, 0, 0]  # both zero and equal -> cos 1 -> delta 0
    a[0, 0, 2, 0] = [0, 0, 0, 0]
    b[0, 0, 2, 0] = [1, 1, 0, 0]  # one zero norm, not equal -> cos 0 -> delta 1
    d64, _ = oracle.deviation(oracle.round_to_bits(a, 1), oracle.round_to_bits(b, 1), 1, 1)
    assert np.array_equal(d64, [1.0, 0.0, 1.0])
    # 45 degrees
    a[0, 0, 0, 0] = [1, 0, 0, 0]
    b[0, 0, 0, 0] = [1, 1, 0, 0]
    d64, _ = oracle.deviation(oracle.round_to_bits(a, 1), oracle.round_to_bits(b, 1), 1, 1)
    assert d64[0] == pytest.approx(1 - 1 / math.sqrt(2), abs=1e-15)


# ------------------------------------------------------------------ Algorithm 2 step 3 / Algorithm 1
def test_select_count_is_floor():
    assert [oracle.select_count(T, 0.15) for T in (512, 2048, 8192, 16384)] == [76, 307, 1228, 2457]
    assert oracle.select_count(100, 0.25) == 25 and oracle.select_count(7, 0.15) == 1 and oracle.select_count(6, 0.15) == 0


def test_topk_matches_library_sort():
    for T in (1, 2, 77, 1000):
        dl = rng.random(T).astype(np.float32)
        dl[rng.integers(0, T, T // 3)] = np.float32(0.5)  # many exact ties
        for k in (0, 1, T // 7, T):
            got = oracle.topk(dl, k)
            want = np.lexsort((np.arange(T), -dl.astype(np.float64)))[:k]  # by delta desc, then index asc
            assert np.array_equal(got, want)
    dl = rng.random(300).astype(np.float32)  # distinct values: torch.topk is unambiguous
    assert np.array_equal(oracle.topk(dl, 40), torch.topk(torch.from_numpy(dl), 40).indices.numpy())


def test_topk_bruteforce_and_plateaus():
    dl = np.array([0.1, 0.3, 0.3, 0.0, -0.0, 0.3, 0.2], np.float32)
    # pure-Python selection: repeatedly take the max, lowest index first
    left = list(range(len(dl)))
    want = []
    for _ in range(5):
        best = max(left, key=lambda i: (float(dl[i]), -i))
        want.append(best)
        left.remove(best)
    assert list(oracle.topk(dl, 5)) == want == [1, 2, 5, 6, 0]
    assert list(oracle.topk(dl, 7)) == [1, 2, 5, 6, 0, 3, 4]  # -0 ties with +0, index decides
    assert list(oracle.topk(np.zeros(6, np.float32), 4)) == [0, 1, 2, 3]  # all equal -> lowest indices
    assert list(oracle.topk(np.array([0.1, np.nan, 0.7], np.float32), 2)) == [1, 2]  # NaN ranks first


def test_seam_windows_closed_form():
    T, C = 1024, 128
    pos = np.arange(0, T, C)
    mode = np.array([2, 2, 0, 0, 2, 0, 3, 1])  # seams at every boundary except between chunks 2|3 (both fresh)
    none = np.zeros(0, np.int32)
    sel = oracle.seam_select(none, pos, mode, T, 16, 0)
    want = sorted(t for c in (1, 2, 4, 5, 6, 7) for t in range(c * C - 16, c * C))
    assert list(sel) == want and len(sel) == 6 * 16  # O(R * N_seams) tokens
    sel = oracle.seam_select(none, pos, mode, T, 0, 16)
    assert list(sel) == sorted(t for c in (1, 2, 4, 5, 6, 7) for t in range(c * C, c * C + 16))
    # clamping at 0 and T, and union with the top-k set without duplicates
    sel = oracle.seam_select(np.array([5, 11, 7], np.int32), np.array([0, 8]), np.array([2, 2]), 12, 16, 16)
    assert list(sel) == list(range(12))
    sel = oracle.seam_select(np.array([300, 120, 5], np.int32), pos, mode, T, 16, 0)
    assert list(sel) == sorted(set(want) | {300, 120, 5}) and len(sel) == 6 * 16 + 2


def test_sink_tokens_are_always_selected():
    T, C = 512, 128
    pos, mode = np.arange(0, T, C), np.array([0, 0, 2, 2])  # seams at 256 and 384 only
    none = np.zeros(0, np.int32)
    assert list(oracle.seam_select(none, pos, mode, T, 0, 0, sinks=4)) == [0, 1, 2, 3]
    sel = oracle.seam_select(np.array([2, 300], np.int32), pos, mode, T, 16, 0, sinks=4)
    assert list(sel) == sorted({0, 1, 2, 3, 300} | set(range(240, 256)) | set(range(368, 384)))
    assert list(oracle.seam_select(none, pos, mode, T, 0, 0, sinks=10**6)) == list(range(T))  # clamped at T
    assert list(oracle.seam_select(none, pos, mode, T, 0, 0)) == []


# ------------------------------------------------------------------ Eq. 2
def _attn_case(L=2, T=24, Hq=4, Hkv=2, d=16, dtype=1, seed=9):
    r = np.random.default_rng(seed)
    kv = _rand_bits((L, 2, T, Hkv, d), dtype, r=r)
    q = _rand_bits((L, T, Hq, d), dtype, 0.5, r=r)
    return kv, q


def test_attention_all_rows_equals_library_causal_sdpa():
    L, T, Hq, Hkv, d = 2, 24, 4, 2, 16
    kv, q = _attn_case(L, T, Hq, Hkv, d)
    sel = np.arange(T, dtype=np.int32)
    scale = 1 / math.sqrt(d)
    out, exact = oracle.attention(q, kv, sel, Hq, 1, scale, want_exact=True)
    Q = torch.from_numpy(oracle.bits_to_f64(q, 1)).permute(0, 2, 1, 3)  # [L,Hq,T,d]
    K = torch.from_numpy(oracle.bits_to_f64(kv[:, 0], 1)).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    V = torch.from_numpy(oracle.bits_to_f64(kv[:, 1], 1)).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    want = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True, scale=scale).permute(0, 2, 1, 3).numpy()
    assert np.allclose(exact, want, rtol=0, atol=1e-13)
    assert np.array_equal(out, oracle.round_to_bits(exact, 1))


def test_attention_selected_rows_and_sampling():
    L, T, Hq, Hkv, d = 2, 24, 4, 2, 16
    kv, q_full = _attn_case(L, T, Hq, Hkv, d)
    full = oracle.attention(q_full, kv, np.arange(T, dtype=np.int32), Hq, 1, 0.25, want_exact=True)[1]
    sel = np.array([0, 3, 4, 17, 23], np.int32)
    cap = 8
    q = np.zeros((L, cap, Hq, d), np.uint16)
    q[:, : len(sel)] = q_full[:, sel]
    out, exact = oracle.attention(q, kv, sel, Hq, 1, 0.25, want_exact=True)
    assert np.array_equal(exact[:, : len(sel)], full[:, sel])  # row i is position sel[i], keys 0..sel[i]
    assert not out[:, len(sel) :].any()
    part = oracle.attention(q, kv, sel, Hq, 1, 0.25, layers=[1], rows=[2, 4], want_exact=True)[1]
    assert np.array_equal(part[1, [2, 4]], exact[1, [2, 4]]) and not part[0].any() and not part[1, [0, 1, 3]].any()


def test_attention_special_cases():
    L, T, Hq, Hkv, d = 1, 10, 2, 2, 8
    kv, q = _attn_case(L, T, Hq, Hkv, d, seed=3)
    sel = np.arange(T, dtype=np.int32)
    exact = oracle.attention(q, kv, sel, Hq, 1, 1.0, want_exact=True)[1]
    V = oracle.bits_to_f64(kv[:, 1], 1)
    assert np.allclose(exact[0, 0], V[0, 0], atol=1e-15)  # position 0 sees only itself
    # all keys equal -> uniform weights -> running mean of the values
    kv2 = kv.copy()
    kv2[:, 0] = kv[:, 0, :1]
    exact = oracle.attention(q, kv2, sel, Hq, 1, 1.0, want_exact=True)[1]
    for t in range(T):
        assert np.allclose(exact[0, t], V[0, : t + 1].mean(0), atol=1e-14)
    # naive softmax in pure Python for one row and head, GQA head mapping hq -> hq // (Hq/Hkv)
    kv, q = _attn_case(1, 6, 4, 2, 4, seed=11)
    exact = oracle.attention(q, kv, np.arange(6, dtype=np.int32), 4, 1, 0.5, want_exact=True)[1]
    K = oracle.bits_to_f64(kv[0, 0], 1)
    V = oracle.bits_to_f64(kv[0, 1], 1)
    Q = oracle.bits_to_f64(q[0], 1)
    t, hq = 4, 3
    hk = 1
    sc = [0.5 * sum(Q[t, hq, j] * K[s, hk, j] for j in range(4)) for s in range(t + 1)]
    w = [math.exp(v - max(sc)) for v in sc]
    want = [sum(w[s] * V[s, hk, j] for s in range(t + 1)) / sum(w) for j in range(4)]
    assert np.allclose(exact[0, t, hq], want, atol=1e-14)


def test_golden_fixture_rope_worked_example():
    """The paper's own worked example: a key cached at t=50 needs R^{1000} to serve t=1050.
    The fixture holds the angles 1000*theta^(-2j/d) for d=8, theta=1e6, written by
    tests/golden/make_golden.py from the closed form."""
    rows = np.loadtxt(os.path.join(GOLD, "rope_delta1000_d8_theta1e6.txt"))
    d, theta = 8, 1e6
    raw = np.eye(d)[None].transpose(1, 0, 2)  # [d,1,d] unit vectors
    at50 = oracle.rope_rotate(raw, theta, 50)
    fixed = oracle.rope_rotate(at50, theta, 1000)
    assert np.allclose(fixed, oracle.rope_rotate(raw, theta, 1050), atol=1e-11)
    R = oracle.rope_rotate(raw, theta, 1000)[:, 0, :].T  # columns = images of unit vectors
    for j, (ang, c, s) in enumerate(rows):
        assert R[j, j] == pytest.approx(c, abs=1e-12) and R[j + 4, j] == pytest.approx(s, abs=1e-12)
        assert R[j, j + 4] == pytest.approx(-s, abs=1e-12) and R[j + 4, j + 4] == pytest.approx(c, abs=1e-12)


# ------------------------------------------------------------------ Algorithm 2 step 4; Eq. 7
def test_patch_replaces_exactly_the_selected_rows():
    L, T, H, d = 3, 20, 2, 8
    kv = _rand_bits((L, 2, T, H, d), 1)
    fresh = _rand_bits((L, 2, T, H, d), 1)
    sel = np.array([0, 3, 4, 19], np.int32)
    got = oracle.patch(kv, fresh, sel)
    want = kv.copy()
    want[:, :, sel] = fresh[:, :, sel]  # numpy indexed assignment as the plain definition
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.patch(kv, fresh, np.zeros(0, np.int32)), kv)
    # a patched position no longer deviates; the others keep their deviation
    d_before = oracle.deviation(kv, fresh, 1, 3)[0]
    d_after = oracle.deviation(got, fresh, 1, 3)[0]
    assert np.all(d_after[sel] == 0.0)
    rest = np.setdiff1d(np.arange(T), sel)
    assert np.array_equal(d_after[rest], d_before[rest])


def test_importance_is_the_mean_key_norm():
    L, T, H, d, C = 2, 12, 2, 16, 4
    kv = _rand_bits((L, 2, T, H, d), 1)
    K = oracle.bits_to_f64(kv[:, 0], 1)  # [L,T,H,d]
    want = np.linalg.norm(K, axis=-1).reshape(L, T // C, C, H).mean(axis=(0, 2, 3))
    assert np.allclose(oracle.importance(kv, C, 1), want, rtol=0, atol=1e-14)
    # closed forms: all-ones keys have norm sqrt(d); values never matter; scaling is linear
    ones = oracle.round_to_bits(np.ones((L, 2, T, H, d)), 1)
    assert np.allclose(oracle.importance(ones, C, 1), math.sqrt(d), atol=1e-15)
    kv2 = kv.copy()
    kv2[:, 1] = ones[:, 1]
    assert np.array_equal(oracle.importance(kv2, C, 1), oracle.importance(kv, C, 1))
    dbl = oracle.round_to_bits(oracle.bits_to_f64(kv, 1) * 2.0, 1)
    assert np.allclose(oracle.importance(dbl, C, 1), 2 * oracle.importance(kv, C, 1), rtol=1e-15)


# ------------------------------------------------------------------ position-free cache population (rotation by -orig_pos)
def test_unrotate_keys_is_the_inverse_rotation_in_float32():
    theta, H, d = 1e6, 2, 16
    bits = _rand_bits((5, H, d), 1, scale=3.0)
    x = oracle.bits_to_f64(bits, 1)
    assert np.array_equal(oracle.unrotate_keys(bits, 1, theta, 0), x)  # position 0: nothing to undo
    for pos in (1, 50, 1000, 123456, (1 << 24) - 128):
        u = oracle.unrotate_keys(bits, 1, theta, pos)
        assert np.array_equal(u, u.astype(np.float32).astype(np.float64))  # float32 values
        # the pinned forward rotation brings the keys back, up to float32 rounding of a pair
        back = oracle.rope_rotate(u, theta, float(pos))
        pair = np.sqrt(x[..., : d // 2] ** 2 + x[..., d // 2 :] ** 2)
        bound = 4 * 2.0**-24 * np.concatenate([pair, pair], -1) + 1e-30
        assert np.all(np.abs(back - x) <= bound)
        # and it is the plain inverse rotation evaluated exactly, to the same bound
        assert np.all(np.abs(u - oracle.rope_rotate(x, theta, -float(pos))) <= bound)
    # closed form on unit vectors: plane 0 has frequency 1, so e_0 -> (cos p, -sin p) on (0, d/2)
    e = np.zeros((1, 1, d))
    e[0, 0, 0] = 1.0
    u = oracle.unrotate_keys(oracle.round_to_bits(e, 1), 1, theta, 1000)[0, 0]
    assert u[0] == np.float32(math.cos(1000.0)) and u[d // 2] == -np.float32(math.sin(1000.0))
    assert np.all(u[1 : d // 2] == 0) and np.all(u[d // 2 + 1 :] == 0)


# ------------------------------------------------------------------ Eq. 6 with compact (binary16) metadata
def test_compact_metadata_quantiser_rounds_outward_and_keeps_the_error_bound():
    r = np.random.default_rng(77)
    x = oracle.bits_to_f64(oracle.round_to_bits(r.standard_normal((64, 2, 32)) * np.exp(r.uniform(-3, 3, (1, 2, 32))), 1), 1)
    for bits, levels in ((8, 255), (4, 15)):
        for which in ("k", "v"):
            if which == "k":
                codes, meta = oracle.quantize_k(x, bits, 32, meta16=True)
                c0, m0 = oracle.quantize_k(x, bits, 32)
                deq = oracle.dequant_k(codes, meta, 32, bits, 32)
                grp_min = x.reshape(2, 32, 2, 32).min(axis=1)        # [G,H,d]
                grp_max = x.reshape(2, 32, 2, 32).max(axis=1)
                s_of = np.repeat(meta[..., 0], 32, axis=0).astype(np.float64)
            else:
                codes, meta = oracle.quantize_v(x, bits, 16, meta16=True)
                c0, m0 = oracle.quantize_v(x, bits, 16)
                deq = oracle.dequant_v(codes, meta, 32, bits, 16)
                grp_min = x.reshape(64, 2, 2, 16).min(axis=3)        # [C,H,G]
                grp_max = x.reshape(64, 2, 2, 16).max(axis=3)
                s_of = np.repeat(meta[..., 0], 16, axis=2).astype(np.float64)
            s16, m16 = meta[..., 0], meta[..., 1]
            # the stored pair is binary16; min is the largest binary16 value not above the true minimum
            assert np.array_equal(meta, meta.astype(np.float16).astype(np.float32))
            assert np.all(m16 <= grp_min)
            above = np.nextafter(m16.astype(np.float16), np.float16(np.inf)).astype(np.float64)
            assert np.all(above > grp_min)
            # scale is the smallest binary16 value not below (max - min16)/levels (float32 division)
            want = ((grp_max.astype(np.float32) - m16) / np.float32(levels)).astype(np.float32)
            assert np.all(s16 >= want)
            below = np.nextafter(s16.astype(np.float16), np.float16(-np.inf)).astype(np.float32)
            assert np.all(below < want)
            # so every value is inside the code range and the error stays half a (rounded) step
            assert np.all(np.abs(deq - x) <= 0.5 * s_of * (1 + 1e-6) + 1e-12)
            # and the float32 variant is untouched by the option
            assert np.array_equal(c0, (oracle.quantize_k(x, bits, 32) if which == "k" else oracle.quantize_v(x, bits, 16))[0])
