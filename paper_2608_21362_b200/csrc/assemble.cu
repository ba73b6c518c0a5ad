// Stitching kernel: dequantise (inverse of KV Quantization Eq. 6), rotate keys by
// R_theta^(new_pos - orig_pos) (Rotary Positional Embeddings, Eq. 3) and write the rows
// of one cached chunk into the request's [L][2][T][H][d] buffer (Prompt Assembly).
//
// One CTA per (chunk, layer, K|V).  The chunk-layer's packed codes and its (scale, min)
// metadata are contiguous in global memory, so one thread fetches them with bulk async
// copies (TMA, mbarrier completion) in four parts; half-warps start on a part as soon as it
// lands.  A half-warp owns one KV head and a run of tokens; lane ln owns channels
// 4ln..4ln+3 and their rotation partners 64+4ln..64+4ln+3, so both operands of every
// rotation pair sit in the same thread and the per-channel affine terms
//     k'_c = A_c q_c + B_c q_(c^64) + C_c
// (scale, min, cos and sin folded together once per token group) stay in registers.
// Output rows go out as 128-byte contiguous stores per half-warp.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "deviation_math.cuh"
#include "f32x2.cuh"
#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

constexpr int kThreads = 256;
constexpr int kParts = 4;
constexpr uint32_t kWaitLimit = 1u << 22;
constexpr int kHeadDim = 128;
constexpr int kChunkTokens = 128;  // the context refuses other chunk and group sizes
constexpr int kInt4Group = 32;

// CTAs per (chunk, layer, K|V): 1 for up to 2 KV heads, H/2 beyond, so a CTA never stages more
// than 256 (token, head) rows.
__host__ __device__ inline int assemble_split(int H) { return H > 2 ? H / 2 : 1; }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kWaitLimit polls (never expected; keeps a bad launch from hanging).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(64);
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// byte k of x in the low mantissa bits of 2^23: the float 2^23 + q
template <int K>
__device__ __forceinline__ float byte_magic(uint32_t x) {
  return __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650u + K));
}
// nibble k of a 16-bit word in the top mantissa bits of 16.0: the float 16 + q
template <int K>
__device__ __forceinline__ float nibble_magic(uint32_t x) {
  return __uint_as_float(((x << (19 - 4 * K)) & 0x00780000u) | 0x41800000u);
}

template <typename T>
struct Pack;
template <>
struct Pack<__nv_bfloat16> {
  static constexpr int DT = KVB_DT_BF16;
  static __device__ __forceinline__ uint32_t two(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
  }
  static __device__ __forceinline__ uint64_t unpack2(uint32_t x) {
    return f2_pack(__uint_as_float(x << 16), __uint_as_float(x & 0xFFFF0000u));
  }
};
template <>
struct Pack<__half> {
  static constexpr int DT = KVB_DT_F16;
  static __device__ __forceinline__ uint32_t two(float a, float b) {
    __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
  }
  static __device__ __forceinline__ uint64_t unpack2(uint32_t x) {
    const float2 t = __half22float2(*reinterpret_cast<__half2*>(&x));
    return f2_pack(t.x, t.y);
  }
};

// rounds four values to the output type, stores them and returns the stored words
template <typename OutT>
__device__ __forceinline__ uint2 store4(OutT* p, const uint64_t (&v)[2]) {
  float a, b, c, e;
  f2_unpack(v[0], a, b);
  f2_unpack(v[1], c, e);
  const uint2 w = make_uint2(Pack<OutT>::two(a, b), Pack<OutT>::two(c, e));
  *reinterpret_cast<uint2*>(p) = w;
  return w;
}

__device__ __forceinline__ void copy_rows(uint8_t* dst, const uint8_t* src, size_t bytes, int tid) {
  const uint4* s = reinterpret_cast<const uint4*>(src);
  uint4* d = reinterpret_cast<uint4*>(dst);
  const size_t n = bytes / 16;
  size_t i = tid;
  for (; i + 3 * kThreads < n; i += 4 * kThreads) {
    uint4 a = __ldcs(s + i), b = __ldcs(s + i + kThreads), c = __ldcs(s + i + 2 * kThreads),
          e = __ldcs(s + i + 3 * kThreads);
    d[i] = a;
    d[i + kThreads] = b;
    d[i + 2 * kThreads] = c;
    d[i + 3 * kThreads] = e;
  }
  for (; i < n; i += kThreads) d[i] = __ldcs(s + i);
}

// Copy of `rows` 256-byte (token, head) rows (a multiple of 32) that also takes each row's sums: a
// half-warp per row, two rows per pass.  dev_on: the row's deviation term against the fresh tensor
// goes to the accumulator of its token (acc_tok points at the first row's token).  norm_on: the
// row's L2 norm is added to norm_part on lanes 0 and 8 of the half-warp (Eq. 7).
template <int DT>
__device__ __forceinline__ void copy_rows_dev(uint8_t* dst, const uint8_t* src, const uint8_t* fresh, int rows, int H,
                                              int tid, unsigned long long* acc_tok, bool dev_on, bool norm_on, float& norm_part) {
  const int lane = tid & 31, s = lane >> 4, ln = lane & 15;
  const int hw = (tid >> 5) * 2 + s;
  const bool heads_paired = (H & 1) == 0;  // rows 2w, 2w+1 of a warp belong to one token
  for (int ua = hw; ua < rows; ua += 32) {
    const int ub = ua + 16;
    const size_t oa = (size_t)ua * 256 + (size_t)ln * 16, ob = (size_t)ub * 256 + (size_t)ln * 16;
    const uint4 a0 = __ldcs(reinterpret_cast<const uint4*>(src + oa)), a1 = __ldcs(reinterpret_cast<const uint4*>(src + ob));
    uint4 b0 = a0, b1 = a1;  // without the deviation only the norms are wanted
    if (dev_on) b0 = __ldcs(reinterpret_cast<const uint4*>(fresh + oa)), b1 = __ldcs(reinterpret_cast<const uint4*>(fresh + ob));
    *reinterpret_cast<uint4*>(dst + oa) = a0;
    *reinterpret_cast<uint4*>(dst + ob) = a1;
    float sa[3], sb[3], na2;
    row_sums<DT>(a0, b0, sa[0], sa[1], sa[2]);
    row_sums<DT>(a1, b1, sb[0], sb[1], sb[2]);
    long long fx = pair_terms_fixed(sa, sb, ln, true, true, na2);
    if (norm_on && (ln & 7) == 0) norm_part += sqrt_fast(na2);
    if (dev_on) {
      if (heads_paired) fx += __shfl_xor_sync(0xffffffffu, fx, 16);
      if ((ln & 7) == 0 && (!heads_paired || s == 0)) atomicAdd(acc_tok + ((ln & 8) ? ub : ua) / H, (unsigned long long)fx);
    }
  }
}

// Sum of the CTA's norm parts (held by lanes 0 and 8 of every half-warp), added up in a fixed order
// and written as one double: the chunk-layer's share of the importance score.
__device__ __forceinline__ void store_norm_sum(float part, int tid, float* s_part, double* out) {
  part += __shfl_xor_sync(0xffffffffu, part, 8);
  part += __shfl_xor_sync(0xffffffffu, part, 16);
  if ((tid & 31) == 0) s_part[tid >> 5] = part;
  __syncthreads();
  if (tid == 0) {
    double tot = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) tot += (double)s_part[w];
    *out = tot;
  }
}

// DEV = true takes the sums of every written row while it is in registers: its deviation against the
// fresh tensor (Algorithm 2, step 2) goes to acc[token] -- K rows when which & 1, V rows when
// which & 2.  NORM = true (a variant of DEV = true) also adds up the L2 norms of the key rows of this
// chunk-layer into norm_sums[chunk][layer][part]: the importance score, Eq. 7, as a by-product of
// the stitch.
template <typename OutT, bool DEV, bool NORM>
__global__ void __launch_bounds__(kThreads, 3)
    assemble_kernel(const ChunkDesc* __restrict__ chunks, const float2* __restrict__ cs_table, ModelDims m,
                    uint32_t* __restrict__ status, int which, unsigned long long* __restrict__ acc,
                    double* __restrict__ norm_sums) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bars[kParts + 1];
  __shared__ float s_norm[kThreads / 32];

  pdl_wait();  // the descriptors and the rotation table come from the kernel before this one
  const int tid = threadIdx.x;
  const int H = m.Hkv;
  const int split = assemble_split(H);  // CTAs per chunk-layer, so that a CTA stages at most 256 rows
  int item = blockIdx.x;
  const int part_id = item % split;
  item /= split;
  const int kv = item & 1;
  const int l = (item >> 1) % m.L;
  const int ci = (item >> 1) / m.L;
  const ChunkDesc cd = chunks[ci];
  const int C = m.C / split;            // tokens of this CTA
  const int tb = part_id * C;           // first token of this CTA within the chunk
  constexpr int d = kHeadDim;
  const size_t row_elems = (size_t)H * d;
  const size_t dst_off = ((size_t)(l * 2 + kv) * cd.T + cd.new_pos + tb) * row_elems;  // in elements
  OutT* dst = reinterpret_cast<OutT*>(cd.kv_buf) + dst_off;
  const size_t out_bytes = (size_t)C * row_elems * 2;
  const size_t layer_out_bytes = (size_t)m.C * row_elems * 2;

  const bool dev_on = DEV && acc != nullptr && (which & (kv ? 2 : 1));
  const bool norm_on = NORM && kv == 0;
  unsigned long long* acc_tok = dev_on ? acc + cd.tok_offset + cd.new_pos + tb : nullptr;  // this CTA's first token
  auto norm_out = [&]() { return norm_sums + ((size_t)ci * m.L + l) * split + part_id; };  // this CTA's slot
  float norm_part = 0.f;  // lanes 0 and 8 of each half-warp: norms of the rows they reduced

  // ---- rows that are plain copies: FRESH chunks (deviation 0); unquantised values; unquantised keys that do not move
  if (cd.mode == KVB_MODE_FRESH) {
    if (norm_on) {
      copy_rows_dev<Pack<OutT>::DT>(reinterpret_cast<uint8_t*>(dst), cd.fresh + dst_off * 2, nullptr, C * H, H, tid, nullptr, false, true, norm_part);
      store_norm_sum(norm_part, tid, s_norm, norm_out());
    } else {
      copy_rows(reinterpret_cast<uint8_t*>(dst), cd.fresh + dst_off * 2, out_bytes, tid);
    }
    return;
  }
  if (cd.mode == KVB_MODE_FP16 && (kv == 1 || cd.delta_pos == 0)) {
    const uint8_t* src = (kv ? cd.v_src : cd.k_src) + (size_t)l * layer_out_bytes + (size_t)tb * row_elems * 2;
    if (dev_on || norm_on) {
      copy_rows_dev<Pack<OutT>::DT>(reinterpret_cast<uint8_t*>(dst), src, cd.fresh + dst_off * 2, C * H, H, tid, acc_tok, dev_on, norm_on, norm_part);
      if (norm_on) store_norm_sum(norm_part, tid, s_norm, norm_out());
    } else {
      copy_rows(reinterpret_cast<uint8_t*>(dst), src, out_bytes, tid);
    }
    return;
  }

  // ---- staged path.  The chunk shape is fixed (128 tokens, head_dim 128, INT4 groups of 32: the
  //      context refuses anything else) and the head count is a power of two, so all the per-row
  //      index arithmetic below is shifts and masks; the code width and the metadata width are
  //      compile-time in the row loops (one instantiation per mode inside this kernel).
  const int lane = tid & 31, warp = tid >> 5;
  const int s = lane >> 4, ln = lane & 15;
  const int hw = warp * 2 + s;  // half-warp 0..15
  const int log_h = __ffs(H) - 1;
  const int h = hw & (H - 1);
  const int log_tok_per = __ffs(C) - 1 - (4 - log_h);  // a CTA's C tokens over 16 / H half-warp slots
  const int tok_per = 1 << log_tok_per;
  const int t0 = (hw >> log_h) << log_tok_per;
  const int log_part = __ffs(C) - 1 - 2;               // tokens per staged part (kParts = 4)
  static_assert(kParts == 4, "the part of a token is a shift");
  const uint8_t* fresh_rows = cd.fresh + dst_off * 2;
  bool ok = true;

  auto staged = [&](auto bits_tag, auto meta16_tag) {
    constexpr int BITS = decltype(bits_tag)::value;
    constexpr bool META16 = decltype(meta16_tag)::value;
    constexpr uint32_t pair_bytes = META16 ? 4 : 8;  // one (scale, min) pair
    const uint32_t code_bytes = (uint32_t)(C * row_elems * BITS / 8);  // this CTA's share of the layer's codes
    const uint8_t* codes_g = (kv ? cd.v_src : cd.k_src) + ((size_t)l * split + part_id) * code_bytes;
    uint32_t meta_bytes = 0;
    const uint8_t* meta_g = nullptr;
    constexpr int G = BITS == 8 ? 1 : kHeadDim / kInt4Group;  // value channel groups per row
    int g_first = 0;                                           // first key token group held in shared memory
    if (BITS != 16) {
      if (!kv) {
        constexpr int G_layer = BITS == 8 ? 1 : kChunkTokens / kInt4Group;
        g_first = BITS == 8 ? 0 : tb / kInt4Group;
        const int n_g = BITS == 8 ? 1 : (tb + C - 1) / kInt4Group - g_first + 1;
        meta_bytes = (uint32_t)(n_g * row_elems * pair_bytes);
        meta_g = reinterpret_cast<const uint8_t*>(cd.k_meta) + ((size_t)l * G_layer + g_first) * row_elems * pair_bytes;
      } else {
        meta_bytes = (uint32_t)(C * H * G * pair_bytes);
        meta_g = reinterpret_cast<const uint8_t*>(cd.v_meta) + ((size_t)l * split + part_id) * meta_bytes;
      }
    }
    uint8_t* s_codes = smem;
    const float* s_meta = reinterpret_cast<const float*>(smem + code_bytes);
    const uint32_t part_bytes = code_bytes / kParts;

    if (tid == 0) {
      for (int i = 0; i <= kParts; ++i) mbar_init(&bars[i], 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
      if (meta_bytes) {
        mbar_expect_tx(&bars[0], meta_bytes);
        bulk_g2s(smem + code_bytes, meta_g, meta_bytes, &bars[0]);
      }
      for (int p = 0; p < kParts; ++p) {
        mbar_expect_tx(&bars[1 + p], part_bytes);
        bulk_g2s(s_codes + (size_t)p * part_bytes, codes_g + (size_t)p * part_bytes, part_bytes, &bars[1 + p]);
      }
    }

    const int off_a = s ? 64 : 0, off_b = s ? 0 : 64;  // second half-warp reads the high half first (bank spread)
    if (meta_bytes) ok = mbar_wait(&bars[0], 0);
    int ready_part = -1;

    // Codes become floats without a conversion instruction: an 8-bit code goes into the low mantissa
    // bits of 2^23 (value 2^23 + q, then one exact subtraction, done on packed pairs); a 4-bit code
    // goes into the top mantissa bits of 16.0 (value 16 + q) and the 16 is folded into the constant
    // term.  All affine arithmetic runs on packed float32 pairs.
    const uint64_t neg_magic2 = f2_pack(-8388608.0f, -8388608.0f);
    auto load_codes = [&](int u, uint64_t (&ql)[2], uint64_t (&qh)[2]) {
      if constexpr (BITS == 8) {
        const uint8_t* row = s_codes + ((size_t)u << 7);
        const uint32_t xa = *reinterpret_cast<const uint32_t*>(row + off_a + 4 * ln);
        const uint32_t xb = *reinterpret_cast<const uint32_t*>(row + off_b + 4 * ln);
        const uint32_t xl = s ? xb : xa, xh = s ? xa : xb;
        ql[0] = f2_add(f2_pack(byte_magic<0>(xl), byte_magic<1>(xl)), neg_magic2);
        ql[1] = f2_add(f2_pack(byte_magic<2>(xl), byte_magic<3>(xl)), neg_magic2);
        qh[0] = f2_add(f2_pack(byte_magic<0>(xh), byte_magic<1>(xh)), neg_magic2);
        qh[1] = f2_add(f2_pack(byte_magic<2>(xh), byte_magic<3>(xh)), neg_magic2);
      } else {
        const uint8_t* row = s_codes + ((size_t)u << 6);
        const uint32_t xl = *reinterpret_cast<const uint16_t*>(row + 2 * ln);
        const uint32_t xh = *reinterpret_cast<const uint16_t*>(row + 32 + 2 * ln);
        ql[0] = f2_pack(nibble_magic<0>(xl), nibble_magic<1>(xl));
        ql[1] = f2_pack(nibble_magic<2>(xl), nibble_magic<3>(xl));
        qh[0] = f2_pack(nibble_magic<0>(xh), nibble_magic<1>(xh));
        qh[1] = f2_pack(nibble_magic<2>(xh), nibble_magic<3>(xh));
      }
    };
    constexpr float bias = BITS == 4 ? 16.f : 0.f;  // what the 4-bit unpacking adds to every code

    // waits (bounded) for the part of the codes that token t lies in; false = give up
    auto part_ready = [&](int t) {
      const int part = t >> log_part;
      if (part != ready_part) {
        ok = ok && mbar_wait(&bars[1 + part], 0);
        ready_part = part;
      }
      if (DEV) ok = __all_sync(0xffffffffu, ok);  // the row sums' shuffles need the whole warp
      return ok;
    };
    // Deviation terms of tokens t and t+1 of this half-warp's head: the stored words are still in
    // registers, the fresh row's matching 2 x 8 bytes per lane come from global memory.
    // The fresh words of a pair are fetched one pair ahead of their use (f[0..1]: token t, f[2..3]: t+1),
    // so the loads' latency is covered by the previous pair's arithmetic.
    auto load_fresh = [&](int t, uint2 (&f)[4]) {
      const uint8_t* f0 = fresh_rows + ((size_t)((t << log_h) + h) << 8) + 8 * ln;
      const uint8_t* f1 = f0 + ((size_t)H << 8);
      f[0] = __ldcs(reinterpret_cast<const uint2*>(f0)), f[1] = __ldcs(reinterpret_cast<const uint2*>(f0 + 128));
      f[2] = __ldcs(reinterpret_cast<const uint2*>(f1)), f[3] = __ldcs(reinterpret_cast<const uint2*>(f1 + 128));
    };
    auto dev_pair = [&](int t, const uint2& wl0, const uint2& wh0, const uint2& wl1, const uint2& wh1, const uint2 (&f)[4]) {
      const uint32_t a0[4] = {wl0.x, wl0.y, wh0.x, wh0.y}, a1[4] = {wl1.x, wl1.y, wh1.x, wh1.y};
      float sa[3], sb[3], na2;
      if (dev_on) {
        const uint32_t b0[4] = {f[0].x, f[0].y, f[1].x, f[1].y}, b1[4] = {f[2].x, f[2].y, f[3].x, f[3].y};
        row_sums4<Pack<OutT>::DT>(a0, b0, sa[0], sa[1], sa[2]);
        row_sums4<Pack<OutT>::DT>(a1, b1, sb[0], sb[1], sb[2]);
      } else {  // only the norms are wanted
        row_sums4<Pack<OutT>::DT>(a0, a0, sa[0], sa[1], sa[2]);
        row_sums4<Pack<OutT>::DT>(a1, a1, sb[0], sb[1], sb[2]);
      }
      long long fx = pair_terms_fixed(sa, sb, ln, true, true, na2);
      if (norm_on && (ln & 7) == 0) norm_part += sqrt_fast(na2);
      if (dev_on) {
        const bool heads_paired = (H & 1) == 0;  // the warp's two half-warps hold two heads of the same tokens
        if (heads_paired) fx += __shfl_xor_sync(0xffffffffu, fx, 16);
        if ((ln & 7) == 0 && (!heads_paired || s == 0)) atomicAdd(acc_tok + t + (ln >> 3), (unsigned long long)fx);
      }
    };
    // the row loop shared by keys and values: two tokens per pass, the next pair's fresh words in flight
    auto run_rows = [&](auto&& one_row) {
      uint2 fr[4] = {}, fr_next[4] = {};
      if (dev_on) load_fresh(t0, fr);
      for (int tt = 0; tt < tok_per; tt += 2) {  // tok_per is even and a pair never straddles a part
        const int t = t0 + tt;
        if (!part_ready(t)) break;
        if (dev_on && tt + 2 < tok_per) load_fresh(t + 2, fr_next);
        uint2 wl0, wh0, wl1, wh1;
        one_row(t, wl0, wh0);
        one_row(t + 1, wl1, wh1);
        if (DEV && (dev_on || norm_on)) {
          dev_pair(t, wl0, wh0, wl1, wh1, fr);
#pragma unroll
          for (int i = 0; i < 4; ++i) fr[i] = fr_next[i];
        }
      }
    };

    if (!kv) {
      // ------------------------------ keys
      uint64_t A_lo[2], B_lo[2], C_lo[2], A_hi[2], B_hi[2], C_hi[2];
      float cs_c[4], cs_s[4];
      {
        const float4* p = reinterpret_cast<const float4*>(cs_table + (size_t)ci * (d / 2) + 4 * ln);
        float4 a = __ldg(p), b = __ldg(p + 1);
        cs_c[0] = a.x, cs_s[0] = a.y, cs_c[1] = a.z, cs_s[1] = a.w;
        cs_c[2] = b.x, cs_s[2] = b.y, cs_c[3] = b.z, cs_s[3] = b.w;
      }
      // folds (scale, min) of token group g with the rotation into the three per-channel constants
      auto fold_group = [&](int g) {
        float sl[4], ml[4], sh[4], mh[4];  // (scale, min) of this lane's 4 low and 4 high channels
        const size_t pair = ((size_t)((g << log_h) + h) << 7) + 4 * ln;
        if constexpr (META16) {
          const uint4 a = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(s_meta) + pair * 4);
          const uint4 b = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(s_meta) + (pair + 64) * 4);
          const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&aw[i]));
            const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&bw[i]));
            sl[i] = lo.x, ml[i] = lo.y, sh[i] = hi.x, mh[i] = hi.y;
          }
        } else {
          const float* mlo = s_meta + pair * 2;
          const float4 a0 = *reinterpret_cast<const float4*>(mlo), a1 = *reinterpret_cast<const float4*>(mlo + 4);
          const float4 b0 = *reinterpret_cast<const float4*>(mlo + 128), b1 = *reinterpret_cast<const float4*>(mlo + 132);
          sl[0] = a0.x, sl[1] = a0.z, sl[2] = a1.x, sl[3] = a1.z, ml[0] = a0.y, ml[1] = a0.w, ml[2] = a1.y, ml[3] = a1.w;
          sh[0] = b0.x, sh[1] = b0.z, sh[2] = b1.x, sh[3] = b1.z, mh[0] = b0.y, mh[1] = b0.w, mh[2] = b1.y, mh[3] = b1.w;
        }
        float al[4], bl[4], cl[4], ah[4], bh[4], ch[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          al[i] = sl[i] * cs_c[i];
          bl[i] = -(sh[i] * cs_s[i]);
          cl[i] = fmaf(ml[i], cs_c[i], -(mh[i] * cs_s[i]));
          ah[i] = sh[i] * cs_c[i];
          bh[i] = sl[i] * cs_s[i];
          ch[i] = fmaf(mh[i], cs_c[i], ml[i] * cs_s[i]);
          cl[i] = fmaf(-bias, al[i] + bl[i], cl[i]);
          ch[i] = fmaf(-bias, ah[i] + bh[i], ch[i]);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          A_lo[i] = f2_pack(al[2 * i], al[2 * i + 1]), B_lo[i] = f2_pack(bl[2 * i], bl[2 * i + 1]), C_lo[i] = f2_pack(cl[2 * i], cl[2 * i + 1]);
          A_hi[i] = f2_pack(ah[2 * i], ah[2 * i + 1]), B_hi[i] = f2_pack(bh[2 * i], bh[2 * i + 1]), C_hi[i] = f2_pack(ch[2 * i], ch[2 * i + 1]);
        }
      };
      int cur_group = -1;
      if constexpr (BITS == 8) {  // one group: the whole chunk
        if (ok) fold_group(0);
      }
      auto key_row = [&](int t, uint2& wl, uint2& wh) {
        const int u = (t << log_h) + h;
        OutT* orow = dst + ((size_t)u << 7);
        uint64_t ol[2], oh[2];
        if constexpr (BITS == 16) {
          const uint64_t c2[2] = {f2_pack(cs_c[0], cs_c[1]), f2_pack(cs_c[2], cs_c[3])};
          const uint64_t s2[2] = {f2_pack(cs_s[0], cs_s[1]), f2_pack(cs_s[2], cs_s[3])};
          const uint64_t ns2[2] = {f2_pack(-cs_s[0], -cs_s[1]), f2_pack(-cs_s[2], -cs_s[3])};
          const uint8_t* row = s_codes + ((size_t)u << 8);
          const uint2 a = *reinterpret_cast<const uint2*>(row + 8 * ln);
          const uint2 b = *reinterpret_cast<const uint2*>(row + 128 + 8 * ln);
          const uint64_t xl[2] = {Pack<OutT>::unpack2(a.x), Pack<OutT>::unpack2(a.y)};
          const uint64_t xh[2] = {Pack<OutT>::unpack2(b.x), Pack<OutT>::unpack2(b.y)};
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            ol[i] = f2_fma(xl[i], c2[i], f2_mul(xh[i], ns2[i]));
            oh[i] = f2_fma(xh[i], c2[i], f2_mul(xl[i], s2[i]));
          }
        } else {
          if constexpr (BITS == 4) {
            const int g = ((tb + t) >> 5) - g_first;
            if (g != cur_group) {
              cur_group = g;
              fold_group(g);
            }
          }
          uint64_t ql[2], qh[2];
          load_codes(u, ql, qh);
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            ol[i] = f2_fma(A_lo[i], ql[i], f2_fma(B_lo[i], qh[i], C_lo[i]));
            oh[i] = f2_fma(A_hi[i], qh[i], f2_fma(B_hi[i], ql[i], C_hi[i]));
          }
        }
        wl = store4(orow + 4 * ln, ol);
        wh = store4(orow + 64 + 4 * ln, oh);
      };
      run_rows(key_row);
    } else if constexpr (BITS != 16) {
      // ------------------------------ values (INT8 / INT4 only; never rotated)
      auto pair_at = [&](size_t pair) {  // (scale, min) pair number `pair` of the staged metadata
        if constexpr (META16) return __half22float2(reinterpret_cast<const __half2*>(s_meta)[pair]);
        else return *reinterpret_cast<const float2*>(s_meta + pair * 2);
      };
      auto value_row = [&](int t, uint2& wl, uint2& wh) {
        const int u = (t << log_h) + h;
        OutT* orow = dst + ((size_t)u << 7);
        float s_lo, m_lo, s_hi, m_hi;
        if constexpr (BITS == 8) {
          const float2 sm = pair_at((size_t)u);
          s_lo = s_hi = sm.x, m_lo = m_hi = sm.y;
        } else {
          const int g_lo = (4 * ln) / kInt4Group, g_hi = (64 + 4 * ln) / kInt4Group;
          const float2 a = pair_at((size_t)u * G + g_lo);
          const float2 b = pair_at((size_t)u * G + g_hi);
          s_lo = a.x, m_lo = fmaf(-bias, a.x, a.y), s_hi = b.x, m_hi = fmaf(-bias, b.x, b.y);
        }
        uint64_t ql[2], qh[2], ol[2], oh[2];
        load_codes(u, ql, qh);
        const uint64_t sl2 = f2_pack(s_lo, s_lo), ml2 = f2_pack(m_lo, m_lo), sh2 = f2_pack(s_hi, s_hi), mh2 = f2_pack(m_hi, m_hi);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          ol[i] = f2_fma(ql[i], sl2, ml2);
          oh[i] = f2_fma(qh[i], sh2, mh2);
        }
        wl = store4(orow + 4 * ln, ol);
        wh = store4(orow + 64 + 4 * ln, oh);
      };
      run_rows(value_row);
    }

    if (norm_on) store_norm_sum(norm_part, tid, s_norm, norm_out());
    if (!ok) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
    // Every thread drains every barrier before the CTA may retire, so no bulk copy can still be
    // writing this CTA's shared memory when it is handed to the next CTA.
    bool all = true;
    if (meta_bytes) all = mbar_wait(&bars[0], 0) && all;
    for (int p = 0; p < kParts; ++p) all = mbar_wait(&bars[1 + p], 0) && all;
    if (!all) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
  };

  using std::integral_constant;
  const bool meta16 = cd.meta16 != 0;  // (scale, min) pairs of 2 x 2 bytes instead of 2 x 4
  if (cd.mode == KVB_MODE_INT8) {
    if (meta16) staged(integral_constant<int, 8>{}, integral_constant<bool, true>{});
    else staged(integral_constant<int, 8>{}, integral_constant<bool, false>{});
  } else if (cd.mode == KVB_MODE_INT4) {
    if (meta16) staged(integral_constant<int, 4>{}, integral_constant<bool, true>{});
    else staged(integral_constant<int, 4>{}, integral_constant<bool, false>{});
  } else {
    staged(integral_constant<int, 16>{}, integral_constant<bool, false>{});
  }
}

// cos/sin of delta_pos * theta^(-2j/d) in double, stored as float (one thread per plane j)
__global__ void rope_table_kernel(const ChunkDesc* __restrict__ chunks, int n_chunks, const double* __restrict__ inv_freq,
                                  int half_d, float2* __restrict__ cs_table) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_chunks * half_d) return;
  const int ci = i / half_d, j = i % half_d;
  const double a = (double)chunks[ci].delta_pos * inv_freq[j];
  double sn, c;
  sincos(a, &sn, &c);
  cs_table[i] = make_float2((float)c, (float)sn);
}

// Eq. 7 from the stitch's by-product: importance of chunk ci = sum of its chunk-layers' norm sums
// (added in layer order) / (L * H * C).  One thread per chunk descriptor.
__global__ void importance_finalize_kernel(const ChunkDesc* __restrict__ chunks, int n_chunks, int parts_per_chunk,
                                           const double* __restrict__ norm_sums, double inv_rows) {
  const int ci = blockIdx.x * blockDim.x + threadIdx.x;
  if (ci >= n_chunks) return;
  float* out = chunks[ci].imp_out;
  if (!out) return;
  double tot = 0.0;
  for (int i = 0; i < parts_per_chunk; ++i) tot += norm_sums[(size_t)ci * parts_per_chunk + i];
  *out = (float)(tot * inv_rows);
}

}  // namespace

int assemble_parts_per_layer(int Hkv) { return assemble_split(Hkv); }

cudaError_t launch_importance_finalize(const ChunkDesc* chunks, int n_chunks, const ModelDims& m, const double* norm_sums,
                                       cudaStream_t st) {
  const int parts = m.L * assemble_split(m.Hkv);
  importance_finalize_kernel<<<(n_chunks + 127) / 128, 128, 0, st>>>(chunks, n_chunks, parts, norm_sums,
                                                                    1.0 / ((double)m.L * m.Hkv * m.C));
  return cudaGetLastError();
}

size_t assemble_smem_bytes(const ModelDims& m, int mode) {
  const size_t E = (size_t)m.Hkv * m.d;
  const size_t C = (size_t)m.C / assemble_split(m.Hkv);  // tokens per CTA
  auto mx = [](size_t a, size_t b) { return a > b ? a : b; };
  switch (mode) {
    case KVB_MODE_FP16:
      return C * E * 2;
    case KVB_MODE_INT8:
      return C * E + mx(E * 8, C * m.Hkv * 8);
    case KVB_MODE_INT4:
      return C * E / 2 + mx(((C + m.int4_group - 1) / m.int4_group) * E * 8, C * m.Hkv * (m.d / m.int4_group) * 8);
    default:
      return 0;
  }
}

cudaError_t assemble_configure(size_t max_smem) {
  const void* fns[6] = {(const void*)assemble_kernel<__nv_bfloat16, false, false>, (const void*)assemble_kernel<__nv_bfloat16, true, false>,
                        (const void*)assemble_kernel<__nv_bfloat16, true, true>,   (const void*)assemble_kernel<__half, false, false>,
                        (const void*)assemble_kernel<__half, true, false>,         (const void*)assemble_kernel<__half, true, true>};
  for (const void* f : fns) {
    cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_rope_table(const ChunkDesc* chunks, int n_chunks, const double* inv_freq, int half_d,
                              float2* cs_table, cudaStream_t st) {
  const int n = n_chunks * half_d;
  rope_table_kernel<<<(n + 127) / 128, 128, 0, st>>>(chunks, n_chunks, inv_freq, half_d, cs_table);
  return cudaGetLastError();
}

cudaError_t launch_assemble(const ChunkDesc* chunks, int n_chunks, const float2* cs_table, const ModelDims& m,
                            size_t smem_bytes, uint32_t* status, int which, unsigned long long* acc, double* norm_sums,
                            bool pdl, cudaStream_t st) {
  const unsigned grid = (unsigned)n_chunks * m.L * 2 * assemble_split(m.Hkv);
  const bool dev = acc != nullptr && (which & 3);
  if (!dev) which = 0, acc = nullptr;
  const dim3 g(grid), b(kThreads);
  if (m.dtype == KVB_DT_BF16) {
    if (norm_sums) return launch_pdl(pdl, assemble_kernel<__nv_bfloat16, true, true>, g, b, smem_bytes, st, chunks, cs_table, m, status, which, acc, norm_sums);
    if (dev) return launch_pdl(pdl, assemble_kernel<__nv_bfloat16, true, false>, g, b, smem_bytes, st, chunks, cs_table, m, status, which, acc, norm_sums);
    return launch_pdl(pdl, assemble_kernel<__nv_bfloat16, false, false>, g, b, smem_bytes, st, chunks, cs_table, m, status, which, acc, norm_sums);
  }
  if (norm_sums) return launch_pdl(pdl, assemble_kernel<__half, true, true>, g, b, smem_bytes, st, chunks, cs_table, m, status, which, acc, norm_sums);
  if (dev) return launch_pdl(pdl, assemble_kernel<__half, true, false>, g, b, smem_bytes, st, chunks, cs_table, m, status, which, acc, norm_sums);
  return launch_pdl(pdl, assemble_kernel<__half, false, false>, g, b, smem_bytes, st, chunks, cs_table, m, status, which, acc, norm_sums);
}

}  // namespace kvb
