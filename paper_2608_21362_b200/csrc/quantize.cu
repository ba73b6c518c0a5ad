// KV Quantization, Eq. 6 (cache-population side): asymmetric min/max quantisation of cached
// chunks, keys per channel over a token group, values per token over a channel group.
// scale = (max-min)/(2^b-1) and min are float32; the code is rint((x-min)/scale) in float32
// (IEEE subtract, divide, round-half-even), clamped.  A constant group gets scale 1, codes 0.
//
// One launch quantises a batch of chunks: a CTA per (chunk, layer, K|V, pair of KV heads), three CTAs per SM.
// The CTA's [128 tokens][<= 2 heads][128 channels] tile is fetched into shared memory by bulk copies
// (four large ones where the tile is contiguous, i.e. up to two KV heads; one per token row
// otherwise), with a barrier per 32 tokens so that work starts when the first quarter has landed.
//   keys    a thread owns a QUAD of neighbouring channels and a part of the tokens: one eight-byte load
//           per token brings the four values; the extremes are taken on the 16-bit values, two per
//           instruction; the parts of a group exchange their extremes through shared memory; the
//           codes come from packed float32 pairs and leave with one store per token.  With `unrotate`
//           every key is first rotated back by R_theta^(-orig_pos) (Rotary Positional Embeddings,
//           Eq. 3), so that the stored chunk is position-free and re-use at new_pos needs the single
//           rotation by new_pos; cos / sin come from a double-precision angle, the rotation itself
//           is float32 in a fixed order: u = fma(x, c, +-(x_partner * s)).
//   values  eight lanes per (token, head) row, 16 channels per lane, the extremes reduced by shuffles
//           of packed 16-bit words.
// The division of the code decision is the hardware reciprocal where that provably gives the same
// integer (the quotient lies away from every half-integer).  The other values -- with 16-bit inputs the
// quotients of a group lie on a coarse lattice, so about one in 250 is a tie or next to one -- are
// marked in a bit mask, collected on a list of the CTA and redone with the IEEE division in a second
// pass, one item per thread, so that neither pass runs with a few lanes of a warp.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

constexpr int kThreads = 256;
constexpr int kTokens = 128;   // tokens of a chunk
constexpr int kD = 128;        // head_dim
constexpr uint32_t kWaitLimit = 1u << 22;

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

// The code of a value: rint((v - mn) / s) clamped to [0, levels], the division being IEEE float32.
// Fast form, on packed pairs of values: q = (v - mn) * (1/s) with the hardware reciprocal (at most
// one unit in the last place off) differs from the real quotient by at most 1.5 * 2^-23 * q and the
// IEEE quotient by at most 2^-24 * q: together 2.5 * 2^-23 * levels < 3e-7 * levels.  When q lies
// further than 4e-7 * levels from every half-integer both therefore round to the same integer.
// q + 2^23 rounds q to that integer (round-half-even, as rint does) and leaves it in the low mantissa
// bits; no clamp is needed, the quotient cannot exceed levels by more than a rounding error.  The
// distance of q from its integer, |q - rint(q)|, is exact in float32; the caller keeps its maximum
// over a few values and lets the IEEE division decide for exactly those whose distance comes within
// the bound of one half (about one value in five thousand for 8-bit codes).
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void f2_unpack(uint64_t d, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(d)); }
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
constexpr float kMagic = 8388608.0f;  // 2^23
// The value pair v2 against (mn2, inv2): m0 / m1 = rint(q) + 2^23 as floats (the code in the low
// mantissa bits), r0 / r1 = rint(q); returns the larger |q - rint(q)| of the two.
__device__ __forceinline__ float code_fast2(uint64_t v2, uint64_t mn2, uint64_t inv2, float& m0, float& m1, float& r0, float& r1) {
  const uint64_t magic2 = f2_pack(kMagic, kMagic);
  const uint64_t q2 = f2_mul(f2_sub(v2, mn2), inv2);
  const uint64_t m2 = f2_add(q2, magic2);
  const uint64_t r2 = f2_sub(m2, magic2);
  float d0, d1;
  f2_unpack(f2_sub(q2, r2), d0, d1);
  f2_unpack(m2, m0, m1);
  f2_unpack(r2, r0, r1);
  return fmaxf(fabsf(d0), fabsf(d1));
}
// not inlined: the compiler must not evaluate the division speculatively on the common path
__device__ __noinline__ uint32_t code_exact(float v, float mn, float s, float levels) {
  float c = rintf(__fdiv_rn(__fsub_rn(v, mn), s));
  c = fminf(fmaxf(c, 0.f), levels);
  return (uint32_t)c;
}
// 1/s for code_fast2; usable: the scale is in the range where the reciprocal is accurate (otherwise
// the IEEE division decides for the whole group)
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ bool scale_usable(float s) { return s >= 1e-30f && s <= 1e30f; }
// Largest |q - rint(q)| for which the fast code is trusted, as the bit pattern of that float (for
// non-negative floats the integer order of the patterns is the order of the values); -1, below every
// pattern, when the scale is not usable.
__device__ __forceinline__ int32_t trust_limit(float s, float levels) { return scale_usable(s) ? __float_as_int(0.5f - 4e-7f * levels) : -1; }
// shifts `marks` left by one and brings in a 1 when dev > limit (dev >= 0): the sign of limit - dev
__device__ __forceinline__ uint32_t mark_near_tie(uint32_t marks, float dev, int32_t limit) {
  return __funnelshift_l((uint32_t)(limit - __float_as_int(dev)), marks, 1);
}

// four codes, each in the low byte of m_i's bit pattern, as one word (code 0 in the lowest byte)
__device__ __forceinline__ uint32_t pack4_u8(float m0, float m1, float m2, float m3) {
  const uint32_t a = __byte_perm(__float_as_uint(m0), __float_as_uint(m1), 0x0040);
  const uint32_t b = __byte_perm(__float_as_uint(m2), __float_as_uint(m3), 0x0040);
  return __byte_perm(a, b, 0x5410);
}
// two 4-bit codes as one byte (code 0 in the low nibble), in the low mantissa bits of the result:
// r1 * 16 + (r0 + 2^23), exact
__device__ __forceinline__ float pack2_u4(float m0, float r1) { return fmaf(r1, 16.f, m0); }

// two 16-bit values of one 32-bit word as a packed float32 pair
template <int DT>
__device__ __forceinline__ uint64_t unpack2(uint32_t w) {
  if (DT == KVB_DT_BF16) return f2_pack(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
  const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w));
  return f2_pack(t.x, t.y);
}
// element-wise minimum / maximum of two words of two 16-bit values each (exact: no rounding is involved)
template <int DT>
__device__ __forceinline__ uint32_t min2_16(uint32_t a, uint32_t b) {
  uint32_t r;
  if (DT == KVB_DT_BF16) {
    const __nv_bfloat162 t = __hmin2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    r = *reinterpret_cast<const uint32_t*>(&t);
  } else {
    const __half2 t = __hmin2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
    r = *reinterpret_cast<const uint32_t*>(&t);
  }
  return r;
}
template <int DT>
__device__ __forceinline__ uint32_t max2_16(uint32_t a, uint32_t b) {
  uint32_t r;
  if (DT == KVB_DT_BF16) {
    const __nv_bfloat162 t = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    r = *reinterpret_cast<const uint32_t*>(&t);
  } else {
    const __half2 t = __hmax2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
    r = *reinterpret_cast<const uint32_t*>(&t);
  }
  return r;
}

// (scale, min) of a group from its extremes.  Compact metadata: min is rounded down to binary16
// first, the scale is taken against the rounded min and rounded up, so no value leaves the code range.
__device__ __forceinline__ void group_params(float& mn, float mx, float levels, int meta16, float& s) {
  if (meta16) mn = __half2float(__float2half_rd(mn));
  s = mx > mn ? __fdiv_rn(__fsub_rn(mx, mn), levels) : 1.0f;
  if (meta16) s = __half2float(__float2half_ru(s));
}
__device__ __forceinline__ void store_meta(float* meta, uint32_t pair, float s, float mn, int meta16) {
  if (meta16) {
    reinterpret_cast<__half2*>(meta)[pair] = __floats2half2_rn(s, mn);  // both already binary16 values
  } else {
    *reinterpret_cast<float2*>(meta + pair * 2) = make_float2(s, mn);
  }
}

// (scale, min) as stored: what the second pass reads back for the values near a tie
__device__ __forceinline__ void load_meta(const float* meta, uint32_t pair, int meta16, float& s, float& mn) {
  if (meta16) {
    const float2 t = __half22float2(reinterpret_cast<const __half2*>(meta)[pair]);
    s = t.x, mn = t.y;
  } else {
    const float2 t = *reinterpret_cast<const float2*>(meta + pair * 2);
    s = t.x, mn = t.y;
  }
}

// the metadata of pair number `pairs` onward
__device__ __forceinline__ float* meta_from(float* meta, size_t pairs, int meta16) {
  return reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(meta) + pairs * (meta16 ? 4 : 8));
}

constexpr int kListCap = 2048;  // deferred items of a CTA (16 bits each)

template <int DT, int HP>  // HP: KV heads of a CTA's tile (1 or 2)
__global__ void __launch_bounds__(kThreads, 3)
    quantize_batch_kernel(const QuantJob* __restrict__ jobs, ModelDims m, const double* __restrict__ inv_freq,
                          uint32_t* __restrict__ status) {
  constexpr int W = HP * kD;            // channels of the tile
  constexpr int NQ = W / 4;             // channel quads of the tile (keys: one thread each)
  constexpr int kParts = kThreads / NQ; // keys: parts of the tokens (4 or 8)
  constexpr int kTokPer = kTokens / kParts;  // keys: tokens of a part (32 or 16)
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bar[4];  // one per quarter of the tokens: work starts when the first has landed
  // keys: extremes of every (part, quad) while the parts of a group exchange them; afterwards, and for
  // values from the start, s_mn holds the list of deferred items and s_mx the rotation coefficients of every quad
  __shared__ float4 s_mn[kThreads], s_mx[kThreads];
  __shared__ uint32_t s_n;                  // deferred items so far
  uint16_t* s_list = reinterpret_cast<uint16_t*>(s_mn);  // kListCap items
  static_assert(kListCap * sizeof(uint16_t) <= sizeof(float4) * kThreads, "the list overlays s_mn");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = m.Hkv;
  const int n_hp = H / HP;
  pdl_wait();  // the job table comes from the kernel before this one
  int item = blockIdx.x;
  const int hb = (item % n_hp) * HP;      // first head
  item /= n_hp;
  const int kv = item & 1;
  const int l = (item >> 1) % m.L;
  const QuantJob jb = jobs[(item >> 1) / m.L];
  const uint16_t* x = static_cast<const uint16_t*>(kv ? jb.v : jb.k);
  if (!x) return;  // this side of the chunk is not wanted
  uint8_t* codes = static_cast<uint8_t*>(kv ? jb.v_codes : jb.k_codes);
  float* meta = static_cast<float*>(kv ? jb.v_meta : jb.k_meta);
  const int bits = jb.bits;
  const float levels = (float)((1 << bits) - 1);
  const int E = H * kD;                   // elements of a token row
  const size_t layer_elems = (size_t)kTokens * E;

  // ------------------------------ the tile [128 tokens][HP heads][128 channels] into shared memory,
  //                                all of it in flight at once, a barrier per 32 tokens
  constexpr uint32_t row_bytes = (uint32_t)W * 2;  // one token row of the tile
  uint16_t* s_x = reinterpret_cast<uint16_t*>(smem);  // [128][W]
  const uint16_t* tile = x + (size_t)l * layer_elems + (size_t)hb * kD;
  if (tid == 0) {
    for (int q = 0; q < 4; ++q) mbar_init(&bar[q], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_n = 0;
  }
  __syncthreads();
  if (warp == 0) {
    if (lane < 4) mbar_expect_tx(&bar[lane], (uint32_t)(kTokens / 4) * row_bytes);
    __syncwarp();
    if (W == E) {  // the tile is one contiguous block -- four large copies
      if (lane < 4) bulk_g2s(s_x + (size_t)lane * (kTokens / 4) * W, tile + (size_t)lane * (kTokens / 4) * W, (uint32_t)(kTokens / 4) * row_bytes, &bar[lane]);
    } else {       // more heads: one copy per token row (the copy engine's request rate, not its bandwidth, sets the pace)
      for (int t = lane; t < kTokens; t += 32) bulk_g2s(s_x + (size_t)t * W, tile + (size_t)t * E, row_bytes, &bar[t / (kTokens / 4)]);
    }
  }
  // Bounded wait for a quarter of the tokens.  A wait that gives up (never expected) reports it and lets the
  // thread carry on over whatever the tile holds, so that no later barrier of the CTA is left waiting.
  auto wait_quarter = [&](int q) {
    if (!mbar_wait(&bar[q], 0)) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
  };
  // Deferred items.  With 16-bit inputs the quotients of a group lie on a coarse lattice, so that about one
  // value in 250 sits on or next to a tie; taking the IEEE division at once would leave nearly every warp
  // running it with one or two lanes.  Instead the first pass stores the fast codes for everything and notes
  // the places in a bit mask; the threads then put their places on a list of the CTA, and a second pass
  // redoes the listed ones with the IEEE division, one item per thread (a thread whose places
  // found no room on the list redoes them itself).
  auto defer = [&](uint32_t mask, auto&& encode) -> uint32_t {  // returns the places that found no room
    const int n = __popc(mask);
    if (n == 0) return 0;
    uint32_t pos = atomicAdd(&s_n, (uint32_t)n);
    while (mask && pos < (uint32_t)kListCap) {
      s_list[pos++] = (uint16_t)encode(__ffs(mask) - 1);
      mask &= mask - 1;
    }
    return mask;
  };
  auto second_pass = [&](uint32_t left, auto&& encode, auto&& fix) {  // after a __syncthreads()
    const int n = min(s_n, (uint32_t)kListCap);
    for (int i = tid; i < n; i += kThreads) fix((uint32_t)s_list[i]);
    for (; left; left &= left - 1) fix(encode(__ffs(left) - 1));
  };

  if (kv) {
    // ------------------------------ values: eight lanes per (token, head) row, a warp takes four rows at
    // a time.  A lane holds two pieces of eight channels, 8 j .. 8 j + 7 and 64 + 8 j .. 64 + 8 j + 7
    // (two conflict-free 16-byte loads); the extremes are taken on the 16-bit values, two per
    // instruction, and reduced over the lanes of a group by shuffles of those words.
    auto values = [&](auto bits_tag) {
      constexpr int BITS = decltype(bits_tag)::value;
      constexpr int G = BITS == 8 ? 1 : kD / 32;  // groups of a row: the whole row, or 32 channels each
      constexpr int kPieces = G == 1 ? 1 : 2;     // groups a lane takes part in
      constexpr int kLanes = G == 1 ? 8 : 4;      // lanes of a group
      constexpr int kSweeps = 4 * HP;             // 32 rows, i.e. 32 / HP tokens, per sweep of the CTA
      const int sub = lane >> 3, lj = lane & 7;
      // this layer's rows: row u = token * H + head, 32-bit offsets from here on
      uint8_t* const codes_l = codes + (size_t)l * kTokens * H * (kD * BITS / 8);
      float* const meta_l = meta_from(meta, (size_t)l * kTokens * H * G, jb.meta16);
      // item: row | piece << 8 | lane of the row << 9 | word of the piece << 12 -- two values, two codes
      auto fix = [&](uint32_t it) {
        const int r = it & 255, p = (it >> 8) & 1, jj = (it >> 9) & 7, i = (it >> 12) & 3;
        const uint32_t u = (uint32_t)((r / HP) * H + hb + r % HP);
        float s, mn, a, b;
        load_meta(meta_l, u * G + (G == 1 ? 0 : 2 * p + (jj >> 2)), jb.meta16, s, mn);
        f2_unpack(unpack2<DT>(*reinterpret_cast<const uint32_t*>(s_x + (size_t)r * kD + 64 * p + 8 * jj + 2 * i)), a, b);
        const uint32_t c0 = code_exact(a, mn, s, levels), c1 = code_exact(b, mn, s, levels);
        if (BITS == 8)
          *reinterpret_cast<uint16_t*>(codes_l + u * kD + 64 * p + 8 * jj + 2 * i) = (uint16_t)(c0 | (c1 << 8));
        else
          codes_l[u * (kD / 2) + 32 * p + 4 * jj + i] = (uint8_t)(c0 | (c1 << 4));
      };
      uint32_t near_tie[2] = {0, 0};  // per piece: a bit per (sweep, word), the last one lowest
#pragma unroll 2
      for (int it = 0; it < kSweeps; ++it) {
        if (it % HP == 0) wait_quarter(it / HP);
        const int r = it * 32 + warp * 4 + sub;
        const int t = r / HP, hh = r % HP;
        const uint32_t u = (uint32_t)(t * H + hb + hh);  // (token, head) row of the layer
        const uint4 wa = *reinterpret_cast<const uint4*>(s_x + (size_t)r * kD + 8 * lj);
        const uint4 wb = *reinterpret_cast<const uint4*>(s_x + (size_t)r * kD + 64 + 8 * lj);
        const uint32_t w[2][4] = {{wa.x, wa.y, wa.z, wa.w}, {wb.x, wb.y, wb.z, wb.w}};
        uint32_t lo[2], hi[2];  // per piece: element-wise extremes of its four words
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          lo[p] = min2_16<DT>(min2_16<DT>(w[p][0], w[p][1]), min2_16<DT>(w[p][2], w[p][3]));
          hi[p] = max2_16<DT>(max2_16<DT>(w[p][0], w[p][1]), max2_16<DT>(w[p][2], w[p][3]));
        }
        if (G == 1) {  // one group: both pieces, all eight lanes
          lo[0] = min2_16<DT>(lo[0], lo[1]);
          hi[0] = max2_16<DT>(hi[0], hi[1]);
        }
        int32_t limit[2];
        uint64_t mn2[2], inv2[2];
#pragma unroll
        for (int p = 0; p < kPieces; ++p) {
#pragma unroll
          for (int o = 1; o < kLanes; o <<= 1) {
            lo[p] = min2_16<DT>(lo[p], __shfl_xor_sync(0xffffffffu, lo[p], o));
            hi[p] = max2_16<DT>(hi[p], __shfl_xor_sync(0xffffffffu, hi[p], o));
          }
          float a, b, c, d, s;
          f2_unpack(unpack2<DT>(lo[p]), a, b);
          f2_unpack(unpack2<DT>(hi[p]), c, d);
          float mn = fminf(a, b);
          group_params(mn, fmaxf(c, d), levels, jb.meta16, s);
          const int g = G == 1 ? 0 : 2 * p + (lj >> 2);  // channels 8 lj (+ 64) lie in group lj / 4 (+ 2)
          if ((lj & (kLanes - 1)) == 0) store_meta(meta_l, u * G + g, s, mn, jb.meta16);
          const float inv = rcp_approx(s);
          mn2[p] = f2_pack(mn, mn);
          inv2[p] = f2_pack(inv, inv);
          limit[p] = trust_limit(s, levels);
        }
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          const int pp = G == 1 ? 0 : p;
          float mq[4][2], rq[4][2];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float dev = code_fast2(unpack2<DT>(w[p][i]), mn2[pp], inv2[pp], mq[i][0], mq[i][1], rq[i][0], rq[i][1]);
            near_tie[p] = mark_near_tie(near_tie[p], dev, limit[pp]);
          }
          if (BITS == 8) {
            *reinterpret_cast<uint2*>(codes_l + u * kD + 64 * p + 8 * lj) =
                make_uint2(pack4_u8(mq[0][0], mq[0][1], mq[1][0], mq[1][1]), pack4_u8(mq[2][0], mq[2][1], mq[3][0], mq[3][1]));
          } else {
            *reinterpret_cast<uint32_t*>(codes_l + u * (kD / 2) + 32 * p + 4 * lj) =
                pack4_u8(pack2_u4(mq[0][0], rq[0][1]), pack2_u4(mq[1][0], rq[1][1]), pack2_u4(mq[2][0], rq[2][1]), pack2_u4(mq[3][0], rq[3][1]));
          }
        }
      }
      auto place0 = [&](int b) {  // bit b: sweep and word number 4 * kSweeps - 1 - b
        const int n = 4 * kSweeps - 1 - b;
        return (uint32_t)((n >> 2) * 32 + warp * 4 + sub) | (lj << 9) | ((n & 3) << 12);
      };
      auto place1 = [&](int b) { return place0(b) | (1u << 8); };
      const uint32_t left0 = defer(near_tie[0], place0), left1 = defer(near_tie[1], place1);
      __syncthreads();
      second_pass(left0, place0, fix);
      for (uint32_t left = left1; left; left &= left - 1) fix(place1(__ffs(left) - 1));
    };
    if (bits == 8) values(std::integral_constant<int, 8>{});
    else values(std::integral_constant<int, 4>{});
    return;
  }

  // ------------------------------ keys: a thread per QUAD of neighbouring channels and part of the tokens.
  // One eight-byte load brings a token's four values; the extremes are taken on the 16-bit values
  // (two per instruction; on the rotated float32 values with `unrotate`), subtract, scale and round
  // run as packed float32 pairs, and a token's four codes leave with one store.
  const int quad = tid % NQ;                 // tile channels 4 quad .. 4 quad + 3
  const int part = tid / NQ;                 // tokens part * kTokPer .. + kTokPer - 1
  const uint2* s_q = reinterpret_cast<const uint2*>(s_x);  // [128][NQ] word pairs of four channels

  auto keys = [&](auto bits_tag, auto rot_tag) {
    constexpr int BITS = decltype(bits_tag)::value;
    constexpr bool ROT = decltype(rot_tag)::value;
    constexpr int kGroupTokens = BITS == 8 ? kTokens : 32;  // one group per chunk, or groups of 32 tokens
    constexpr int G = kTokens / kGroupTokens;
    constexpr int kPartsPerGroup = kGroupTokens / kTokPer;
    constexpr int kBatch = 4;
    const uint32_t row_stride = (uint32_t)E * BITS / 8;  // bytes of a token row of the layer's codes
    uint8_t* const out_tile = codes + (((size_t)l * layer_elems + (size_t)hb * kD) * BITS) / 8;  // 32-bit offsets from here on
    float* const meta_l = meta_from(meta, (size_t)l * G * H * kD, jb.meta16);
    float4 cs4 = make_float4(0.f, 0.f, 0.f, 0.f), sn4 = cs4;
    if (ROT) {  // channel j pairs with j + 64: low half + x_hi * s, high half - x_lo * s
      const int j = (4 * quad) % kD;
      float cs[4], sn[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        double s_d, c_d;
        sincos((double)jb.unrotate_from * inv_freq[(j + i) & 63], &s_d, &c_d);
        cs[i] = (float)c_d;
        sn[i] = j < 64 ? (float)s_d : -(float)s_d;
      }
      cs4 = make_float4(cs[0], cs[1], cs[2], cs[3]);
      sn4 = make_float4(sn[0], sn[1], sn[2], sn[3]);
    }
    // the four values of token t, quad qd, as two packed pairs (c, s: the quad's rotation coefficients)
    auto value4 = [&](int t, int qd, const float4& c, const float4& s, uint64_t& v01, uint64_t& v23) {
      const uint2 w = s_q[t * NQ + qd];
      v01 = unpack2<DT>(w.x), v23 = unpack2<DT>(w.y);
      if (ROT) {  // per value: fma(x, c, x_partner * s), as the one-chunk form
        const uint2 wp = s_q[t * NQ + (qd ^ 16)];
        v01 = f2_fma(v01, f2_pack(c.x, c.y), f2_mul(unpack2<DT>(wp.x), f2_pack(s.x, s.y)));
        v23 = f2_fma(v23, f2_pack(c.z, c.w), f2_mul(unpack2<DT>(wp.y), f2_pack(s.z, s.w)));
      }
    };
    // item: token | quad << 7 -- the token's four codes of that quad, redone with the IEEE division against
    // the (scale, min) the group stored
    auto fix = [&](uint32_t it) {
      const int t = it & 127, qd = it >> 7;
      const int h = hb + (4 * qd) / kD, j = (4 * qd) % kD;
      const uint32_t pair = (uint32_t)(((t / kGroupTokens) * H + h) * kD + j);
      uint64_t v01, v23;
      if (ROT) value4(t, qd, s_mx[qd], s_mx[NQ + qd], v01, v23);
      else value4(t, qd, cs4, sn4, v01, v23);
      float v[4];
      f2_unpack(v01, v[0], v[1]);
      f2_unpack(v23, v[2], v[3]);
      uint32_t w = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float s, mn;
        load_meta(meta_l, pair + e, jb.meta16, s, mn);
        w |= code_exact(v[e], mn, s, levels) << (BITS * e);
      }
      uint8_t* o = out_tile + (uint32_t)t * row_stride + (uint32_t)(4 * qd * BITS) / 8;
      if (BITS == 8) *reinterpret_cast<uint32_t*>(o) = w;
      else *reinterpret_cast<uint16_t*>(o) = (uint16_t)w;
    };
    // ---- extremes of this part's tokens
    const int t0 = part * kTokPer;
    wait_quarter(t0 / (kTokens / 4));
    float mn[4], mx[4];
    if (!ROT) {
      uint2 lo = s_q[t0 * NQ + quad], hi = lo;
#pragma unroll 8
      for (int t = t0 + 1; t < t0 + kTokPer; ++t) {
        const uint2 w = s_q[t * NQ + quad];
        lo.x = min2_16<DT>(lo.x, w.x), lo.y = min2_16<DT>(lo.y, w.y);
        hi.x = max2_16<DT>(hi.x, w.x), hi.y = max2_16<DT>(hi.y, w.y);
      }
      f2_unpack(unpack2<DT>(lo.x), mn[0], mn[1]);
      f2_unpack(unpack2<DT>(lo.y), mn[2], mn[3]);
      f2_unpack(unpack2<DT>(hi.x), mx[0], mx[1]);
      f2_unpack(unpack2<DT>(hi.y), mx[2], mx[3]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) mn[i] = INFINITY, mx[i] = -INFINITY;
#pragma unroll 4
      for (int t = t0; t < t0 + kTokPer; ++t) {
        uint64_t v01, v23;
        value4(t, quad, cs4, sn4, v01, v23);
        float v[4];
        f2_unpack(v01, v[0], v[1]);
        f2_unpack(v23, v[2], v[3]);
#pragma unroll
        for (int i = 0; i < 4; ++i) mn[i] = fminf(mn[i], v[i]), mx[i] = fmaxf(mx[i], v[i]);
      }
    }
    // ---- the parts of a group exchange their extremes
    s_mn[part * NQ + quad] = make_float4(mn[0], mn[1], mn[2], mn[3]);
    s_mx[part * NQ + quad] = make_float4(mx[0], mx[1], mx[2], mx[3]);
    __syncthreads();
    const int g = part / kPartsPerGroup;
#pragma unroll
    for (int q = 0; q < kPartsPerGroup; ++q) {
      const float4 a = s_mn[(g * kPartsPerGroup + q) * NQ + quad], b = s_mx[(g * kPartsPerGroup + q) * NQ + quad];
      mn[0] = fminf(mn[0], a.x), mn[1] = fminf(mn[1], a.y), mn[2] = fminf(mn[2], a.z), mn[3] = fminf(mn[3], a.w);
      mx[0] = fmaxf(mx[0], b.x), mx[1] = fmaxf(mx[1], b.y), mx[2] = fmaxf(mx[2], b.z), mx[3] = fmaxf(mx[3], b.w);
    }
    float s[4];
    int32_t limit = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      group_params(mn[i], mx[i], levels, jb.meta16, s[i]);
      limit = min(limit, trust_limit(s[i], levels));
    }
    if (part % kPartsPerGroup == 0) {
      const uint32_t pair = (uint32_t)((g * H + hb + (4 * quad) / kD) * kD + (4 * quad) % kD);
#pragma unroll
      for (int i = 0; i < 4; ++i) store_meta(meta_l, pair + i, s[i], mn[i], jb.meta16);
    }
    // ---- first pass: the fast codes of every token, kBatch tokens at a time; a bit per token near a tie
    const uint64_t mn01 = f2_pack(mn[0], mn[1]), mn23 = f2_pack(mn[2], mn[3]);
    const uint64_t inv01 = f2_pack(rcp_approx(s[0]), rcp_approx(s[1])), inv23 = f2_pack(rcp_approx(s[2]), rcp_approx(s[3]));
    uint32_t out = (uint32_t)t0 * row_stride + (uint32_t)(4 * quad * BITS) / 8;  // offset in out_tile
    uint32_t near_tie = 0;  // a bit per token, the last one lowest
#pragma unroll 1
    for (int tb = 0; tb < kTokPer; tb += kBatch, out += kBatch * row_stride) {
      uint32_t cw[kBatch];
#pragma unroll
      for (int i = 0; i < kBatch; ++i) {
        uint64_t v01, v23;
        value4(t0 + tb + i, quad, cs4, sn4, v01, v23);
        float ma[2], mb[2], ra[2], rb[2];
        const float dev = fmaxf(code_fast2(v01, mn01, inv01, ma[0], ma[1], ra[0], ra[1]), code_fast2(v23, mn23, inv23, mb[0], mb[1], rb[0], rb[1]));
        near_tie = mark_near_tie(near_tie, dev, limit);
        if (BITS == 8)
          cw[i] = pack4_u8(ma[0], ma[1], mb[0], mb[1]);
        else
          cw[i] = __float_as_uint(fmaf(pack2_u4(rb[0], rb[1]), 256.f, pack2_u4(ma[0], ra[1])));  // low 16 bits
      }
#pragma unroll
      for (int i = 0; i < kBatch; ++i) {
        if (BITS == 8)
          *reinterpret_cast<uint32_t*>(out_tile + (out + i * row_stride)) = cw[i];
        else
          *reinterpret_cast<uint16_t*>(out_tile + (out + i * row_stride)) = (uint16_t)cw[i];
      }
    }
    // ---- second pass.  The exchange arrays are free once every thread has read them.
    __syncthreads();
    if (ROT && part == 0) s_mx[quad] = cs4, s_mx[NQ + quad] = sn4;
    auto place = [&](int b) { return (uint32_t)(t0 + kTokPer - 1 - b) | ((uint32_t)quad << 7); };
    const uint32_t left = defer(near_tie, place);
    __syncthreads();
    second_pass(left, place, fix);
  };
  using std::integral_constant;
  const bool rot = jb.unrotate_from >= 0;
  if (bits == 8) {
    if (rot) keys(integral_constant<int, 8>{}, integral_constant<bool, true>{});
    else keys(integral_constant<int, 8>{}, integral_constant<bool, false>{});
  } else {
    if (rot) keys(integral_constant<int, 4>{}, integral_constant<bool, true>{});
    else keys(integral_constant<int, 4>{}, integral_constant<bool, false>{});
  }
}

size_t quantize_smem(int hp) { return (size_t)kTokens * hp * kD * 2; }  // the 16-bit tile

template <int DT, int HP>
cudaError_t configure_one() {
  return cudaFuncSetAttribute(quantize_batch_kernel<DT, HP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem(HP));
}

}  // namespace

cudaError_t quantize_configure() {
  cudaError_t e = configure_one<KVB_DT_BF16, 1>();
  if (e == cudaSuccess) e = configure_one<KVB_DT_BF16, 2>();
  if (e == cudaSuccess) e = configure_one<KVB_DT_F16, 1>();
  if (e == cudaSuccess) e = configure_one<KVB_DT_F16, 2>();
  return e;
}

cudaError_t launch_quantize_batch(const QuantJob* jobs, int n_jobs, const ModelDims& m, const double* inv_freq, uint32_t* status,
                                  bool pdl, cudaStream_t st) {
  const int hp = m.Hkv < 2 ? 1 : 2;
  const dim3 grid((unsigned)n_jobs * m.L * 2 * (m.Hkv / hp)), block(kThreads);
  const bool bf16 = m.dtype == KVB_DT_BF16;
  if (hp == 2) {
    if (bf16) return launch_pdl(pdl, quantize_batch_kernel<KVB_DT_BF16, 2>, grid, block, quantize_smem(2), st, jobs, m, inv_freq, status);
    return launch_pdl(pdl, quantize_batch_kernel<KVB_DT_F16, 2>, grid, block, quantize_smem(2), st, jobs, m, inv_freq, status);
  }
  if (bf16) return launch_pdl(pdl, quantize_batch_kernel<KVB_DT_BF16, 1>, grid, block, quantize_smem(1), st, jobs, m, inv_freq, status);
  return launch_pdl(pdl, quantize_batch_kernel<KVB_DT_F16, 1>, grid, block, quantize_smem(1), st, jobs, m, inv_freq, status);
}

}  // namespace kvb
