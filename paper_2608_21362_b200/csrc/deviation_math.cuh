// Per-row arithmetic of the cosine deviation (Algorithm 2, step 2), shared by the streaming
// deviation kernel and the stitching kernel's fused variant.
//
// A (token, head) row pair a (stored) / b (fresh) yields ||a-b||^2, ||a||^2 and ||b||^2 in
// float32, and
//     1 - cos = (||a-b||^2 - (||a|| - ||b||)^2) / (2 ||a|| ||b||),
//     ||a|| - ||b|| = (||a||^2 - ||b||^2) / (||a|| + ||b||),
// which has no cancellation for nearly equal rows (1 - dot/(|a||b|) in float32 does).
// Row terms are summed in 2^-40 fixed point with integer atomics (exact, order independent).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "f32x2.cuh"
#include "kvb.h"

namespace kvb {


// One 32-bit word holds two 16-bit values: unpack them into a packed float32 pair.
template <int DT>
__device__ __forceinline__ uint64_t unpack_pair(uint32_t w) {
  if (DT == KVB_DT_BF16) return f2_pack(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
  const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w));
  return f2_pack(t.x, t.y);
}

// ||a-b||^2, ||a||^2, ||b||^2 over 8 elements (four words each side), in packed float32 pairs
template <int DT>
__device__ __forceinline__ void row_sums4(const uint32_t (&aw)[4], const uint32_t (&bw)[4], float& d2, float& na2,
                                          float& nb2) {
  uint64_t sd = 0ull, sa = 0ull, sb = 0ull;  // bit pattern of (+0, +0)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint64_t x = unpack_pair<DT>(aw[i]), y = unpack_pair<DT>(bw[i]);
    const uint64_t df = f2_sub(x, y);
    sd = f2_fma(df, df, sd);
    sa = f2_fma(x, x, sa);
    sb = f2_fma(y, y, sb);
  }
  d2 = f2_hsum(sd);
  na2 = f2_hsum(sa);
  nb2 = f2_hsum(sb);
}

template <int DT>
__device__ __forceinline__ void row_sums(const uint4& a, const uint4& b, float& d2, float& na2, float& nb2) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  row_sums4<DT>(aw, bw, d2, na2, nb2);
}

__device__ __forceinline__ float sqrt_fast(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_fast(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The square root and the two reciprocals are the hardware approximations (one instruction each,
// relative error about 2^-22): the term's error stays at the level of the float32 sums it is built
// from, and the full-precision forms would cost three times the instructions of the whole formula.
__device__ __forceinline__ float one_minus_cos(float d2, float na2, float nb2) {
  if (d2 == 0.f) return 0.f;                 // identical rows (zero rows included): cos = 1
  if (na2 == 0.f || nb2 == 0.f) return 1.f;  // one zero row: cos = 0
  const float na = sqrt_fast(na2), nb = sqrt_fast(nb2);
  const float dn = (na2 - nb2) * rcp_fast(na + nb);
  const float r = (d2 - dn * dn) * rcp_fast(2.f * na * nb);
  return fminf(fmaxf(r, 0.f), 2.f);
}

// A row term in the accumulator's 2^-40 fixed point.  The term lies in [0, 2]: it is rounded to
// 2^-30 units with a 32-bit conversion (one instruction; a 64-bit conversion is several) and shifted,
// which keeps 9e-10 of absolute resolution per term against a float32 delta of at least 1e-7 relative.
__device__ __forceinline__ long long term_to_fixed(float term) {
  return (long long)((unsigned long long)__float2uint_rn(term * 1073741824.0f) << 10);
}

// Two rows per half-warp, each lane holding its partial (d2, na2, nb2) of row A and of row B:
// reduces the six values over the 16 lanes; lanes 0-7 end with row A's sums, lanes 8-15 with row
// B's.  Returns the lane's row term in fixed point (0 where its row is not live) and, through
// na2_row, the squared norm of the lane's stored row.
__device__ __forceinline__ long long pair_terms_fixed(const float (&a)[3], const float (&b)[3], int ln, bool live_a,
                                                      bool live_b, float& na2_row) {
  const bool up = ln & 8;
  float r0 = up ? b[0] : a[0], r1 = up ? b[1] : a[1], r2 = up ? b[2] : a[2];
  r0 += __shfl_xor_sync(0xffffffffu, up ? a[0] : b[0], 8);
  r1 += __shfl_xor_sync(0xffffffffu, up ? a[1] : b[1], 8);
  r2 += __shfl_xor_sync(0xffffffffu, up ? a[2] : b[2], 8);
#pragma unroll
  for (int o = 4; o >= 1; o >>= 1) {
    r0 += __shfl_xor_sync(0xffffffffu, r0, o);
    r1 += __shfl_xor_sync(0xffffffffu, r1, o);
    r2 += __shfl_xor_sync(0xffffffffu, r2, o);
  }
  na2_row = r1;
  float term = one_minus_cos(r0, r1, r2);
  if (up ? !live_b : !live_a) term = 0.f;
  return term_to_fixed(term);
}
__device__ __forceinline__ long long pair_terms_fixed(const float (&a)[3], const float (&b)[3], int ln, bool live_a,
                                                      bool live_b) {
  float unused;
  return pair_terms_fixed(a, b, ln, live_a, live_b, unused);
}

}  // namespace kvb
