// KV Quantization, Eq. 6 (cache-population side): asymmetric min/max quantisation of cached
// chunks, keys per channel over a token group, values per token over a channel group.
// scale = (max-min)/(2^b-1) and min are float32; the code is rint((x-min)/scale) in float32
// (IEEE subtract, divide, round-half-even), clamped.  A constant group gets scale 1, codes 0.
//
// One launch quantises a batch of chunks: a CTA per (chunk, layer, K|V, pair of KV heads).
//   keys    the CTA's [128 tokens][<= 2 heads][128 channels] tile is fetched into shared memory by
//           bulk copies (four large ones where the tile is contiguous, i.e. up to two KV heads;
//           one per token row otherwise); a thread owns one channel, walks its token groups
//           twice (extremes, then codes) and leaves the codes in a shared-memory tile that the
//           CTA writes out in 16-byte pieces.  With `unrotate` every key is first rotated back
//           by R_theta^(-orig_pos) (Rotary Positional Embeddings, Eq. 3), so that the stored
//           chunk is position-free and re-use at new_pos needs the single rotation by new_pos;
//           cos / sin come from a double-precision angle, the rotation itself is float32 in a
//           fixed order: u = fma(x, c, +-(x_partner * s)).
//   values  the same tile, staged the same way; a warp per (token, head) row, 4 channels per lane.
// The division of the code decision is the hardware reciprocal where that provably gives the
// same integer (the quotient lies away from every half-integer) and the IEEE division otherwise,
// decided per warp so that the common case carries no division at all.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kvb_internal.h"

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

template <int DT>
__device__ __forceinline__ float from16(uint32_t bits16) {
  if (DT == KVB_DT_BF16) return __uint_as_float(bits16 << 16);
  const __half_raw r{(unsigned short)bits16};
  return __half2float(__half(r));
}

// The code of one value: rint((v - mn) / s) clamped to [0, levels], the division being IEEE float32.
// Fast form: q = (v - mn) * (1/s) with the hardware reciprocal is within 2e-7 * q <= 5e-5 of the exact
// quotient, and so is the IEEE quotient (1.5e-5): when q lies further than 2.5e-4 from every
// half-integer both round to the same integer.  q + 2^23 rounds q to that integer (round-half-even,
// as rint does) and leaves it in the low mantissa bits; no clamp is needed, the quotient cannot
// exceed levels by more than a rounding error.  `unsafe` tells the caller that the IEEE division must
// decide instead (about one value in a thousand; NaN or infinite q as well).
struct FastCode {
  uint32_t code;
  bool unsafe;
};
__device__ __forceinline__ FastCode code_fast(float v, float mn, float inv_s) {
  const float t = __fsub_rn(v, mn);
  const float q = t * inv_s;
  const float m = __fadd_rn(q, 8388608.0f);
  const float d = q - __fsub_rn(m, 8388608.0f);
  FastCode r;
  r.code = __float_as_uint(m) & 0x1FFu;
  r.unsafe = !(fabsf(fabsf(d) - 0.5f) >= 2.5e-4f) || !(q <= 300.f);
  return r;
}
// not inlined: the compiler must not evaluate the division speculatively on the common path
__device__ __noinline__ uint32_t code_exact(float v, float mn, float s, float levels) {
  float c = rintf(__fdiv_rn(__fsub_rn(v, mn), s));
  c = fminf(fmaxf(c, 0.f), levels);
  return (uint32_t)c;
}
// 1/s for code_fast; a scale too small for an accurate reciprocal gives NaN, which sends every value
// of the group through the IEEE division
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return x >= 1e-30f ? y : __int_as_float(0x7FC00000);
}

// (scale, min) of a group from its extremes.  Compact metadata: min is rounded down to binary16
// first, the scale is taken against the rounded min and rounded up, so no value leaves the code range.
__device__ __forceinline__ void group_params(float& mn, float mx, float levels, int meta16, float& s) {
  if (meta16) mn = __half2float(__float2half_rd(mn));
  s = mx > mn ? __fdiv_rn(__fsub_rn(mx, mn), levels) : 1.0f;
  if (meta16) s = __half2float(__float2half_ru(s));
}
__device__ __forceinline__ void store_meta(float* meta, size_t pair, float s, float mn, int meta16) {
  if (meta16) {
    reinterpret_cast<__half2*>(meta)[pair] = __floats2half2_rn(s, mn);  // both already binary16 values
  } else {
    *reinterpret_cast<float2*>(meta + pair * 2) = make_float2(s, mn);
  }
}

template <int DT>
__global__ void __launch_bounds__(kThreads)
    quantize_batch_kernel(const QuantJob* __restrict__ jobs, ModelDims m, const double* __restrict__ inv_freq,
                          uint32_t* __restrict__ status) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bar;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = m.Hkv;
  const int hp = H < 2 ? 1 : 2;           // heads of this CTA's tile
  const int n_hp = H / hp;
  int item = blockIdx.x;
  const int hb = (item % n_hp) * hp;      // first head
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

  // ------------------------------ the tile [128 tokens][hp heads][128 channels] through shared memory,
  //                                all of it in flight at once
  const int W = hp * kD;                       // channels of the tile
  const uint32_t row_bytes = (uint32_t)W * 2;  // one token row of the tile
  uint16_t* s_x = reinterpret_cast<uint16_t*>(smem);                    // [128][W]
  uint8_t* s_codes = smem + (size_t)kTokens * row_bytes;                // keys: [128][W * bits / 8]
  const uint16_t* tile = x + (size_t)l * layer_elems + (size_t)hb * kD;
  if (tid == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 0) {
    if (lane == 0) mbar_expect_tx(&bar, (uint32_t)kTokens * row_bytes);
    __syncwarp();
    if (W == E) {  // up to two KV heads: the tile is one contiguous block -- four large copies
      if (lane < 4) bulk_g2s(s_x + (size_t)lane * (kTokens / 4) * W, tile + (size_t)lane * (kTokens / 4) * W, (uint32_t)(kTokens / 4) * row_bytes, &bar);
    } else {       // more heads: one copy per token row (the copy engine's request rate, not its bandwidth, sets the pace)
      for (int t = lane; t < kTokens; t += 32) bulk_g2s(s_x + (size_t)t * W, tile + (size_t)t * E, row_bytes, &bar);
    }
  }

  if (kv) {
    // ------------------------------ values: a warp per (token, head) row, 4 channels per lane
    const int group_ch = bits == 8 ? kD : m.int4_group;
    const int G = kD / group_ch;
    const int lanes_per_group = group_ch / 4;  // 32 (int8, whole row) or 8 (groups of 32 channels)
    const bool ok = mbar_wait(&bar, 0);
    if (!ok) {
      if (tid == 0) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
      return;
    }
    for (int r = warp; r < kTokens * hp; r += kThreads / 32) {
      const int t = r / hp, hh = r % hp;
      const size_t u = (size_t)l * kTokens * H + (size_t)t * H + hb + hh;  // (layer, token, head) row
      const uint2 w = *reinterpret_cast<const uint2*>(s_x + (size_t)t * W + hh * kD + 4 * lane);
      float v[4] = {from16<DT>(w.x & 0xFFFFu), from16<DT>(w.x >> 16), from16<DT>(w.y & 0xFFFFu), from16<DT>(w.y >> 16)};
      float mn = fminf(fminf(v[0], v[1]), fminf(v[2], v[3])), mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
      for (int o = 1; o < lanes_per_group; o <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
      float s;
      group_params(mn, mx, levels, jb.meta16, s);
      const float inv_s = rcp_approx(s);
      if ((lane % lanes_per_group) == 0) store_meta(meta, u * G + (4 * lane) / group_ch, s, mn, jb.meta16);
      uint32_t q[4];
      bool unsafe = false;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const FastCode f = code_fast(v[i], mn, inv_s);
        q[i] = f.code;
        unsafe |= f.unsafe;
      }
      if (__any_sync(0xffffffffu, unsafe)) {  // rare: the whole warp takes the IEEE division
#pragma unroll
        for (int i = 0; i < 4; ++i) q[i] = code_exact(v[i], mn, s, levels);
      }
      if (bits == 8) {
        *reinterpret_cast<uint32_t*>(codes + u * kD + 4 * lane) = q[0] | (q[1] << 8) | (q[2] << 16) | (q[3] << 24);
      } else {
        *reinterpret_cast<uint16_t*>(codes + ((u * kD) >> 1) + 2 * lane) = (uint16_t)(q[0] | (q[1] << 4) | (q[2] << 8) | (q[3] << 12));
      }
    }
    return;
  }

  // ------------------------------ keys: a thread per channel of the tile
  const int group_tokens = bits == 8 ? kTokens : m.int4_group;
  const int G = kTokens / group_tokens;
  const bool rot = jb.unrotate_from >= 0;
  const int c = tid;  // channel of the tile (W <= kThreads)
  float cs = 1.f, sn = 0.f;
  int partner = c;
  if (rot && c < W) {
    const int j = c & 127;  // channel within the head; planes pair j with j + 64
    double s_d, c_d;
    sincos((double)jb.unrotate_from * inv_freq[j & 63], &s_d, &c_d);
    cs = (float)c_d;
    sn = j < 64 ? (float)s_d : -(float)s_d;  // low half: + x_hi * s; high half: - x_lo * s
    partner = c ^ 64;
  }
  const bool ok = mbar_wait(&bar, 0);
  if (!ok && tid == 0) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
  if (ok && c < W) {
    auto value = [&](int t) {
      const float v = from16<DT>(s_x[(size_t)t * W + c]);
      if (!rot) return v;
      return fmaf(v, cs, __fmul_rn(from16<DT>(s_x[(size_t)t * W + partner]), sn));
    };
    const int h = hb + c / kD, j = c % kD;
    for (int g = 0; g < G; ++g) {
      float mn = INFINITY, mx = -INFINITY;
#pragma unroll 8
      for (int t = g * group_tokens; t < (g + 1) * group_tokens; ++t) {
        const float v = value(t);
        mn = fminf(mn, v);
        mx = fmaxf(mx, v);
      }
      float s;
      group_params(mn, mx, levels, jb.meta16, s);
      const float inv_s = rcp_approx(s);
      store_meta(meta, (((size_t)l * G + g) * H + h) * kD + j, s, mn, jb.meta16);
#pragma unroll 8
      for (int t = g * group_tokens; t < (g + 1) * group_tokens; ++t) {
        const float v = value(t);
        const FastCode f = code_fast(v, mn, inv_s);
        uint32_t q = f.code;
        if (__any_sync(0xffffffffu, f.unsafe)) q = code_exact(v, mn, s, levels);  // rare; whole warps are here
        if (bits == 8) {
          s_codes[(size_t)t * W + c] = (uint8_t)q;
        } else {
          const uint32_t other = __shfl_xor_sync(0xffffffffu, q, 1);  // W is a multiple of 32: whole warps are here
          if ((c & 1) == 0) s_codes[((size_t)t * W + c) >> 1] = (uint8_t)(q | (other << 4));
        }
      }
    }
  }
  __syncthreads();
  if (ok) {  // the code tile leaves in 16-byte pieces: a token row of the tile is contiguous in the layer's codes
    const int row_code_bytes = W * bits / 8, pieces = row_code_bytes / 16;
    uint8_t* out = codes + (((size_t)l * layer_elems + (size_t)hb * kD) * bits) / 8;
    for (int i = tid; i < kTokens * pieces; i += kThreads) {
      const int t = i / pieces, p = i % pieces;
      *reinterpret_cast<uint4*>(out + (size_t)t * (E * bits / 8) + p * 16) =
          *reinterpret_cast<const uint4*>(s_codes + (size_t)t * row_code_bytes + p * 16);
    }
  }
}

size_t quantize_smem() { return (size_t)kTokens * 2 * kD * 2 + (size_t)kTokens * 2 * kD; }  // tile + int8 code tile, 2 heads

}  // namespace

cudaError_t quantize_configure() {
  cudaError_t e = cudaFuncSetAttribute(quantize_batch_kernel<KVB_DT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(quantize_batch_kernel<KVB_DT_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)quantize_smem());
}

cudaError_t launch_quantize_batch(const QuantJob* jobs, int n_jobs, const ModelDims& m, const double* inv_freq, uint32_t* status,
                                  cudaStream_t st) {
  const int n_hp = m.Hkv < 2 ? 1 : m.Hkv / 2;
  const unsigned grid = (unsigned)n_jobs * m.L * 2 * n_hp;
  if (m.dtype == KVB_DT_BF16)
    quantize_batch_kernel<KVB_DT_BF16><<<grid, kThreads, quantize_smem(), st>>>(jobs, m, inv_freq, status);
  else
    quantize_batch_kernel<KVB_DT_F16><<<grid, kThreads, quantize_smem(), st>>>(jobs, m, inv_freq, status);
  return cudaGetLastError();
}

}  // namespace kvb
