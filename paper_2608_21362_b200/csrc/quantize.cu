// KV Quantization, Eq. 6 (cache-population side): asymmetric min/max quantisation of one
// chunk, keys per channel over a token group, values per token over a channel group.
// scale = (max-min)/(2^b-1) and min are float32; the code is rint((x-min)/scale) in float32
// (IEEE subtract, divide, round-half-even), clamped.  A constant group gets scale 1, codes 0.
// One CTA per layer; not a bandwidth-tuned kernel (it runs when a chunk enters the cache, not
// on the stitching path).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kvb_internal.h"

namespace kvb {
namespace {

template <int DT>
__device__ __forceinline__ float load16(const uint16_t* p) {
  if (DT == KVB_DT_BF16) return __uint_as_float(((uint32_t)*p) << 16);
  return __half2float(*reinterpret_cast<const __half*>(p));
}

__device__ __forceinline__ uint32_t code_of(float v, float mn, float s, float levels) {
  float c = rintf(__fdiv_rn(__fsub_rn(v, mn), s));
  c = fminf(fmaxf(c, 0.f), levels);
  return (uint32_t)c;
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
    meta[pair * 2 + 0] = s;
    meta[pair * 2 + 1] = mn;
  }
}

// keys: thread = channel (h, j); loops over the tokens of each group.
// ROT: the chunk was encoded at positions orig_pos..; every key is first rotated back by
// R_theta^(-orig_pos) (Rotary Positional Embeddings, Eq. 3), so that the stored chunk is position-free
// and re-use at new_pos needs the single rotation by new_pos.  cos / sin come from a double-precision
// angle, the rotation itself is float32 in a fixed order: u = fma(x, c, +-(x_partner * s)).
template <int DT, bool ROT>
__global__ void quantize_k_kernel(const uint16_t* __restrict__ x, uint8_t* __restrict__ codes, float* __restrict__ meta,
                                  int C, int E, int bits, int group_tokens, int orig_pos, const double* __restrict__ inv_freq,
                                  int meta16) {
  const int l = blockIdx.x;
  const int G = C / group_tokens;
  const float levels = (float)((1 << bits) - 1);
  const uint16_t* xl = x + (size_t)l * C * E;
  uint8_t* cl = codes + (size_t)l * C * E * bits / 8;
  const size_t pair0 = (size_t)l * G * E;  // first (scale, min) pair of this layer
  for (int c = threadIdx.x; c < E; c += blockDim.x) {  // blockDim.x is even and E is even: c keeps its parity
    float cs = 1.f, sn = 0.f;
    int partner = c;
    if (ROT) {
      const int j = c & 127;  // channel within the head (d = 128); planes pair j with j + 64
      double s_d, c_d;
      sincos((double)orig_pos * inv_freq[j & 63], &s_d, &c_d);
      cs = (float)c_d;
      sn = j < 64 ? (float)s_d : -(float)s_d;  // low half: + x_hi * s; high half: - x_lo * s
      partner = c ^ 64;
    }
    auto value = [&](int t) {
      const float v = load16<DT>(xl + (size_t)t * E + c);
      if (!ROT) return v;
      return fmaf(v, cs, __fmul_rn(load16<DT>(xl + (size_t)t * E + partner), sn));
    };
    for (int g = 0; g < G; ++g) {
      float mn = INFINITY, mx = -INFINITY;
      for (int t = g * group_tokens; t < (g + 1) * group_tokens; ++t) {
        const float v = value(t);
        mn = fminf(mn, v);
        mx = fmaxf(mx, v);
      }
      float s;
      group_params(mn, mx, levels, meta16, s);
      store_meta(meta, pair0 + (size_t)g * E + c, s, mn, meta16);
      for (int t = g * group_tokens; t < (g + 1) * group_tokens; ++t) {
        const uint32_t q = code_of(value(t), mn, s, levels);
        if (bits == 8) {
          cl[(size_t)t * E + c] = (uint8_t)q;
        } else {
          const uint32_t other = __shfl_xor_sync(0xffffffffu, q, 1);
          if ((c & 1) == 0) cl[((size_t)t * E + c) >> 1] = (uint8_t)(q | (other << 4));
        }
      }
    }
  }
}

// values: one warp per (token, head) row of 128 channels, 4 channels per lane
template <int DT>
__global__ void quantize_v_kernel(const uint16_t* __restrict__ x, uint8_t* __restrict__ codes, float* __restrict__ meta,
                                  int C, int H, int bits, int group_ch, int meta16) {
  const int l = blockIdx.x;
  const int d = 128;
  const int G = d / group_ch;
  const float levels = (float)((1 << bits) - 1);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  const int lanes_per_group = group_ch / 4;  // 32 (int8, whole row) or 8 (groups of 32 channels)
  for (int u = warp; u < C * H; u += n_warps) {
    const size_t base = ((size_t)l * C * H + u) * d;
    float v[4];
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[i] = load16<DT>(x + base + 4 * lane + i);
      mn = fminf(mn, v[i]);
      mx = fmaxf(mx, v[i]);
    }
    for (int o = 1; o < lanes_per_group; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    float s;
    group_params(mn, mx, levels, meta16, s);
    const int g = (4 * lane) / group_ch;
    if ((lane % lanes_per_group) == 0) store_meta(meta, ((size_t)l * C * H + u) * G + g, s, mn, meta16);
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) q[i] = code_of(v[i], mn, s, levels);
    if (bits == 8) {
      *reinterpret_cast<uint32_t*>(codes + base + 4 * lane) = q[0] | (q[1] << 8) | (q[2] << 16) | (q[3] << 24);
    } else {
      *reinterpret_cast<uint16_t*>(codes + (base >> 1) + 2 * lane) =
          (uint16_t)(q[0] | (q[1] << 4) | (q[2] << 8) | (q[3] << 12));
    }
  }
}

}  // namespace

cudaError_t launch_quantize(const void* x, int is_value, int bits, void* codes, void* meta, const ModelDims& m,
                            int unrotate, int orig_pos, const double* inv_freq, int meta16, cudaStream_t st) {
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  uint8_t* cp = static_cast<uint8_t*>(codes);
  float* mp = static_cast<float*>(meta);
  const int E = m.Hkv * m.d;
  const bool bf = m.dtype == KVB_DT_BF16;
  if (!is_value) {
    const int gt = bits == 8 ? m.C : m.int4_group;
    if (unrotate) {
      if (bf)
        quantize_k_kernel<KVB_DT_BF16, true><<<m.L, 256, 0, st>>>(xp, cp, mp, m.C, E, bits, gt, orig_pos, inv_freq, meta16);
      else
        quantize_k_kernel<KVB_DT_F16, true><<<m.L, 256, 0, st>>>(xp, cp, mp, m.C, E, bits, gt, orig_pos, inv_freq, meta16);
    } else {
      if (bf)
        quantize_k_kernel<KVB_DT_BF16, false><<<m.L, 256, 0, st>>>(xp, cp, mp, m.C, E, bits, gt, 0, nullptr, meta16);
      else
        quantize_k_kernel<KVB_DT_F16, false><<<m.L, 256, 0, st>>>(xp, cp, mp, m.C, E, bits, gt, 0, nullptr, meta16);
    }
  } else {
    const int gc = bits == 8 ? m.d : m.int4_group;
    if (bf)
      quantize_v_kernel<KVB_DT_BF16><<<m.L, 256, 0, st>>>(xp, cp, mp, m.C, m.Hkv, bits, gc, meta16);
    else
      quantize_v_kernel<KVB_DT_F16><<<m.L, 256, 0, st>>>(xp, cp, mp, m.C, m.Hkv, bits, gc, meta16);
  }
  return cudaGetLastError();
}

}  // namespace kvb
