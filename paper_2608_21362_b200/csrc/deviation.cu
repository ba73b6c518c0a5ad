// Cosine deviation (Algorithm 2, step 2): for every position t,
//     delta_t = 1 - mean over layers, KV heads (and K/V) of cos(stored row, fresh row).
//
// Pure streaming: every 256-byte (token, head) row of the stitched buffer and of the fresh
// tensor is read once with 16-byte loads, a half-warp per row, 8 elements per lane.  Each
// row pair yields ||a-b||^2, ||a||^2 and ||b||^2 (float32, warp-shuffle reduced), and
//     1 - cos = (||a-b||^2 - (||a|| - ||b||)^2) / (2 ||a|| ||b||),
//     ||a|| - ||b|| = (||a||^2 - ||b||^2) / (||a|| + ||b||),
// which has no cancellation for nearly equal rows (1 - dot/(|a||b|) in float32 does).
// The per-row terms are summed over layers, heads and K/V in 2^-40 fixed point with integer
// atomics, so the sum is exact and independent of the order CTAs run in.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "deviation_math.cuh"
#include "f32x2.cuh"
#include "kvb_internal.h"

namespace kvb {
namespace {

constexpr int kThreads = 256;
constexpr int kTileTokens = 64;

// grid (tiles over all requests, L).  A tile is kTileTokens consecutive positions of one request.
template <int DT>
__global__ void __launch_bounds__(kThreads)
    deviation_kernel(const ReqDesc* __restrict__ reqs, int n_req, ModelDims m, int which,
                     unsigned long long* __restrict__ acc) {
  // request of this tile: last r with tile_offset <= tile
  const int tile = blockIdx.x;
  int lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].tile_offset <= tile) lo = mid; else hi = mid - 1;
  }
  const ReqDesc rq = reqs[lo];
  const int l = blockIdx.y;
  const int H = m.Hkv;
  const int t_begin = (tile - rq.tile_offset) * kTileTokens;
  const int t_end = min(rq.T, t_begin + kTileTokens);
  const int u_begin = t_begin * H, u_end = t_end * H;  // (token, head) rows of 256 bytes
  const size_t plane = (size_t)rq.T * H * 256;           // bytes of one [T][H][d] plane, d = 128
  const uint8_t* stK = rq.kv_buf + (size_t)(2 * l) * plane;
  const uint8_t* frK = rq.fresh + (size_t)(2 * l) * plane;
  const bool useK = which & 1, useV = which & 2;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int s = lane >> 4, ln = lane & 15;
  const int n_hw = (kThreads / 32) * 2;
  const bool pair_same_token = (H % 2) == 0;  // rows u, u+1 (u even) belong to one token

#pragma unroll 2
  for (int u0 = u_begin + warp * 2; u0 < u_end; u0 += n_hw) {
    const int u = u0 + s;
    const bool live = u < u_end;
    const size_t off = (size_t)u * 256 + (size_t)ln * 16;
    uint4 ak = make_uint4(0, 0, 0, 0), bk = ak, av = ak, bv = ak;
    if (live && useK) {
      ak = __ldcs(reinterpret_cast<const uint4*>(stK + off));
      bk = __ldcs(reinterpret_cast<const uint4*>(frK + off));
    }
    if (live && useV) {
      av = __ldcs(reinterpret_cast<const uint4*>(stK + plane + off));
      bv = __ldcs(reinterpret_cast<const uint4*>(frK + plane + off));
    }
    float kd, ka, kb, vd, va, vb;
    row_sums<DT>(ak, bk, kd, ka, kb);
    row_sums<DT>(av, bv, vd, va, vb);
    // reduce 6 values over the 16 lanes of the half-warp: first step splits K (lanes 0-7) / V (lanes 8-15)
    const bool up = ln & 8;
    float r0 = up ? vd : kd, r1 = up ? va : ka, r2 = up ? vb : kb;
    r0 += __shfl_xor_sync(0xffffffffu, up ? kd : vd, 8);
    r1 += __shfl_xor_sync(0xffffffffu, up ? ka : va, 8);
    r2 += __shfl_xor_sync(0xffffffffu, up ? kb : vb, 8);
#pragma unroll
    for (int o = 4; o >= 1; o >>= 1) {
      r0 += __shfl_xor_sync(0xffffffffu, r0, o);
      r1 += __shfl_xor_sync(0xffffffffu, r1, o);
      r2 += __shfl_xor_sync(0xffffffffu, r2, o);
    }
    // lanes 0-7 hold the key sums of row u, lanes 8-15 the value sums
    float term = one_minus_cos(r0, r1, r2);
    if ((up && !useV) || (!up && !useK) || !live) term = 0.f;
    long long fx = term_to_fixed(term);
    fx += __shfl_xor_sync(0xffffffffu, fx, 8);  // K + V of row u
    if (pair_same_token) {
      fx += __shfl_xor_sync(0xffffffffu, fx, 16);  // both heads of the token
      if (lane == 0 && live) atomicAdd(&acc[rq.tok_offset + u / H], (unsigned long long)fx);
    } else if (ln == 0 && live) {
      atomicAdd(&acc[rq.tok_offset + u / H], (unsigned long long)fx);
    }
  }
}

}  // namespace

int deviation_tile_tokens() { return kTileTokens; }

cudaError_t launch_deviation(const ReqDesc* reqs, int n_req, int total_tiles, const ModelDims& m, int which,
                             unsigned long long* acc, cudaStream_t st) {
  dim3 grid((unsigned)total_tiles, (unsigned)m.L);
  if (m.dtype == KVB_DT_BF16)
    deviation_kernel<KVB_DT_BF16><<<grid, kThreads, 0, st>>>(reqs, n_req, m, which, acc);
  else
    deviation_kernel<KVB_DT_F16><<<grid, kThreads, 0, st>>>(reqs, n_req, m, which, acc);
  return cudaGetLastError();
}

}  // namespace kvb
