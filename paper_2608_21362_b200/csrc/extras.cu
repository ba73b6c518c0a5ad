// Two small HBM-bound steps next to the main path:
//   patch       Algorithm 2 step 4 / Algorithm 1 splice: the K and V rows of every selected
//               position, in every layer, are replaced by the freshly projected ones
//   importance  Eq. 7: mean L2 norm of a chunk's keys (the eviction score of the cache manager),
//               read from the stitched buffer (rotation leaves norms unchanged)
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "f32x2.cuh"
#include "kvb_internal.h"

namespace kvb {
namespace {

constexpr int kThreads = 256;

// grid (row tiles over all requests, L*2).  One warp copies one [H][d] row (H*256 bytes).
__global__ void __launch_bounds__(kThreads)
    patch_kernel(const ReqDesc* __restrict__ reqs, int n_req, int rows_per_cta, ModelDims m) {
  const int tile = blockIdx.x;
  int lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].tile_offset <= tile) lo = mid; else hi = mid - 1;
  }
  const ReqDesc rq = reqs[lo];
  const int n_sel = min(*rq.n_sel, rq.sel_capacity);
  const int i0 = (tile - rq.tile_offset) * rows_per_cta;
  const int plane_idx = blockIdx.y;  // layer * 2 + (0 keys | 1 values)
  const size_t row_bytes = (size_t)m.Hkv * 256;
  const size_t plane = (size_t)rq.T * row_bytes;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint8_t* dst_plane = const_cast<uint8_t*>(rq.kv_buf) + (size_t)plane_idx * plane;
  const uint8_t* src_plane = rq.fresh + (size_t)plane_idx * plane;
  for (int i = i0 + warp; i < min(i0 + rows_per_cta, n_sel); i += kThreads / 32) {
    const int t = rq.sel[i];
    if (t < 0 || t >= rq.T) continue;
    const uint4* s = reinterpret_cast<const uint4*>(src_plane + (size_t)t * row_bytes);
    uint4* d = reinterpret_cast<uint4*>(dst_plane + (size_t)t * row_bytes);
    for (int c = lane; c < (int)(row_bytes / 16); c += 32) d[c] = __ldcs(s + c);
  }
}

// One CTA per (request, chunk): loops over layers and the chunk's (token, head) rows in a fixed
// order, so the float result is reproducible.  A half-warp reads one 256-byte key row.
template <int DT>
__global__ void __launch_bounds__(kThreads)
    importance_kernel(const ReqDesc* __restrict__ reqs, int n_req, ModelDims m) {
  __shared__ double s_part[kThreads / 32];
  const int item = blockIdx.x;
  int lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].tile_offset <= item) lo = mid; else hi = mid - 1;
  }
  const ReqDesc rq = reqs[lo];
  const int chunk = item - rq.tile_offset;
  const int H = m.Hkv, C = m.C;
  const size_t plane = (size_t)rq.T * H * 256;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, s = lane >> 4, ln = lane & 15;
  const int rows = C * H;  // (token, head) rows of the chunk in one layer
  double acc = 0.0;        // this half-warp's rows, summed in row order
  for (int l = 0; l < m.L; ++l) {
    const uint8_t* base = rq.kv_buf + (size_t)(2 * l) * plane + (size_t)chunk * C * H * 256;
    for (int u0 = warp * 2; u0 < rows; u0 += (kThreads / 32) * 2) {
      const int u = u0 + s;
      float n2 = 0.f;
      if (u < rows) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(base + (size_t)u * 256 + ln * 16));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint64_t sq = 0ull;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint64_t x;
          if (DT == KVB_DT_BF16) {
            x = f2_pack(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
          } else {
            const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            x = f2_pack(t.x, t.y);
          }
          sq = f2_fma(x, x, sq);
        }
        n2 = f2_hsum(sq);
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
      if (u < rows && ln == 0) acc += (double)sqrtf(n2);
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 16);  // the warp's two half-warps
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) tot += s_part[w];
    rq.delta[chunk] = (float)(tot / ((double)m.L * H * C));  // the descriptor's float output slot
  }
}

}  // namespace

cudaError_t launch_patch(const ReqDesc* reqs, int n_req, int total_tiles, int rows_per_cta, const ModelDims& m, cudaStream_t st) {
  dim3 grid((unsigned)total_tiles, (unsigned)(m.L * 2));
  patch_kernel<<<grid, kThreads, 0, st>>>(reqs, n_req, rows_per_cta, m);
  return cudaGetLastError();
}

cudaError_t launch_importance(const ReqDesc* reqs, int n_req, int total_chunks, const ModelDims& m, cudaStream_t st) {
  if (m.dtype == KVB_DT_BF16)
    importance_kernel<KVB_DT_BF16><<<total_chunks, kThreads, 0, st>>>(reqs, n_req, m);
  else
    importance_kernel<KVB_DT_F16><<<total_chunks, kThreads, 0, st>>>(reqs, n_req, m);
  return cudaGetLastError();
}

}  // namespace kvb
