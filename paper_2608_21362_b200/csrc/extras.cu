// Two small HBM-bound steps next to the main path:
//   patch       Algorithm 2 step 4 / Algorithm 1 splice: the K and V rows of every selected
//               position, in every layer, are replaced by the freshly projected ones
//   importance  Eq. 7: mean L2 norm of a chunk's keys (the eviction score of the cache manager),
//               read from the stitched buffer (rotation leaves norms unchanged); two launches
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "f32x2.cuh"
#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

constexpr int kThreads = 256;
constexpr int kPatchCtasPerSm = 4;  // measured: 4 CTAs per SM x 4 rows in flight per warp; 8 rows per warp was 15 % slower

// A fixed grid of warps.  A warp owns one 512-byte piece of the row of one plane (layer x K|V) and
// every rows_par-th selected row; it takes four rows at a time: four independent index loads, then
// four 16-byte loads per lane, then the stores -- the step is a chain of dependent loads, so what
// counts is how many are in flight (and that no division sits between them).  The number of selected
// rows is only known on the device; no CTA is launched for the unused part of a selection's capacity.
// `fetch(r)` returns request r's descriptor: from the kernel's own arguments for up to kPatchInline
// requests (no upload and no second launch), from a table in device memory beyond that.
template <typename Fetch>
__device__ __forceinline__ void patch_body(Fetch fetch, int n_req, const ModelDims& m) {
  constexpr int kUnroll = 4;
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t n_warps = gridDim.x * (kThreads / 32);
  const uint32_t gw = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  const uint32_t row_bytes = (uint32_t)m.Hkv * 256;
  const uint32_t pieces = row_bytes >= 512 ? row_bytes / 512 : 1;  // a 256-byte row: half a warp
  const uint32_t piece_bytes = row_bytes / pieces;
  const uint32_t n_pp = (uint32_t)m.L * 2 * pieces;                // (plane, piece) pairs
  const uint32_t pp_warps = n_warps >= n_pp ? n_pp : n_warps;      // warps along that axis
  const uint32_t rows_par = n_warps / pp_warps;                    // rows in flight along the other
  const uint32_t ri = gw / pp_warps;
  if (ri >= rows_par || lane * 16 >= piece_bytes) return;
  for (uint32_t pp = gw % pp_warps; pp < n_pp; pp += pp_warps) {
    const uint32_t pl = pp / pieces, piece = pp % pieces;  // plane = layer * 2 + (0 keys | 1 values)
    for (int r = 0; r < n_req; ++r) {
      const PatchDesc rq = fetch(r);
      const int n_sel = min(*rq.n_sel, rq.sel_capacity);
      const size_t base = (size_t)pl * rq.T * row_bytes + piece * piece_bytes + lane * 16;
      // another starting row per request, so that the last, partly filled round does not always fall to the same warps
      for (int i0 = (int)((ri + (uint32_t)r * 7u) % rows_par); i0 < n_sel; i0 += kUnroll * (int)rows_par) {
        int t[kUnroll];
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) {
          const int i = i0 + k * (int)rows_par;
          t[k] = i < n_sel ? rq.sel[i] : -1;
          if (t[k] >= rq.T) t[k] = -1;
        }
        uint4 v[kUnroll];
#pragma unroll
        for (int k = 0; k < kUnroll; ++k)
          if (t[k] >= 0) v[k] = __ldcs(reinterpret_cast<const uint4*>(rq.fresh + base + (size_t)t[k] * row_bytes));
#pragma unroll
        for (int k = 0; k < kUnroll; ++k)
          if (t[k] >= 0) *reinterpret_cast<uint4*>(rq.kv_buf + base + (size_t)t[k] * row_bytes) = v[k];
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads) patch_inline_kernel(const __grid_constant__ PatchInline a, int n_req, ModelDims m) {
  pdl_wait();  // the selection (and the table) come from the kernels before this one
  patch_body([&](int r) { return a.d[r]; }, n_req, m);
}
__global__ void __launch_bounds__(kThreads) patch_table_kernel(const PatchDesc* __restrict__ table, int n_req, ModelDims m) {
  pdl_wait();
  patch_body([&](int r) { return table[r]; }, n_req, m);
}

__device__ __forceinline__ int request_of(const ReqDesc* __restrict__ reqs, int n_req, int item) {
  int lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].tile_offset <= item) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Eq. 7, first step: a CTA per (chunk, layer) adds up the L2 norms of the chunk-layer's (token, head)
// key rows in a fixed order -- a half-warp per 256-byte row, four rows in flight, the half-warps'
// double-precision sums combined in warp order -- into part[chunk][layer].
template <int DT>
__global__ void __launch_bounds__(kThreads)
    importance_kernel(const ReqDesc* __restrict__ reqs, int n_req, ModelDims m, double* __restrict__ part) {
  constexpr int kUnroll = 4;
  __shared__ double s_part[kThreads / 32];
  const int item = blockIdx.x, l = blockIdx.y;
  pdl_wait();  // the table and the buffer come from the kernels before this one
  const ReqDesc rq = reqs[request_of(reqs, n_req, item)];
  const int chunk = item - rq.tile_offset;
  const int H = m.Hkv, C = m.C;
  const size_t plane = (size_t)rq.T * H * 256;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, s = lane >> 4, ln = lane & 15;
  const int rows = C * H;  // (token, head) rows of the chunk in one layer
  const uint8_t* base = rq.kv_buf + (size_t)(2 * l) * plane + (size_t)chunk * C * H * 256 + ln * 16;
  constexpr int kRowsPerSweep = (kThreads / 32) * 2;
  double acc = 0.0;        // this half-warp's rows, summed in row order
  for (int u0 = warp * 2 + s; u0 < rows; u0 += kUnroll * kRowsPerSweep) {
    uint4 v[kUnroll];
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
      const int u = u0 + k * kRowsPerSweep;
      v[k] = u < rows ? __ldcs(reinterpret_cast<const uint4*>(base + (size_t)u * 256)) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
      const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
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
      float n2 = f2_hsum(sq);
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
      acc += (double)sqrtf(n2);  // a row beyond the chunk adds sqrt(0) = 0
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 16);  // the warp's two half-warps
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int w = 0; w < kThreads / 32; ++w) tot += s_part[w];
    part[(size_t)item * m.L + l] = tot;
  }
}

// Second step: a thread per chunk adds the layers' sums in layer order and takes the mean.
__global__ void importance_mean_kernel(const ReqDesc* __restrict__ reqs, int n_req, int total_chunks, ModelDims m,
                                       const double* __restrict__ part) {
  const int item = blockIdx.x * blockDim.x + threadIdx.x;
  pdl_wait();
  if (item >= total_chunks) return;
  const ReqDesc rq = reqs[request_of(reqs, n_req, item)];
  double tot = 0.0;
  for (int l = 0; l < m.L; ++l) tot += part[(size_t)item * m.L + l];
  rq.delta[item - rq.tile_offset] = (float)(tot / ((double)m.L * m.Hkv * m.C));  // the descriptor's float output slot
}

}  // namespace

cudaError_t launch_patch_inline(const PatchInline& descs, int n_req, int n_sm, const ModelDims& m, bool pdl, cudaStream_t st) {
  return launch_pdl(pdl, patch_inline_kernel, dim3((unsigned)(n_sm * kPatchCtasPerSm)), dim3(kThreads), 0, st, descs, n_req, m);
}

cudaError_t launch_patch_table(const PatchDesc* table, int n_req, int n_sm, const ModelDims& m, bool pdl, cudaStream_t st) {
  return launch_pdl(pdl, patch_table_kernel, dim3((unsigned)(n_sm * kPatchCtasPerSm)), dim3(kThreads), 0, st, table, n_req, m);
}

cudaError_t launch_importance(const ReqDesc* reqs, int n_req, int total_chunks, const ModelDims& m, double* part, bool pdl, cudaStream_t st) {
  const dim3 grid((unsigned)total_chunks, (unsigned)m.L);
  cudaError_t e = m.dtype == KVB_DT_BF16 ? launch_pdl(pdl, importance_kernel<KVB_DT_BF16>, grid, dim3(kThreads), 0, st, reqs, n_req, m, part)
                                         : launch_pdl(pdl, importance_kernel<KVB_DT_F16>, grid, dim3(kThreads), 0, st, reqs, n_req, m, part);
  if (e != cudaSuccess) return e;
  return launch_pdl(pdl, importance_mean_kernel, dim3((unsigned)((total_chunks + 127) / 128)), dim3(128), 0, st, reqs, n_req, total_chunks, m,
                    static_cast<const double*>(part));
}

}  // namespace kvb
