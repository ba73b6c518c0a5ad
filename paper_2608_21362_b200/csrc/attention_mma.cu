// Selected-row causal attention (Eq. 2), warp-level tensor-core version (mma.sync m16n8k16).
//
// One CTA per (layer, KV head, tile of selected tokens).  A tile packs TOK = 128/rep selected
// tokens times the rep = Hq/Hkv query heads that share the KV head into 128 query rows, so
// every K/V block fetched serves all heads of the group.  Keys are streamed in blocks of 64
// through a double-buffered cp.async pipeline; softmax is the usual running max / running sum
// in float32, row i masked to keys 0..sel[i].
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kvb_internal.h"

namespace kvb {
namespace {

constexpr int kThreads = 256;
constexpr int kRows = 128;   // query rows per CTA
constexpr int kBlockKeys = 64;
constexpr int kD = 128;
constexpr int kRowBytes = kD * 2;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * kRowBytes + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
template <int DT>
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  if (DT == KVB_DT_BF16) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  } else {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  }
}
template <int DT>
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  if (DT == KVB_DT_BF16) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
  } else {
    __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
  }
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
    attn_mma_kernel(const ReqDesc* __restrict__ reqs, int n_req, int total_tiles, ModelDims m, float scale_log2) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* sQ = smem;                          // 128 rows x 256 B
  uint8_t* sK = smem + kRows * kRowBytes;      // 2 x 64 x 256 B
  uint8_t* sV = sK + 2 * kBlockKeys * kRowBytes;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_tile = m.Hkv * m.L;
  const int lin = blockIdx.x;
  const int tile_flat = total_tiles - 1 - lin / per_tile;  // longest tiles first
  const int hk = (lin % per_tile) % m.Hkv;
  const int l = (lin % per_tile) / m.Hkv;
  int lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (reqs[mid].tile_offset <= tile_flat) lo = mid; else hi = mid - 1;
  }
  const ReqDesc rq = reqs[lo];
  const int rep = m.Hq / m.Hkv;
  const int TOK = kRows / rep;
  const int tile = tile_flat - rq.tile_offset;
  const int n_sel = min(*rq.n_sel, rq.sel_capacity);
  const int i_base = tile * TOK;
  if (i_base >= n_sel) return;
  const int T = rq.T;
  const int t_max = min(rq.sel[min(i_base + TOK, n_sel) - 1], T - 1);
  const int nkb = t_max / kBlockKeys + 1;

  const size_t plane = (size_t)T * m.Hkv * kRowBytes;
  const uint8_t* gK = rq.kv_buf + (size_t)(2 * l) * plane + (size_t)hk * kRowBytes;
  const uint8_t* gV = gK + plane;
  const size_t kv_stride = (size_t)m.Hkv * kRowBytes;

  // ---- Q tile
  for (int c = tid; c < kRows * 16; c += kThreads) {
    const int row = c >> 4, chunk = c & 15;
    const int i = i_base + row / rep;
    const int hq = hk * rep + row % rep;
    const bool valid = i < n_sel;
    const uint8_t* src = rq.q + (((size_t)l * rq.sel_capacity + (valid ? i : 0)) * m.Hq + hq) * kRowBytes + chunk * 16;
    cp_async16(smem_u32(sQ) + swz(row, chunk), src, valid);
  }
  auto load_block = [&](int kb, int buf) {
    for (int c = tid; c < kBlockKeys * 16; c += kThreads) {
      const int row = c >> 4, chunk = c & 15;
      const int key = kb * kBlockKeys + row;
      const bool valid = key < T;
      const size_t off = (size_t)(valid ? key : 0) * kv_stride + chunk * 16;
      cp_async16(smem_u32(sK) + buf * kBlockKeys * kRowBytes + swz(row, chunk), gK + off, valid);
      cp_async16(smem_u32(sV) + buf * kBlockKeys * kRowBytes + swz(row, chunk), gV + off, valid);
    }
  };
  load_block(0, 0);
  cp_commit();

  // this thread's two rows and their causal limits
  const int g = lane >> 2, qd = lane & 3;
  const int r0 = warp * 16 + g, r1 = r0 + 8;
  const int i0 = i_base + r0 / rep, i1 = i_base + r1 / rep;
  const int t0 = i0 < n_sel ? rq.sel[i0] : -1;
  const int t1 = i1 < n_sel ? rq.sel[i1] : -1;
  int warp_tmax = max(t0, t1);
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) warp_tmax = max(warp_tmax, __shfl_xor_sync(0xffffffffu, warp_tmax, o));

  float o_acc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
  float mx0 = -INFINITY, mx1 = -INFINITY, sum0 = 0.f, sum1 = 0.f;

  const uint32_t sQ_u = smem_u32(sQ);
  for (int kb = 0; kb < nkb; ++kb) {
    const int buf = kb & 1;
    if (kb + 1 < nkb) load_block(kb + 1, buf ^ 1);
    cp_commit();
    cp_wait<1>();
    __syncthreads();
    if (kb * kBlockKeys <= warp_tmax) {
      const uint32_t sK_u = smem_u32(sK) + buf * kBlockKeys * kRowBytes;
      const uint32_t sV_u = smem_u32(sV) + buf * kBlockKeys * kRowBytes;
      float s_acc[8][4];
#pragma unroll
      for (int i = 0; i < 8; ++i) s_acc[i][0] = s_acc[i][1] = s_acc[i][2] = s_acc[i][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t a[4];
        {
          const int mi = lane >> 3;
          const int row = warp * 16 + (mi & 1) * 8 + (lane & 7);
          ldsm4(sQ_u + swz(row, 2 * ks + (mi >> 1)), a);
        }
#pragma unroll
        for (int np = 0; np < 4; ++np) {
          uint32_t b[4];
          const int mi = lane >> 3;
          const int key = np * 16 + (mi >> 1) * 8 + (lane & 7);
          ldsm4(sK_u + swz(key, 2 * ks + (mi & 1)), b);
          mma16816<DT>(s_acc[2 * np], a, b[0], b[1]);
          mma16816<DT>(s_acc[2 * np + 1], a, b[2], b[3]);
        }
      }
      // scale, mask, running max
      const int key0 = kb * kBlockKeys + 2 * qd;
      float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int key = key0 + nt * 8 + e;
          s_acc[nt][e] = key <= t0 ? s_acc[nt][e] * scale_log2 : -INFINITY;
          s_acc[nt][2 + e] = key <= t1 ? s_acc[nt][2 + e] * scale_log2 : -INFINITY;
          bm0 = fmaxf(bm0, s_acc[nt][e]);
          bm1 = fmaxf(bm1, s_acc[nt][2 + e]);
        }
      }
      bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 1));
      bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 2));
      bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 1));
      bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 2));
      const float nm0 = fmaxf(mx0, bm0), nm1 = fmaxf(mx1, bm1);
      // rows with nothing visible yet keep max = -inf; use 0 as the exponent base there
      const float base0 = nm0 == -INFINITY ? 0.f : nm0, base1 = nm1 == -INFINITY ? 0.f : nm1;
      const float corr0 = exp2f(mx0 - base0), corr1 = exp2f(mx1 - base1);
      mx0 = nm0, mx1 = nm1;
      float ps0 = 0.f, ps1 = 0.f;
      uint32_t pa[4][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const float p00 = exp2f(s_acc[nt][0] - base0), p01 = exp2f(s_acc[nt][1] - base0);
        const float p10 = exp2f(s_acc[nt][2] - base1), p11 = exp2f(s_acc[nt][3] - base1);
        ps0 += p00 + p01;
        ps1 += p10 + p11;
        pa[nt >> 1][(nt & 1) * 2 + 0] = pack2<DT>(p00, p01);
        pa[nt >> 1][(nt & 1) * 2 + 1] = pack2<DT>(p10, p11);
      }
      sum0 = sum0 * corr0 + ps0;
      sum1 = sum1 * corr1 + ps1;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        o_acc[i][0] *= corr0, o_acc[i][1] *= corr0;
        o_acc[i][2] *= corr1, o_acc[i][3] *= corr1;
      }
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
        for (int np = 0; np < 8; ++np) {
          uint32_t b[4];
          const int mi = lane >> 3;
          const int key = ks * 16 + (mi & 1) * 8 + (lane & 7);
          ldsm4_t(sV_u + swz(key, np * 2 + (mi >> 1)), b);
          mma16816<DT>(o_acc[2 * np], pa[ks], b[0], b[1]);
          mma16816<DT>(o_acc[2 * np + 1], pa[ks], b[2], b[3]);
        }
      }
    }
    __syncthreads();
  }
  cp_wait<0>();

  // ---- normalise and store
  sum0 += __shfl_xor_sync(0xffffffffu, sum0, 1);
  sum0 += __shfl_xor_sync(0xffffffffu, sum0, 2);
  sum1 += __shfl_xor_sync(0xffffffffu, sum1, 1);
  sum1 += __shfl_xor_sync(0xffffffffu, sum1, 2);
  const float inv0 = sum0 > 0.f ? 1.f / sum0 : 0.f, inv1 = sum1 > 0.f ? 1.f / sum1 : 0.f;
  const int hq0 = hk * rep + r0 % rep, hq1 = hk * rep + r1 % rep;
  uint8_t* o0 = rq.out + (((size_t)l * rq.sel_capacity + i0) * m.Hq + hq0) * kRowBytes;
  uint8_t* o1 = rq.out + (((size_t)l * rq.sel_capacity + i1) * m.Hq + hq1) * kRowBytes;
#pragma unroll
  for (int nt = 0; nt < 16; ++nt) {
    const int col = nt * 8 + 2 * qd;
    if (i0 < n_sel) *reinterpret_cast<uint32_t*>(o0 + col * 2) = pack2<DT>(o_acc[nt][0] * inv0, o_acc[nt][1] * inv0);
    if (i1 < n_sel) *reinterpret_cast<uint32_t*>(o1 + col * 2) = pack2<DT>(o_acc[nt][2] * inv1, o_acc[nt][3] * inv1);
  }
}

constexpr size_t kSmem = (size_t)kRows * kRowBytes + 4 * (size_t)kBlockKeys * kRowBytes;

}  // namespace

cudaError_t attention_mma_configure() {
  cudaError_t e = cudaFuncSetAttribute(attn_mma_kernel<KVB_DT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_mma_kernel<KVB_DT_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
}

cudaError_t launch_attention_mma(const ReqDesc* reqs, int n_req, int total_tiles, const ModelDims& m, float scale,
                                 cudaStream_t st) {
  const unsigned grid = (unsigned)total_tiles * m.Hkv * m.L;
  const float scale_log2 = scale * 1.4426950408889634f;
  if (m.dtype == KVB_DT_BF16)
    attn_mma_kernel<KVB_DT_BF16><<<grid, kThreads, kSmem, st>>>(reqs, n_req, total_tiles, m, scale_log2);
  else
    attn_mma_kernel<KVB_DT_F16><<<grid, kThreads, kSmem, st>>>(reqs, n_req, total_tiles, m, scale_log2);
  return cudaGetLastError();
}

}  // namespace kvb
