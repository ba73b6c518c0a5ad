// Selection (Algorithm 2 step 3 + the token windows of Algorithm 1), one CTA per request:
//   1. delta_t from the fixed-point sums of the deviation kernel (and clear them for the next call);
//   2. radix select (4 passes of 8 bits over order-preserving integer keys) for the k-th largest
//      delta; ties at the threshold are taken in index order, so the set is the first k of the
//      order (delta descending, index ascending);
//   3. bitonic sort of the k (key, index) pairs -> rank, most deviated first;
//   4. bitmask union with the seam windows, prefix sum -> ascending sel and n_sel.
// All decisions are integer comparisons: the result is a pure function of the float32 delta.
#include "kvb_internal.h"

namespace kvb {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxT = 32768;  // one 32-bit mask word per thread
constexpr int kMaxK = 8192;

// float -> uint32 whose unsigned order is the float order; NaN ranks as +inf, -0 as +0
__device__ __forceinline__ uint32_t order_key(float v) {
  uint32_t u = __float_as_uint(v);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) u = 0x7F800000u;
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// exclusive prefix sum of one value per thread over the CTA; total returned through *total
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* warp_sums, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = warp_sums[lane];
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_sums[lane] = winc - w;  // exclusive
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  const uint32_t res = warp_sums[warp] + inc - v;
  *total = warp_sums[32];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kThreads, 1)
    topk_kernel(const ReqDesc* __restrict__ reqs, const SeamWindow* __restrict__ seams, double inv_terms,
                unsigned long long* __restrict__ acc, int t_pad, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem);                           // [t_pad]
  uint32_t* s_mask = s_keys + t_pad;                                              // [kThreads] selection bitmask
  unsigned long long* s_comp = reinterpret_cast<unsigned long long*>(s_mask + kThreads);  // [k_pad] / histograms
  uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_comp);                         // [kWarps][256], aliases s_comp
  __shared__ uint32_t s_warp_sums[33];
  __shared__ uint32_t s_bins[256];
  __shared__ uint32_t s_sel[2];  // chosen bin, remaining need

  const ReqDesc rq = reqs[blockIdx.x];
  const int T = rq.T, k = min(rq.k, T);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- 1. delta and keys
  for (int t = tid; t < T; t += kThreads) {
    const unsigned long long a = acc[rq.tok_offset + t];
    acc[rq.tok_offset + t] = 0ull;
    const float dl = (float)((double)(long long)a * (1.0 / 1099511627776.0) * inv_terms);
    rq.delta[t] = dl;
    s_keys[t] = order_key(dl);
  }
  s_mask[tid] = 0u;
  __syncthreads();

  // ---- 2. radix select: threshold key `prefix`, and how many keys equal to it are taken (`need`)
  uint32_t prefix = 0, mask = 0, need = (uint32_t)k;
  if (k > 0 && k < T) {
    for (int pass = 3; pass >= 0; --pass) {
      for (int i = tid; i < kWarps * 256; i += kThreads) s_hist[i] = 0;
      __syncthreads();
      const int shift = pass * 8;
      for (int t = tid; t < T; t += kThreads) {
        const uint32_t key = s_keys[t];
        if ((key & mask) == prefix) atomicAdd(&s_hist[warp * 256 + ((key >> shift) & 255u)], 1u);
      }
      __syncthreads();
      if (tid < 256) {
        uint32_t c = 0;
        for (int w = 0; w < kWarps; ++w) c += s_hist[w * 256 + tid];
        s_bins[tid] = c;
      }
      __syncthreads();
      if (warp == 0) {
        // lane j owns bins 255-8j .. 248-8j (descending); find the bin where the running count reaches need
        uint32_t local[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          local[i] = s_bins[255 - (lane * 8 + i)];
          sum += local[i];
        }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t n = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += n;
        }
        uint32_t before = inc - sum;  // keys in strictly larger bins owned by lower lanes
        if (before < need && inc >= need) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (before < need && before + local[i] >= need) {
              s_sel[0] = 255 - (lane * 8 + i);
              s_sel[1] = need - before;
            }
            before += local[i];
          }
        }
      }
      __syncthreads();
      prefix |= s_sel[0] << shift;
      mask |= 255u << shift;
      need = s_sel[1];
      __syncthreads();
    }
  }

  // ---- 3. the top-k set in index order; thread w owns positions 32w .. 32w+31
  uint32_t gt_mask = 0, eq_mask = 0;
  {
    const int base = tid * 32;
    if (k >= T) {
      for (int i = 0; i < 32; ++i)
        if (base + i < T) gt_mask |= 1u << i;
    } else if (k > 0) {
      for (int i = 0; i < 32; ++i) {
        if (base + i < T) {
          const uint32_t key = s_keys[base + i];
          if (key > prefix) gt_mask |= 1u << i;
          if (key == prefix) eq_mask |= 1u << i;
        }
      }
    }
  }
  uint32_t tot_eq, tot_sel;
  const uint32_t eq_before = block_exclusive_scan(__popc(eq_mask), s_warp_sums, &tot_eq);
  uint32_t sel_mask = gt_mask;
  {
    uint32_t e = eq_mask, r = eq_before;
    while (e) {
      const int b = __ffs(e) - 1;
      e &= e - 1;
      if (r < need && k < T) sel_mask |= 1u << b;
      ++r;
    }
  }
  const uint32_t sel_before = block_exclusive_scan(__popc(sel_mask), s_warp_sums, &tot_sel);
  int k_pad = 1;
  while (k_pad < k) k_pad <<= 1;
  // composite sort keys: larger delta first, then lower index
  for (int i = tid; i < k_pad; i += kThreads) s_comp[i] = ~0ull;
  __syncthreads();
  {
    uint32_t e = sel_mask, pos = sel_before;
    while (e) {
      const int b = __ffs(e) - 1;
      e &= e - 1;
      const uint32_t t = tid * 32 + b;
      if (pos < (uint32_t)k_pad) s_comp[pos] = ((unsigned long long)(~s_keys[t]) << 32) | t;
      ++pos;
    }
  }
  s_mask[tid] = sel_mask;
  __syncthreads();

  // ---- bitonic sort of s_comp[0..k_pad)
  for (int size = 2; size <= k_pad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = tid; i < (k_pad >> 1); i += kThreads) {
        const int lo = 2 * i - (i & (stride - 1));
        const int hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned long long a = s_comp[lo], b = s_comp[hi];
        if ((a > b) == up) {
          s_comp[lo] = b;
          s_comp[hi] = a;
        }
      }
      __syncthreads();
    }
  }
  for (int i = tid; i < k; i += kThreads) rq.rank[i] = (int32_t)(uint32_t)(s_comp[i] & 0xFFFFFFFFull);

  // ---- 4. union with the seam windows, ascending list
  for (int w = 0; w < rq.n_seams; ++w) {
    const SeamWindow sw = seams[rq.seam_offset + w];
    for (int t = sw.lo + tid; t < sw.hi; t += kThreads) atomicOr(&s_mask[t >> 5], 1u << (t & 31));
  }
  __syncthreads();
  const uint32_t word = s_mask[tid];
  uint32_t n_sel;
  uint32_t pos = block_exclusive_scan(__popc(word), s_warp_sums, &n_sel);
  {
    uint32_t e = word;
    while (e) {
      const int b = __ffs(e) - 1;
      e &= e - 1;
      if (pos < (uint32_t)rq.sel_capacity) rq.sel[pos] = tid * 32 + b;
      ++pos;
    }
  }
  if (tid == 0) {
    if (n_sel > (uint32_t)rq.sel_capacity) {
      atomicOr(status, DEV_STATUS_SEL_OVERFLOW);
      n_sel = rq.sel_capacity;
    }
    *rq.n_sel = (int32_t)n_sel;
    if (tot_sel != (uint32_t)k) atomicOr(status, DEV_STATUS_BAD_DESC);
  }
}

}  // namespace

int topk_max_T() { return kMaxT; }
int topk_max_k() { return kMaxK; }

static size_t topk_smem(int t_pad, int k_pad) {
  size_t comp = (size_t)k_pad * 8;
  if (comp < (size_t)kWarps * 256 * 4) comp = (size_t)kWarps * 256 * 4;
  return (size_t)t_pad * 4 + kThreads * 4 + comp;
}

cudaError_t topk_configure() {
  return cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)topk_smem(kMaxT, kMaxK));
}

cudaError_t launch_topk(const ReqDesc* reqs, int n_req, const SeamWindow* seams, const ModelDims& m, int n_terms,
                        int max_T, int max_k, unsigned long long* acc, uint32_t* status, cudaStream_t st) {
  (void)m;
  int t_pad = (max_T + 31) & ~31;
  int k_pad = 1;
  while (k_pad < max_k) k_pad <<= 1;
  topk_kernel<<<n_req, kThreads, topk_smem(t_pad, k_pad), st>>>(reqs, seams, 1.0 / (double)n_terms, acc, t_pad, status);
  return cudaGetLastError();
}

}  // namespace kvb
