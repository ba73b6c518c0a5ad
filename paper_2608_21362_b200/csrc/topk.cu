// Selection (Algorithm 2 step 3 + the token windows of Algorithm 1), one CTA per request:
//   1. delta_t from the fixed-point sums of the deviation kernel (and clear them for the next call);
//   2. radix select (4 passes of 8 bits over order-preserving integer keys) for the k-th largest
//      delta; ties at the threshold are taken in index order, so the set is the first k of the
//      order (delta descending, index ascending);
//   3. bitonic sort of the k (key, index) pairs -> rank, most deviated first;
//   4. bitmask union with the seam windows, prefix sum -> ascending sel and n_sel.
// All decisions are integer comparisons: the result is a pure function of the float32 delta.
// The kernel is latency-bound (one CTA, at most 128 KB of keys), so it is written to need few
// block-wide barriers: warp-aggregated histogram updates, one combined prefix sum for the
// selection, conflict-free shared-memory access, and the bitonic stages with stride < 32 done
// in registers with shuffles.
#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

constexpr int kThreads = 1024;
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

__device__ __forceinline__ unsigned long long shfl_xor64(unsigned long long v, int o) {
  return __shfl_xor_sync(0xffffffffu, v, o);
}
// one compare-exchange step of a bitonic network held one element per lane
__device__ __forceinline__ unsigned long long ce_step(unsigned long long v, int lane, int stride, bool up) {
  const unsigned long long o = shfl_xor64(v, stride);
  const bool take_min = ((lane & stride) == 0) == up;
  return take_min ? (v < o ? v : o) : (v > o ? v : o);
}

__global__ void __launch_bounds__(kThreads, 1)
    topk_kernel(const ReqDesc* __restrict__ reqs, const SeamWindow* __restrict__ seams, float inv_scale,
                unsigned long long* __restrict__ acc, int t_pad, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem);                                   // [t_pad]
  uint32_t* s_mask = s_keys + t_pad;                                                      // [kThreads] selection bitmask
  unsigned long long* s_comp = reinterpret_cast<unsigned long long*>(s_mask + kThreads);  // [k_pad]
  __shared__ uint32_t s_warp_sums[33];
  __shared__ uint32_t s_eqm[kThreads];   // per word of 32 positions: keys equal to the threshold
  __shared__ uint32_t s_base[kThreads];  // per word: how many selected positions precede it
  __shared__ uint32_t s_hist[2][256];  // two buffers: one is cleared while the other is scanned
  __shared__ uint32_t s_pick[2];       // chosen bin, remaining need

  pdl_wait();  // descriptors and deviation sums come from the kernels before this one
  const ReqDesc rq = reqs[blockIdx.x];
  const int T = rq.T, k = min(rq.k, T);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- 1. delta and keys.  The sums are integers below 2^50 (units of 2^-40); one conversion to
  //      float32 and one multiplication by 2^-40 / n_terms give delta to 1.2e-7 relative.
  for (int t = tid; t < T; t += kThreads) {
    const unsigned long long a = acc[rq.tok_offset + t];
    acc[rq.tok_offset + t] = 0ull;
    const float dl = __ll2float_rn((long long)a) * inv_scale;
    rq.delta[t] = dl;
    s_keys[t] = order_key(dl);
  }
  if (tid < 256) s_hist[1][tid] = 0u;  // the first pass (pass 3) counts into buffer 1
  __syncthreads();

  // ---- 2. radix select: threshold key `prefix`, and how many keys equal to it are taken (`need`)
  uint32_t prefix = 0, mask = 0, need = (uint32_t)k;
  if (k > 0 && k < T) {
    for (int pass = 3; pass >= 0; --pass) {
      uint32_t* hist = s_hist[pass & 1];
      const int shift = pass * 8;
      for (int t0 = 0; t0 < T; t0 += kThreads) {  // whole warps stay together for the votes
        const int t = t0 + tid;
        const uint32_t key = t < T ? s_keys[t] : 0u;
        const bool in = t < T && (key & mask) == prefix;
        const uint32_t digit = (key >> shift) & 255u;
        const uint32_t members = __ballot_sync(0xffffffffu, in);
        if (members == 0u) continue;
        const int leader = __ffs(members) - 1;
        const uint32_t d0 = __shfl_sync(0xffffffffu, digit, leader);
        if (__all_sync(0xffffffffu, !in || digit == d0)) {  // the high digits of nearby deviations mostly agree
          if (lane == leader) atomicAdd(&hist[d0], (uint32_t)__popc(members));
        } else if (in) {
          atomicAdd(&hist[digit], 1u);
        }
      }
      if (tid < 256) s_hist[(pass & 1) ^ 1][tid] = 0u;  // the next pass's histogram
      __syncthreads();
      if (warp == 0) {
        // lane j owns bins 255-8j .. 248-8j (descending); find the bin where the running count reaches need
        uint32_t local[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          local[i] = hist[255 - (lane * 8 + i)];
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
              s_pick[0] = 255 - (lane * 8 + i);
              s_pick[1] = need - before;
            }
            before += local[i];
          }
        }
      }
      __syncthreads();
      prefix |= s_pick[0] << shift;
      mask |= 255u << shift;
      need = s_pick[1];
    }
  }

  // ---- 3. the top-k set in index order.  Positions go by words of 32: a warp votes a word's
  //      "above the threshold" and "equal to it" masks, thread w then owns word w for the prefix
  //      scan, and warps write the word's selected positions side by side.
  const int n_words = (T + 31) >> 5;  // <= kThreads
  const uint32_t lanes_below = (1u << lane) - 1u;
  for (int w = warp; w < n_words; w += kThreads / 32) {
    const int t = w * 32 + lane;
    const bool live = t < T;
    const uint32_t key = live ? s_keys[t] : 0u;
    const uint32_t gt = __ballot_sync(0xffffffffu, live && (k >= T || (k > 0 && key > prefix)));
    const uint32_t eq = __ballot_sync(0xffffffffu, live && k > 0 && k < T && key == prefix);
    if (lane == 0) {
      s_mask[w] = gt;
      s_eqm[w] = eq;
    }
  }
  __syncthreads();
  const uint32_t gt_mask = tid < n_words ? s_mask[tid] : 0u, eq_mask = tid < n_words ? s_eqm[tid] : 0u;
  // one scan for both counts (each at most 32768: 16 bits apiece)
  uint32_t tot_packed;
  const uint32_t packed_before =
      block_exclusive_scan((uint32_t)__popc(gt_mask) | ((uint32_t)__popc(eq_mask) << 16), s_warp_sums, &tot_packed);
  const uint32_t gt_before = packed_before & 0xFFFFu, eq_before = packed_before >> 16;
  const uint32_t n_take_eq = (k > 0 && k < T) ? need : 0u;  // threshold-valued keys taken, lowest indices first
  int k_pad = 1;
  while (k_pad < k) k_pad <<= 1;
  if (tid < n_words) {
    // of this word's threshold-valued positions the lowest `take` join the selection
    uint32_t sel_mask = gt_mask, e = eq_mask;
    int take = (int)min((uint32_t)__popc(eq_mask), n_take_eq > eq_before ? n_take_eq - eq_before : 0u);
    while (take-- > 0) {
      const uint32_t low = e & (0u - e);
      sel_mask |= low;
      e ^= low;
    }
    s_mask[tid] = sel_mask;
    s_base[tid] = gt_before + min(eq_before, n_take_eq);
  }
  for (int i = k + tid; i < k_pad; i += kThreads) s_comp[i] = ~0ull;  // padding sorts last
  const uint32_t tot_sel = (tot_packed & 0xFFFFu) + min(tot_packed >> 16, n_take_eq);
  __syncthreads();
  // composite sort keys (larger delta first, then lower index) of the selected positions, in index order
  for (int w = warp; w < n_words; w += kThreads / 32) {
    const uint32_t m = s_mask[w];
    if ((m >> lane) & 1u) {
      const uint32_t pos = s_base[w] + __popc(m & lanes_below);
      const uint32_t t = w * 32 + lane;
      if (pos < (uint32_t)k_pad) s_comp[pos] = ((unsigned long long)(~s_keys[t]) << 32) | t;
    }
  }
  __syncthreads();

  // ---- bitonic sort of s_comp[0..k_pad): element i lives in lane i % 32 of its warp for the steps
  //      with stride < 32 (registers + shuffles); larger strides go through shared memory
  if (k_pad >= 64 && k_pad <= kThreads && (size_t)k_pad * 8 <= (size_t)t_pad * 4) {
    // One element per thread, held in a register for the whole sort.  Strides below 32 are shuffles;
    // larger strides publish the element and read the partner's, alternating between s_comp and the
    // key array (no longer needed) so that one barrier per step is enough.  Only the k_pad threads
    // that hold an element take part (named barrier 1).
    if (tid < k_pad) {
      unsigned long long* bufs[2] = {s_comp, reinterpret_cast<unsigned long long*>(s_keys)};
      unsigned long long v = s_comp[tid];
#pragma unroll
      for (int size = 2; size <= 32; size <<= 1) {
        const bool up = (tid & size) == 0;
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) v = ce_step(v, lane, stride, up);
      }
      int b = 1;
      for (int size = 64; size <= k_pad; size <<= 1) {
        const bool up = (tid & size) == 0;
        for (int stride = size >> 1; stride >= 32; stride >>= 1) {
          bufs[b][tid] = v;
          asm volatile("bar.sync 1, %0;" ::"r"(k_pad) : "memory");
          const unsigned long long o = bufs[b][tid ^ stride];
          const bool take_min = ((tid & stride) == 0) == up;
          v = take_min ? (v < o ? v : o) : (v > o ? v : o);
          b ^= 1;
        }
#pragma unroll
        for (int stride = 16; stride > 0; stride >>= 1) v = ce_step(v, lane, stride, up);
      }
      asm volatile("bar.sync 1, %0;" ::"r"(k_pad) : "memory");  // the last partner reads are done
      s_comp[tid] = v;
    }
    __syncthreads();
  } else if (k_pad >= 32) {
    for (int i0 = 0; i0 < k_pad; i0 += kThreads) {  // sizes 2..32 entirely in registers
      const int i = i0 + tid;
      if (i0 + (tid & ~31) >= k_pad) break;  // whole warps only (k_pad is a multiple of 32)
      unsigned long long v = s_comp[i];
#pragma unroll
      for (int size = 2; size <= 32; size <<= 1) {
        const bool up = (i & size) == 0;
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) v = ce_step(v, lane, stride, up);
      }
      s_comp[i] = v;
    }
    __syncthreads();
    for (int size = 64; size <= k_pad; size <<= 1) {
      for (int stride = size >> 1; stride >= 32; stride >>= 1) {
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
      for (int i0 = 0; i0 < k_pad; i0 += kThreads) {  // strides 16..1 of this size
        const int i = i0 + tid;
        if (i0 + (tid & ~31) >= k_pad) break;
        unsigned long long v = s_comp[i];
        const bool up = (i & size) == 0;
#pragma unroll
        for (int stride = 16; stride > 0; stride >>= 1) v = ce_step(v, lane, stride, up);
        s_comp[i] = v;
      }
      __syncthreads();
    }
  } else {
    if (warp == 0) {  // fewer than 32 elements: one warp, padded with keys that sort last
      unsigned long long v = lane < k_pad ? s_comp[lane] : ~0ull;
#pragma unroll
      for (int size = 2; size <= 32; size <<= 1) {
        const bool up = (lane & size) == 0;
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) v = ce_step(v, lane, stride, up);
      }
      if (lane < k_pad) s_comp[lane] = v;
    }
    __syncthreads();
  }
  for (int i = tid; i < k; i += kThreads) rq.rank[i] = (int32_t)(uint32_t)(s_comp[i] & 0xFFFFFFFFull);

  // ---- 4. union with the seam windows, ascending list
  //      (a warp per window, a lane per mask word of the window)
  for (int w = warp; w < rq.n_seams; w += kThreads / 32) {
    const SeamWindow sw = seams[rq.seam_offset + w];
    if (sw.hi <= sw.lo) continue;
    const int last = (sw.hi - 1) >> 5;
    for (int j = (sw.lo >> 5) + lane; j <= last; j += 32) {
      const int lo_bit = max(sw.lo - j * 32, 0), hi_bit = min(sw.hi - j * 32, 32);  // bits [lo_bit, hi_bit) of word j
      const uint32_t upto = hi_bit >= 32 ? 0xFFFFFFFFu : ((1u << hi_bit) - 1u);
      atomicOr(&s_mask[j], upto & ~((1u << lo_bit) - 1u));
    }
  }
  __syncthreads();
  const uint32_t word = tid < n_words ? s_mask[tid] : 0u;
  uint32_t n_sel;
  const uint32_t word_base = block_exclusive_scan(__popc(word), s_warp_sums, &n_sel);
  if (tid < n_words) s_base[tid] = word_base;
  __syncthreads();
  for (int w = warp; w < n_words; w += kThreads / 32) {
    const uint32_t m = s_mask[w];
    if ((m >> lane) & 1u) {
      const uint32_t pos = s_base[w] + __popc(m & lanes_below);
      if (pos < (uint32_t)rq.sel_capacity) rq.sel[pos] = w * 32 + lane;
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

static size_t topk_smem(int t_pad, int k_pad) { return (size_t)t_pad * 4 + kThreads * 4 + (size_t)(k_pad < 32 ? 32 : k_pad) * 8; }

cudaError_t topk_configure() {
  return cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)topk_smem(kMaxT, kMaxK));
}

cudaError_t launch_topk(const ReqDesc* reqs, int n_req, const SeamWindow* seams, const ModelDims& m, int n_terms,
                        int max_T, int max_k, unsigned long long* acc, uint32_t* status, bool pdl, cudaStream_t st) {
  (void)m;
  int t_pad = (max_T + 31) & ~31;
  int k_pad = 1;
  while (k_pad < max_k) k_pad <<= 1;
  const float inv_scale = (float)(1.0 / (1099511627776.0 * (double)n_terms));  // 2^-40 / n_terms
  return launch_pdl(pdl, topk_kernel, dim3(n_req), dim3(kThreads), topk_smem(t_pad, k_pad), st, reqs, seams, inv_scale, acc, t_pad, status);
}

}  // namespace kvb
