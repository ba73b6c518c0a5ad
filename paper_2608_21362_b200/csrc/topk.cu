// Selection (Algorithm 2 step 3 + the token windows of Algorithm 1):
//   1. delta_t from the fixed-point sums of the deviation step (and clear them for the next call),
//      order-preserving integer keys;
//   2. radix select (4 passes of 8 bits) for the k-th largest delta; ties at the threshold are taken
//      in index order, so the set is the first k of the order (delta descending, index ascending);
//   3. the k winners sorted in that order -> rank;
//   4. bitmask union with the seam windows, prefix sums -> ascending sel and n_sel.
// All decisions are integer comparisons: the result is a pure function of the float32 delta.
// Two kernels.  Prompts of up to 2048 positions take one CTA per request (warps sort runs of 32
// winners and every winner is ranked against the other runs by binary searches).  Longer prompts
// take a thread-block cluster of up to 8 CTAs per request,
// each owning a contiguous slice of the positions: every CTA counts its slice's histogram, sums all
// CTAs' histograms through distributed shared memory and takes the same decision (one cluster
// barrier per radix pass, histograms double-buffered); the prefix sums run locally, then over the
// cluster; every CTA sorts its own winners and ranks them against the other slices' sorted lists
// (a merge sort in the first CTA remains for a slice that holds more winners than a CTA has threads).
// The kernels are latency-bound (at most 128 KB of keys), so they are written to need few barriers:
// warp-aggregated histogram updates, one combined prefix sum for the selection, conflict-free
// shared-memory access.
#include <cooperative_groups.h>

#include "kvb_internal.h"
#include "pdl.cuh"

namespace cg = cooperative_groups;

namespace kvb {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxT = 32768;
constexpr int kMaxK = 8192;
constexpr int kMaxCluster = 8;
constexpr int kSingleTokens = 2048;              // prompts up to this length take one CTA
constexpr int kSplitTokens = 1024;               // longer ones: positions per CTA of the cluster (measured: T = 4096 on 4 CTAs
                                                 // 17.2 us against 19.3 on 2, T = 8192 on 8 CTAs 20.5 against 21.2 on 4)
constexpr int kMaxSlice = kMaxT / kMaxCluster;   // positions per CTA at the largest prompt
constexpr int kMaxWords = kMaxSlice / 32;        // 32-position mask words per CTA


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

// Ranks n <= kThreads distinct values, value i held by thread i (v; threads beyond n pass anything):
// every warp sorts a run of 32 of them (one per lane, bitonic network in registers) into
// runs[32 w .. 32 w + 31], padded with all ones, then each value finds by a binary search per other
// run how many of that run's values precede it; own place in the run + those counts = its rank.
// On return v is the value this thread holds after its warp's sort and the result is its rank (only
// meaningful when v is not the padding).  Contains a block-wide barrier: every thread calls it.
__device__ __forceinline__ uint32_t rank_by_runs(unsigned long long& v, int n, int tid, int lane, int warp, unsigned long long* runs) {
  const int n_runs = (n + 31) >> 5;
  if (tid >= n) v = ~0ull;
  if (warp < n_runs) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
      const bool up = (lane & size) == 0 || size == 32;  // the last stage leaves the run ascending
#pragma unroll
      for (int stride = size >> 1; stride > 0; stride >>= 1) v = ce_step(v, lane, stride, up);
    }
    runs[tid] = v;
  }
  __syncthreads();
  uint32_t place = (uint32_t)lane;
  if (warp < n_runs && v != ~0ull) {
    for (int r = 0; r < n_runs; ++r) {
      if (r == warp) continue;
      const unsigned long long* run = runs + (r << 5);
      uint32_t lo = 0;  // entries of run r below v
#pragma unroll
      for (int step = 16; step > 0; step >>= 1)
        if (run[lo + step - 1] < v) lo += step;
      if (run[lo] < v) ++lo;  // lo <= 31 here
      place += lo;
    }
  }
  return place;
}

// One CTA per request: the form for prompts of up to kSingleTokens positions, where a cluster's
// barriers would cost more than its CTAs save.  Steps as in the cluster kernel below, except that the
// k winners are sorted by a bitonic network (one element per thread, in a register).
__global__ void __launch_bounds__(kThreads, 1)
    topk_single_kernel(const ReqDesc* __restrict__ reqs, const SeamWindow* __restrict__ seams, float inv_scale,
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

  // ---- rank.  Up to kThreads winners: runs of 32 sorted by the warps, every winner ranked against the
  //      other runs (rank_by_runs), its position written at once.
  bool ranked = false;
  if (k_pad >= 64 && k_pad <= kThreads) {
    unsigned long long v = tid < k ? s_comp[tid] : ~0ull;
    __syncthreads();  // s_comp becomes the runs
    const uint32_t place = rank_by_runs(v, k, tid, lane, warp, s_comp);
    if (v != ~0ull) rq.rank[place] = (int32_t)(uint32_t)(v & 0xFFFFFFFFull);
    ranked = true;
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
  if (!ranked)
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


// What the other CTAs of a cluster read from this one (same offsets in every CTA).
struct Shared {
  uint32_t hist[2][256];  // radix histograms of this CTA's slice; two buffers, alternating by pass
  uint32_t n_win;         // winners of the slice (entries of the local winner list)
  uint32_t n_union;       // selected positions of the slice after the union with the windows
};

__global__ void __launch_bounds__(kThreads, 1)
    topk_cluster_kernel(const ReqDesc* __restrict__ reqs, const SeamWindow* __restrict__ seams, float inv_scale,
                        unsigned long long* __restrict__ acc, int slice_pad, int k_pad, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) uint8_t smem[];
  // dynamic: keys of the slice; inverted keys and positions of the slice's winners (index order);
  // two buffers for the request's winners (all slices' sorted lists side by side; the merge sort of
  // the fallback); two buffers for the sort of this slice's winners
  const int loc_pad = slice_pad < k_pad ? slice_pad : k_pad;
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem);  // [slice_pad]
  uint32_t* s_lkey = s_keys + slice_pad;                 // [loc_pad]
  uint32_t* s_lidx = s_lkey + loc_pad;                   // [loc_pad]
  unsigned long long* s_grp = reinterpret_cast<unsigned long long*>(s_lidx + loc_pad);  // 2 x [k_pad rounded up to 32]
  unsigned long long* s_sort = s_grp + 2 * ((k_pad + 31) & ~31);  // 2 x [kThreads]: this slice's winners, sorted (read by the other CTAs)
  __shared__ Shared sh;
  __shared__ uint32_t s_tot[256];          // histogram summed over the cluster
  __shared__ uint32_t s_warp_sums[33];
  __shared__ uint32_t s_mask[kMaxWords];   // per word of 32 positions: in the top-k set
  __shared__ uint32_t s_eqm[kMaxWords];    // per word: keys equal to the threshold
  __shared__ uint32_t s_umask[kMaxWords];  // per word: top-k set or inside a window
  __shared__ uint32_t s_base[kMaxWords];   // per word: how many winners of the slice precede it
  __shared__ uint32_t s_ubase[kMaxWords];  // per word: how many selected positions of the slice precede it
  __shared__ uint32_t s_pick[2];           // chosen bin, remaining need
  __shared__ uint32_t s_eq_lower;          // threshold-valued keys in the slices before this one

  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks();
  const int c = (int)cluster.block_rank();
  const bool clustered = S > 1;
  auto cluster_barrier = [&]() {
    if (clustered) cluster.sync(); else __syncthreads();
  };
  pdl_wait();  // descriptors and deviation sums come from the kernels before this one
  const ReqDesc rq = reqs[blockIdx.x / S];
  const int T = rq.T, k = min(rq.k, T);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = ((T + 32 * S - 1) / (32 * S)) * 32;  // positions per CTA, a whole number of mask words
  const int p0 = min(c * P, T), p1 = min(p0 + P, T);
  const int n_loc = p1 - p0;
  const int n_words = (n_loc + 31) >> 5;
  const bool selecting = k > 0 && k < T;  // the same in every CTA of the cluster

  if (tid < 256) sh.hist[0][tid] = sh.hist[1][tid] = 0u;
  if (tid == 0) s_eq_lower = 0u;
  __syncthreads();

  // warp-aggregated histogram update: nearby deviations mostly share their high digits
  auto count_digit = [&](uint32_t* hist, bool in, uint32_t digit) {
    const uint32_t members = __ballot_sync(0xffffffffu, in);
    if (members == 0u) return;
    const int leader = __ffs(members) - 1;
    const uint32_t d0 = __shfl_sync(0xffffffffu, digit, leader);
    if (__all_sync(0xffffffffu, !in || digit == d0)) {
      if (lane == leader) atomicAdd(&hist[d0], (uint32_t)__popc(members));
    } else if (in) {
      atomicAdd(&hist[digit], 1u);
    }
  };

  // ---- 1. delta, keys and the histogram of the top digit.  The sums are integers below 2^50 (units
  //      of 2^-40); one conversion to float32 and one multiplication by 2^-40 / n_terms give delta to
  //      1.2e-7 relative.
  for (int t0 = 0; t0 < n_loc; t0 += kThreads) {  // whole warps stay together for the votes
    const int t = t0 + tid;
    const bool live = t < n_loc;
    uint32_t key = 0u;
    if (live) {
      const size_t at = (size_t)rq.tok_offset + p0 + t;
      const unsigned long long a = acc[at];
      acc[at] = 0ull;
      const float dl = __ll2float_rn((long long)a) * inv_scale;
      rq.delta[p0 + t] = dl;
      key = order_key(dl);
      s_keys[t] = key;
    }
    if (selecting) count_digit(sh.hist[1], live, key >> 24);  // pass 3 counts into buffer 1
  }
  // ---- 2. radix select: threshold key `prefix`, and how many keys equal to it are taken (`need`).
  //      One cluster barrier per pass: a pass's histograms sit in buffer pass & 1, and the other
  //      buffer is cleared only after the barrier that follows everybody's reads of it.
  uint32_t prefix = 0, mask = 0, need = (uint32_t)k;
  if (selecting) {
    for (int pass = 3; pass >= 0; --pass) {
      const int buf = pass & 1;
      const int shift = pass * 8;
      if (pass < 3) {
        for (int t0 = 0; t0 < n_loc; t0 += kThreads) {
          const int t = t0 + tid;
          const uint32_t key = t < n_loc ? s_keys[t] : 0u;
          count_digit(sh.hist[buf], t < n_loc && (key & mask) == prefix, (key >> shift) & 255u);
        }
      }
      cluster_barrier();
      uint32_t part[kMaxCluster];
      if (tid < 256) {
#pragma unroll
        for (int r = 0; r < kMaxCluster; ++r)  // all remote reads in flight together
          part[r] = r < S ? cluster.map_shared_rank(&sh.hist[buf][0], r)[tid] : 0u;
        uint32_t sum = 0;
#pragma unroll
        for (int r = 0; r < kMaxCluster; ++r) sum += part[r];
        s_tot[tid] = sum;
        sh.hist[buf ^ 1][tid] = 0u;  // the next pass's histogram (nobody reads that buffer any more)
      }
      __syncthreads();
      if (warp == 0) {
        // lane j owns bins 255-8j .. 248-8j (descending); find the bin where the running count reaches need
        uint32_t local[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          local[i] = s_tot[255 - (lane * 8 + i)];
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
      // the last pass's bins are whole keys: the thread that summed the chosen bin knows how many
      // threshold-valued keys every slice holds, hence how many lie before this slice
      if (pass == 0 && tid == (int)s_pick[0]) {
        uint32_t lower = 0;
#pragma unroll
        for (int r = 0; r < kMaxCluster; ++r) lower += r < c ? part[r] : 0u;
        s_eq_lower = lower;
      }
      prefix |= s_pick[0] << shift;
      mask |= 255u << shift;
      need = s_pick[1];
    }
  }
  // ---- 3. the top-k set in index order.  Positions go by words of 32: a warp votes a word's
  //      "above the threshold" and "equal to it" masks, thread w then owns word w for the prefix
  //      scan, and warps write the word's selected positions side by side.
  const uint32_t lanes_below = (1u << lane) - 1u;
  for (int w = warp; w < n_words; w += kWarps) {
    const int t = w * 32 + lane;
    const bool live = t < n_loc;
    const uint32_t key = live ? s_keys[t] : 0u;
    const uint32_t gt = __ballot_sync(0xffffffffu, live && (k >= T || (k > 0 && key > prefix)));
    const uint32_t eq = __ballot_sync(0xffffffffu, live && selecting && key == prefix);
    if (lane == 0) {
      s_mask[w] = gt;
      s_eqm[w] = eq;
    }
  }
  __syncthreads();  // also orders s_eq_lower
  const uint32_t gt_mask = tid < n_words ? s_mask[tid] : 0u, eq_mask = tid < n_words ? s_eqm[tid] : 0u;
  // one scan for both counts (each at most 4096 per slice: 16 bits apiece)
  uint32_t tot_packed;
  const uint32_t packed_before =
      block_exclusive_scan((uint32_t)__popc(gt_mask) | ((uint32_t)__popc(eq_mask) << 16), s_warp_sums, &tot_packed);
  const uint32_t gt_before = packed_before & 0xFFFFu, eq_before = packed_before >> 16;
  // threshold-valued keys are taken lowest index first: the slices before this one come first
  const uint32_t eq_lower = s_eq_lower;
  const uint32_t n_take_eq = selecting ? need : 0u;
  const uint32_t eq_budget = n_take_eq > eq_lower ? n_take_eq - eq_lower : 0u;  // how many of them this slice may take
  const uint32_t n_win = (tot_packed & 0xFFFFu) + min(tot_packed >> 16, eq_budget);
  if (tid < n_words) {
    // of this word's threshold-valued positions the lowest `take` join the selection
    uint32_t sel_mask = gt_mask, e = eq_mask;
    int take = (int)min((uint32_t)__popc(eq_mask), eq_budget > eq_before ? eq_budget - eq_before : 0u);
    while (take-- > 0) {
      const uint32_t low = e & (0u - e);
      sel_mask |= low;
      e ^= low;
    }
    s_mask[tid] = sel_mask;
    s_umask[tid] = sel_mask;
    s_base[tid] = gt_before + min(eq_before, eq_budget);
  }
  __syncthreads();
  // inverted keys and positions of the slice's winners, in index order ...
  for (int w = warp; w < n_words; w += kWarps) {
    const uint32_t m = s_mask[w];
    if ((m >> lane) & 1u) {
      const uint32_t pos = s_base[w] + __popc(m & lanes_below);
      const uint32_t t = w * 32 + lane;
      s_lkey[pos] = ~s_keys[t];
      s_lidx[pos] = (uint32_t)(p0 + t);
    }
  }
  // ... and the union with the seam windows (a thread per window, so one round of loads covers 1024
  // windows; only the part inside this slice)
  for (int w = tid; w < rq.n_seams; w += kThreads) {
    const SeamWindow sw = seams[rq.seam_offset + w];
    const int lo = max(sw.lo, p0) - p0, hi = min(sw.hi, p1) - p0;  // in slice coordinates
    if (hi <= lo) continue;
    const int last = (hi - 1) >> 5;
    for (int j = lo >> 5; j <= last; ++j) {
      const int lo_bit = max(lo - j * 32, 0), hi_bit = min(hi - j * 32, 32);  // bits [lo_bit, hi_bit) of word j
      const uint32_t upto = hi_bit >= 32 ? 0xFFFFFFFFu : ((1u << hi_bit) - 1u);
      atomicOr(&s_umask[j], upto & ~((1u << lo_bit) - 1u));
    }
  }
  __syncthreads();
  const uint32_t word = tid < n_words ? s_umask[tid] : 0u;
  uint32_t n_union;
  const uint32_t word_base = block_exclusive_scan(__popc(word), s_warp_sums, &n_union);
  if (tid < n_words) s_ubase[tid] = word_base;
  if (tid == 0) {
    sh.n_win = n_win;
    sh.n_union = n_union;
  }
  cluster_barrier();  // every slice's winner list and counts are complete

  // ---- 4. ascending sel and n_sel: this slice's selected positions follow those of the slices before it
  uint32_t win_r[kMaxCluster], uni_r[kMaxCluster];
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r) {
    win_r[r] = r < S ? *cluster.map_shared_rank(&sh.n_win, r) : 0u;
    uni_r[r] = r < S ? *cluster.map_shared_rank(&sh.n_union, r) : 0u;
  }
  uint32_t sel_lower = 0, n_sel = 0, n_all = 0;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r) {
    if (r < c) sel_lower += uni_r[r];
    n_sel += uni_r[r];
    n_all += win_r[r];
  }
  for (int w = warp; w < n_words; w += kWarps) {
    const uint32_t m = s_umask[w];
    if ((m >> lane) & 1u) {
      const uint32_t pos = sel_lower + s_ubase[w] + __popc(m & lanes_below);
      if (pos < (uint32_t)rq.sel_capacity) rq.sel[pos] = p0 + w * 32 + lane;
    }
  }
  if (c == 0 && tid == 0) {
    if (n_sel > (uint32_t)rq.sel_capacity) {
      atomicOr(status, DEV_STATUS_SEL_OVERFLOW);
      n_sel = rq.sel_capacity;
    }
    *rq.n_sel = (int32_t)n_sel;
    if (n_all != (uint32_t)k) atomicOr(status, DEV_STATUS_BAD_DESC);
  }

  // ---- 5. rank: the winners' composite values (inverted key, index) in ascending order = key
  //      descending, index ascending.  Every CTA sorts its slice's winners (rank_by_runs, then each
  //      value stored at its place); after a cluster barrier it copies all slices' sorted lists into its own
  //      shared memory and each of its winners finds, by a binary search per other list, how many
  //      winners of the other slices precede it: own place + those counts = its rank.  All values are
  //      distinct.  The same in every CTA of the cluster: whether every slice's list fits a CTA.
  bool spread = n_all == (uint32_t)k && k > 0;
#pragma unroll
  for (int r = 0; r < kMaxCluster; ++r) spread = spread && win_r[r] <= (uint32_t)kThreads;
  if (spread) {
    unsigned long long v = ~0ull;
    if (tid < (int)n_win) v = ((unsigned long long)s_lkey[tid] << 32) | s_lidx[tid];
    const uint32_t local_place = rank_by_runs(v, (int)n_win, tid, lane, warp, s_sort + kThreads);
    if (v != ~0ull) s_sort[local_place] = v;  // this slice's winners in ascending order
    cluster_barrier();  // every slice's sorted list is complete
    uint32_t off_r[kMaxCluster];
    {
      uint32_t o = 0;
#pragma unroll
      for (int r = 0; r < kMaxCluster; ++r) {
        off_r[r] = o;
        o += win_r[r];
      }
    }
    for (uint32_t e = tid; e < n_all; e += kThreads) {  // entry e of the side-by-side lists is entry e - off_r of slice r's
      int r = 0;
#pragma unroll
      for (int rr = 1; rr < kMaxCluster; ++rr)
        if (rr < S && e >= off_r[rr]) r = rr;
      s_grp[e] = cluster.map_shared_rank(s_sort, r)[e - off_r[r]];
    }
    __syncthreads();
    if (v != ~0ull) {
      uint32_t place = local_place;
#pragma unroll
      for (int r = 0; r < kMaxCluster; ++r) {
        if (r >= S || r == c) continue;
        const unsigned long long* a = s_grp + off_r[r];
        uint32_t lo = 0, hi = win_r[r];  // entries of slice r below v
        while (lo < hi) {
          const uint32_t mid = (lo + hi) >> 1;
          if (a[mid] < v) lo = mid + 1; else hi = mid;
        }
        place += lo;
      }
      rq.rank[place] = (int32_t)(uint32_t)(v & 0xFFFFFFFFull);
    }
  } else if (c == 0 && n_all == (uint32_t)k && k > 0) {
    // fallback (a slice with more winners than threads), by the first CTA: a merge sort.  Runs of 32 are
    // sorted by a bitonic network in registers (one element per lane), then runs are merged pairwise:
    // every element finds its place in the merged run by a binary search of the sibling run; the
    // padding (all ones) sorts last and the merge keeps equal values in run order.
    constexpr int kPer = kMaxK / kThreads;  // elements per thread
    const uint32_t n_pad = (n_all + 31u) & ~31u;
    unsigned long long *src = s_grp, *dst = s_grp + ((k_pad + 31) & ~31);
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      const uint32_t e = (uint32_t)tid + (uint32_t)q * kThreads;
      if ((e & ~31u) >= n_pad) continue;  // whole warps
      unsigned long long v = ~0ull;
      if (e < n_all) {  // winner e of the request (index order) is entry e - first of slice r's list
        uint32_t first = 0;
        int r = 0;
#pragma unroll
        for (int rr = 0; rr < kMaxCluster - 1; ++rr)
          if (r == rr && e >= first + win_r[rr]) {  // e < n_all, so the walk stops inside the cluster
            first += win_r[rr];
            r = rr + 1;
          }
        const uint32_t ik = cluster.map_shared_rank(s_lkey, r)[e - first];
        const uint32_t ix = cluster.map_shared_rank(s_lidx, r)[e - first];
        v = ((unsigned long long)ik << 32) | ix;
      }
#pragma unroll
      for (int size = 2; size <= 32; size <<= 1) {
        const bool up = (lane & size) == 0 || size == 32;  // the last stage leaves the run ascending
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
          const unsigned long long o = __shfl_xor_sync(0xffffffffu, v, stride);
          const bool take_min = ((lane & stride) == 0) == up;
          v = take_min ? (v < o ? v : o) : (v > o ? v : o);
        }
      }
      src[e] = v;
    }
    __syncthreads();
    for (uint32_t run = 32; run < n_pad; run <<= 1) {
#pragma unroll
      for (int q = 0; q < kPer; ++q) {
        const uint32_t e = (uint32_t)tid + (uint32_t)q * kThreads;
        if (e >= n_pad) continue;
        const unsigned long long v = src[e];
        const uint32_t base = e & ~(2u * run - 1u);          // first element of the pair of runs
        const uint32_t mid = min(base + run, n_pad), end = min(base + 2u * run, n_pad);
        uint32_t lo, hi;
        const bool second = e >= mid;
        if (!second) lo = mid, hi = end; else lo = base, hi = mid;
        // elements of the sibling run that precede v: strictly smaller ones, and for the second run
        // also equal ones (the first run's elements come first among equals)
        while (lo < hi) {
          const uint32_t m = (lo + hi) >> 1;
          const unsigned long long o = src[m];
          if (second ? o <= v : o < v) lo = m + 1; else hi = m;
        }
        const uint32_t place = second ? base + (e - mid) + (lo - base) : e + (lo - mid);
        dst[place] = v;
      }
      __syncthreads();
      unsigned long long* t = src;
      src = dst;
      dst = t;
    }
    for (uint32_t e = tid; e < n_all; e += kThreads) rq.rank[e] = (int32_t)(uint32_t)(src[e] & 0xFFFFFFFFull);
  }
  // no CTA leaves while another may still be reading its shared memory
  if (clustered) cluster.sync();
}

int cluster_size(int max_T) {
  if (max_T <= kSingleTokens) return 1;
  const int s = (max_T + kSplitTokens - 1) / kSplitTokens;
  return s > kMaxCluster ? kMaxCluster : s;
}

size_t cluster_smem(int slice_pad, int k_pad) {
  const size_t loc = (size_t)(slice_pad < k_pad ? slice_pad : k_pad);
  return (size_t)slice_pad * 4 + loc * 8 + (size_t)((k_pad + 31) & ~31) * 16 + (size_t)kThreads * 16;
}

size_t single_smem(int t_pad, int k_pad) { return (size_t)t_pad * 4 + kThreads * 4 + (size_t)(k_pad < 32 ? 32 : k_pad) * 8; }

}  // namespace

int topk_max_T() { return kMaxT; }
int topk_max_k() { return kMaxK; }

cudaError_t topk_configure() {
  cudaError_t e = cudaFuncSetAttribute(topk_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cluster_smem(kMaxSlice, kMaxK));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(topk_single_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)single_smem(kSingleTokens, kSingleTokens));
}

cudaError_t launch_topk(const ReqDesc* reqs, int n_req, const SeamWindow* seams, const ModelDims& m, int n_terms,
                        int max_T, int max_k, unsigned long long* acc, uint32_t* status, bool pdl, cudaStream_t st) {
  (void)m;
  const int S = cluster_size(max_T);
  const float inv_scale = (float)(1.0 / (1099511627776.0 * (double)n_terms));  // 2^-40 / n_terms
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n_req * S);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)S;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  if (S == 1) {  // short prompts: one CTA per request
    const int t_pad = (max_T + 31) & ~31;
    int k_pow2 = 1;
    while (k_pow2 < max_k) k_pow2 <<= 1;
    cfg.dynamicSmemBytes = single_smem(t_pad, k_pow2);
    return cudaLaunchKernelEx(&cfg, topk_single_kernel, reqs, seams, inv_scale, acc, t_pad, status);
  }
  const int slice_pad = ((max_T + 32 * S - 1) / (32 * S)) * 32;  // the largest slice of the batch
  const int k_pad = ((max_k < 1 ? 1 : max_k) + 3) & ~3;
  cfg.dynamicSmemBytes = cluster_smem(slice_pad, k_pad);
  return cudaLaunchKernelEx(&cfg, topk_cluster_kernel, reqs, seams, inv_scale, acc, slice_pad, k_pad, status);
}

}  // namespace kvb
