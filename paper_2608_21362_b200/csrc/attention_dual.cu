// Selected-row causal attention (Eq. 2), two tiles per CTA.
//
// The same tile, streams and softmax as the one-tile kernel (a tile = (layer, KV head, 128/rep
// selected tokens) x the rep query heads of the KV head; keys by sub-blocks of 64 on two alternating
// streams; S = Q K^T and O += P V by tcgen05.mma with S, P and O in TMEM; lazy running maximum), but
// a CTA takes TWO neighbouring tiles of one (layer, KV head) plane at a time and owns the SM: both
// tiles read the same K and V sub-blocks from shared memory, so every K/V byte crosses from L2 once
// per 256 rows instead of once per 128.  One TMA thread serves both tiles; each tile has its own
// MMA-issuing warp (one issuing thread for both measured 9-12 % slower than the one-tile kernel: a
// wait for one tile's P held back the other's ready work), its own four softmax warps, its own S/P
// and O columns (2 x 256 = all 512 TMEM columns) and its own barriers; a K or V buffer is refilled
// when both tiles' MMAs have read it.  The tiles of a pair are neighbours in the ascending selection, so the second needs at
// most a sub-block or two more than the first; both run over the pair's sub-blocks, the first
// tile's surplus is masked out like every key beyond a row's own position.
// Every wait is bounded, as in the one-tile kernel.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

constexpr int kThreads = 352;               // TMA warp, an MMA warp per tile, 2 x 4 softmax warps
constexpr int kRows = 128;
constexpr int kSubKeys = 64;                         // keys per sub-block (one stream's MMA N)
constexpr int kD = 128;
constexpr uint32_t kTileBytes = kRows * kD * 2;      // 32 KB: Q, K or V tile
constexpr uint32_t kHalfBytes = kTileBytes / 2;      // one 64-element-wide TMA box of Q (128 rows)
constexpr uint32_t kSubBytes = kSubKeys * kD * 2;    // 16 KB: one stream's K or V sub-block
constexpr uint32_t kTmemCols = 512;                  // per tile of the pair: S/P columns 0..127, O columns 128..255
constexpr uint32_t kWaitHintNs = 20000;              // per try; 2 us .. 200 us measured alike
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // a wait that lasts two seconds gives up
constexpr float kLazyThreshold = 8.0f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One try with a suspend-time hint: the hardware parks the thread until the phase completes or the
// hint (nanoseconds) runs out instead of returning at once.  Twelve warps per SM wait on barriers most
// of the time; without the hint their re-issued tries crowd the queue that the MMA issue, the TMEM
// loads and the global stores also go through (measured: +4 % on the whole kernel).
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kWaitHintNs)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait (limit_ns of wall time); also gives up as soon as another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait_ns(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag, unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > limit_ns) break;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  return mbar_wait_ns(bar, parity, abort_flag, kWaitLimitNs);
}

// ---- TMA
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
                   smem_u32(dst)),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}
__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(
                   smem_u32(dst)),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
               : "memory");
}
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* map) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---- tcgen05
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xffffffff;\n @e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with the accumulate flag fixed to 1 (no register, no setp on a register: the issuing
// thread's instruction count matters).
__device__ __forceinline__ void mma_ss_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.eq.b32 p, 0, 0;\n @e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc)
      : "memory");
}
__device__ __forceinline__ void mma_ts_acc(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.eq.b32 p, 0, 0;\n @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc)
      : "memory");
}
// Load 32 columns of this thread's TMEM lane and wait for them: the wait sits in the same asm
// statement so that no use of the registers can be scheduled before it.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
      "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
      "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (128-byte swizzle, 8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFFu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;  // descriptor version of this architecture
  d |= 2ull << 61;  // SWIZZLE_128B
  return d;
}

// Instruction descriptor: float32 accumulate, A/B bf16 or fp16, M = 128, N = n.
template <int DT>
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, bool b_mn_major) {
  const uint32_t fmt = DT == KVB_DT_BF16 ? 1u : 0u;
  uint32_t d = 0;
  d |= 1u << 4;                      // D format f32
  d |= fmt << 7;                     // A format
  d |= fmt << 10;                    // B format
  d |= (b_mn_major ? 1u : 0u) << 16; // B major: 0 = K, 1 = MN
  d |= (n >> 3) << 17;               // N
  d |= (128u >> 4) << 24;            // M
  return d;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed float32 pairs (one instruction for two lanes of work) and the three-input maximum.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void f2_unpack(uint64_t d, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(d)); }
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// One 32-byte store (the address must be 32-byte aligned).
__device__ __forceinline__ void st_global_256(void* p, const uint32_t (&w)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]),
               "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
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

constexpr int kStages = 4;  // K and V sub-block buffers each (the two tiles may drift apart by that much)

struct __align__(8) Barriers {
  // shared by the two tiles
  uint64_t tile_full[2], tile_empty[2], q_full, q_empty;
  uint64_t k_full[kStages], v_full[kStages], k_empty[kStages], v_empty[kStages];  // empty: both tiles' MMAs have read the buffer
  // per tile u and S/P stream x
  uint64_t s_full[2][2], p_full[2][2], pv_done[2][2], o_full[2], o_empty[2];
};

// What the producer hands to the other roles for one tile (a two-slot ring in shared memory).
struct TileInfo {
  const int32_t* sel;
  uint8_t* out;
  int32_t n_sel, i_base, l, hk, nsb, sel_capacity;  // nsb = 0: no more tiles
};

// What the producer knows about the tile it will load next.
struct NextTile {
  TileInfo ti;
  const CUtensorMap *map_q, *map_kv;
};

// Next tile that has rows, in the order: request, then groups of rq.lhk_group (layer, KV head) pairs
// whose K/V planes fit L2 together, inside a group tile-major from the longest tile down with the
// group's pairs interleaved.  `drawn` is the linear tile number already drawn for this call; the
// one after it is drawn here (persistent CTAs) so that its latency is hidden.  ti.nsb = 0: none left.
template <bool PERSISTENT>
__device__ __forceinline__ NextTile decode_next_tile(unsigned int& drawn, unsigned int* tile_counter, const ReqDesc* __restrict__ reqs,
                                                     const CUtensorMap* maps, int n_req, int total_tiles, int per_tile, int TOK, int Hkv) {
  const unsigned int kNoTile = 0xFFFFFFFFu;
    NextTile nx;
    nx.ti.nsb = 0;
    nx.map_q = nx.map_kv = nullptr;
    for (;;) {  // next tile that has rows
      const long long lin_ll = drawn;
      if (lin_ll >= (long long)total_tiles * per_tile) break;
      const int lin = (int)lin_ll;
      drawn = PERSISTENT ? gridDim.x + atomicAdd(tile_counter, 1u) : kNoTile;  // the first gridDim.x tiles went by block index
      int lo = 0, hi = n_req - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (reqs[mid].tile_offset * per_tile <= lin) lo = mid; else hi = mid - 1;
      }
      const ReqDesc& rq = reqs[lo];
      const int cap = rq.sel_capacity;
      const int tiles_r = (cap + TOK - 1) / TOK;
      const int idx = lin - rq.tile_offset * per_tile;
      const int G = rq.lhk_group;
      const int grp = idx / (G * tiles_r);
      const int rem = idx - grp * G * tiles_r;
      const int g_eff = min(G, per_tile - grp * G);
      const int lhk = grp * G + rem % g_eff;
      const int tile = tiles_r - 1 - rem / g_eff;
      const int n_sel = min(*rq.n_sel, cap);
      const int i_base = tile * TOK;
      if (i_base >= n_sel) continue;
      const int t_max = min(rq.sel[min(i_base + TOK, n_sel) - 1], rq.T - 1);
      nx.ti.sel = rq.sel;
      nx.ti.out = rq.out;
      nx.ti.n_sel = n_sel;
      nx.ti.i_base = i_base;
      nx.ti.l = lhk / Hkv;
      nx.ti.hk = lhk % Hkv;
      nx.ti.nsb = max(t_max, 0) / kSubKeys + 1;  // 64-key sub-blocks to visit
      nx.ti.sel_capacity = cap;
      nx.map_q = maps + 2 * lo;
      nx.map_kv = maps + 2 * lo + 1;
      break;
    }
    return nx;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
    attn_dual_kernel(const ReqDesc* __restrict__ reqs, const CUtensorMap* __restrict__ maps, int n_req, int total_pairs,
                     ModelDims m, float scale_log2, uint32_t* __restrict__ status, unsigned int* __restrict__ tile_counter) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Barriers bars;
  __shared__ TileInfo s_tiles[2];
  __shared__ uint32_t s_tmem_base;
  __shared__ uint32_t s_abort;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_tile = m.Hkv * m.L;
  const int rep = m.Hq / m.Hkv;
  const int TOK = kRows / rep;  // tokens of one tile; a pair covers 2 * TOK neighbouring entries of the selection

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                   // tile u at + u * 32 KB: two 64-wide boxes of 16 KB
  uint8_t* sK = smem + 2 * kTileBytes;                       // buffer b at + b * 16 KB: two 64-wide boxes of 8 KB (64 keys)
  uint8_t* sV = smem + 2 * kTileBytes + kStages * kSubBytes;  // same
  volatile uint32_t* abort_flag = &s_abort;

  unsigned int drawn = 0xFFFFFFFFu;  // only the producer thread draws
  if (tid == 0) {
    pdl_wait();  // descriptors, tensor maps and the tile counter come from the kernel before this one
    drawn = blockIdx.x;
  }
  // a pair is decoded as one tile of 2 * TOK tokens
  auto decode_next = [&]() { return decode_next_tile<true>(drawn, tile_counter, reqs, maps, n_req, total_pairs, per_tile, 2 * TOK, m.Hkv); };
  NextTile next;
  next.ti.nsb = 0;
  next.map_q = next.map_kv = nullptr;
  if (tid == 0) next = decode_next();

  if (tid == 64) {
    for (int x = 0; x < 2; ++x) {
      mbar_init(&bars.tile_full[x], 1);
      mbar_init(&bars.tile_empty[x], 258);  // the two MMA threads and the 256 softmax threads
      for (int u = 0; u < 2; ++u) {
        mbar_init(&bars.s_full[u][x], 1);
        mbar_init(&bars.p_full[u][x], 128);
        mbar_init(&bars.pv_done[u][x], 1);
      }
      mbar_init(&bars.o_full[x], 1);
      mbar_init(&bars.o_empty[x], 128);
    }
    for (int b = 0; b < kStages; ++b) {
      mbar_init(&bars.k_full[b], 1);
      mbar_init(&bars.v_full[b], 1);
      mbar_init(&bars.k_empty[b], 2);  // both tiles' MMA threads
      mbar_init(&bars.v_empty[b], 2);
    }
    mbar_init(&bars.q_full, 1);
    mbar_init(&bars.q_empty, 2);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // TMEM allocation is a warp-wide operation; this CTA owns the SM and takes all of it
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  // tile u: S/P of stream x at columns 256 u + 64 x (P packed over the first 32 of them), O at 256 u + 128
  auto tmem_S = [&](int u, int x) { return tmem_base + (uint32_t)(u * 256 + x * kSubKeys); };
  auto tmem_O = [&](int u) { return tmem_base + (uint32_t)(u * 256 + 128); };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      uint32_t g = 0;  // sub-blocks of the pairs before this one: streams, buffers and phases follow the running number
      for (int n = 0; ok; ++n) {
        const TileInfo ti = next.ti;
        const CUtensorMap *map_q = next.map_q, *map_kv = next.map_kv;
        const int slot = n & 1;
        if (n >= 2) ok = mbar_wait(&bars.tile_empty[slot], ((n >> 1) & 1) ^ 1, abort_flag);  // pair n-2 has been read
        if (!ok) break;
        s_tiles[slot] = ti;
        mbar_arrive(&bars.tile_full[slot]);
        if (ti.nsb == 0) break;
        const int nsb = ti.nsb, l = ti.l, hk = ti.hk;
        if (n >= 1) ok = mbar_wait(&bars.q_empty, (n - 1) & 1, abort_flag);  // the previous pair's S MMAs have read Q
        if (!ok) break;
        tensormap_acquire(map_q);
        tensormap_acquire(map_kv);
        mbar_expect_tx(&bars.q_full, 2 * kTileBytes);
#pragma unroll
        for (int u = 0; u < 2; ++u) {  // rows beyond the selection's capacity arrive as zeros
          tma_load_4d(sQ + u * kTileBytes, map_q, 0, hk * rep, ti.i_base + u * TOK, l, &bars.q_full);
          tma_load_4d(sQ + u * kTileBytes + kHalfBytes, map_q, 64, hk * rep, ti.i_base + u * TOK, l, &bars.q_full);
        }
        // K(sb) and V(sb) go into buffer (running number) % kStages as soon as both tiles' MMAs have read what it held
        auto load_k = [&](int sb) {  // false: gave up waiting for the buffer
          const uint32_t gg = g + sb;
          const int b = gg % kStages;
          if (gg >= kStages && !mbar_wait(&bars.k_empty[b], ((gg / kStages) & 1) ^ 1, abort_flag)) return false;
          mbar_expect_tx(&bars.k_full[b], kSubBytes);
          tma_load_5d(sK + b * kSubBytes, map_kv, 0, hk, sb * kSubKeys, 0, l, &bars.k_full[b]);
          tma_load_5d(sK + b * kSubBytes + kSubBytes / 2, map_kv, 64, hk, sb * kSubKeys, 0, l, &bars.k_full[b]);
          return true;
        };
        auto load_v = [&](int sb) {
          const uint32_t gg = g + sb;
          const int b = gg % kStages;
          if (gg >= kStages && !mbar_wait(&bars.v_empty[b], ((gg / kStages) & 1) ^ 1, abort_flag)) return false;
          mbar_expect_tx(&bars.v_full[b], kSubBytes);
          tma_load_5d(sV + b * kSubBytes, map_kv, 0, hk, sb * kSubKeys, 1, l, &bars.v_full[b]);
          tma_load_5d(sV + b * kSubBytes + kSubBytes / 2, map_kv, 64, hk, sb * kSubKeys, 1, l, &bars.v_full[b]);
          return true;
        };
        for (int sb = 0; sb < kStages - 1 && sb < nsb && ok; ++sb) ok = load_k(sb);  // K runs kStages - 1 sub-blocks ahead of V
        const int sb_decode = nsb > 4 ? nsb - 4 : 0;  // a few sub-blocks before the pair's end
        for (int sb = 0; sb < nsb && ok; ++sb) {
          ok = load_v(sb);
          if (ok && sb + kStages - 1 < nsb) ok = load_k(sb + kStages - 1);
          if (ok && sb == sb_decode) next = decode_next();
        }
        g += nsb;
      }
    }
  } else if (warp <= 2) {
    // ------------------------------------------------------------------ MMA issuer of tile u (whole warp, one elected lane issues)
    const int u = warp - 1;
    const uint32_t idesc_s = instr_desc<DT>(kSubKeys, false);
    const uint32_t idesc_pv = instr_desc<DT>(kD, true);
    const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
    bool ok = true;
    const uint64_t q_desc = smem_desc(q_addr, 16, 1024);
    const uint64_t k_desc = smem_desc(k_addr, 16, 1024);
    const uint64_t v_desc = smem_desc(v_addr, kSubBytes / 2, 1024);
    // sb below is the sub-block's number through all pairs of this CTA
    auto issue_s = [&](uint32_t sb) {  // S_u,x = Q_u K_x^T, N = 64 keys
      const int x = sb & 1, b = sb % kStages;
      if (!mbar_wait(&bars.k_full[b], (sb / kStages) & 1, abort_flag)) return false;
      tc_fence_after();
      const uint64_t qd = q_desc + (uint64_t)(u * (kTileBytes >> 4));
      const uint64_t kd = k_desc + (uint64_t)(b * (kSubBytes >> 4));
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {  // 16 elements of d per step; 4 steps per 64-element box
        const uint32_t qo = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
        const uint32_t ko = (ks >> 2) * (kSubBytes / 2) + (ks & 3) * 32;
        if (ks == 0)
          mma_ss(tmem_S(u, x), qd + (qo >> 4), kd + (ko >> 4), idesc_s, 0);
        else
          mma_ss_acc(tmem_S(u, x), qd + (qo >> 4), kd + (ko >> 4), idesc_s);
      }
      tc_commit(&bars.s_full[u][x]);
      tc_commit(&bars.k_empty[b]);
      return true;
    };
    auto issue_pv = [&](uint32_t sb, bool first) {  // O_u (+)= P_u,x V_x, 64 keys = 4 steps of 16
      const int x = sb & 1, b = sb % kStages;
      if (!mbar_wait(&bars.p_full[u][x], (sb >> 1) & 1, abort_flag) || !mbar_wait(&bars.v_full[b], (sb / kStages) & 1, abort_flag)) return false;
      tc_fence_after();
      const uint64_t vd = v_desc + (uint64_t)(b * (kSubBytes >> 4));
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {  // 16 keys = 2048 bytes of V; the two 64-wide halves of d are 8 KB apart
        if (ks == 0)
          mma_ts(tmem_O(u), tmem_S(u, x), vd, idesc_pv, !first);
        else
          mma_ts_acc(tmem_O(u), tmem_S(u, x) + ks * 8, vd + (ks * 2048 >> 4), idesc_pv);
      }
      tc_commit(&bars.pv_done[u][x]);
      tc_commit(&bars.v_empty[b]);
      return true;
    };
    uint32_t g = 0;
    for (int n = 0; ok; ++n) {
      const int slot = n & 1;
      ok = mbar_wait(&bars.tile_full[slot], (n >> 1) & 1, abort_flag);
      if (!ok) break;
      const int nsb = s_tiles[slot].nsb;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.tile_empty[slot]);
      if (nsb == 0) break;
      ok = mbar_wait(&bars.q_full, n & 1, abort_flag);
      if (!ok) break;
      ok = issue_s(g);
      if (ok && nsb > 1) ok = issue_s(g + 1);
      // the first P V of a pair overwrites O: the previous pair's epilogue must have read it
      if (ok && n > 0) {
        ok = mbar_wait(&bars.o_empty[u], (n - 1) & 1, abort_flag);
        tc_fence_after();
      }
      int sb = 0;
      for (; sb + 2 < nsb && ok; ++sb) ok = issue_pv(g + sb, sb == 0) && issue_s(g + sb + 2);
      if (ok) tc_commit(&bars.q_empty);
      for (; sb < nsb && ok; ++sb) ok = issue_pv(g + sb, sb == 0);
      if (ok) tc_commit(&bars.o_full[u]);
      g += nsb;
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (warps 3..6: first tile, 7..10: second)
    const int u = (warp - 3) >> 2;
    const int quarter = warp & 3;              // TMEM lanes this warp may touch
    const int row = quarter * 32 + lane;       // row of the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t my_O = tmem_O(u);
    bool ok = true;
    uint32_t g = 0;  // sub-blocks of the pairs before this one
    for (int n = 0; ok; ++n) {
      const int slot = n & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars.tile_full[slot], (n >> 1) & 1, abort_flag));
      if (!ok) break;
      const int nsb = s_tiles[slot].nsb;
      if (nsb == 0) {
        mbar_arrive(&bars.tile_empty[slot]);
        break;
      }
      int t_row;
      {
        const int i_row = s_tiles[slot].i_base + u * TOK + row / rep;
        t_row = i_row < s_tiles[slot].n_sel ? s_tiles[slot].sel[i_row] : -1;
      }
      int warp_tmin = t_row;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) warp_tmin = min(warp_tmin, __shfl_xor_sync(0xffffffffu, warp_tmin, o));
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int sb = 0; sb < nsb; ++sb) {
        const uint32_t gg = g + sb;
        const int x = gg & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(&bars.s_full[u][x], (gg >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        const int key0 = sb * kSubKeys;
        const bool need_mask = key0 + kSubKeys - 1 > warp_tmin;
        const uint32_t s_addr = tmem_S(u, x) + lane_addr;
        uint32_t r0[32], r1[32];
        tmem_ld32(s_addr, r0);
        tmem_ld32(s_addr + 32, r1);
        if (need_mask) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (key0 + i > t_row) r0[i] = 0xFF800000u;  // -inf
            if (key0 + 32 + i > t_row) r1[i] = 0xFF800000u;
          }
        }
        float mx[4] = {__uint_as_float(r0[0]), __uint_as_float(r0[1]), __uint_as_float(r1[0]), __uint_as_float(r1[1])};
#pragma unroll
        for (int i = 2; i < 32; i += 4) {
          mx[0] = fmax3(mx[0], __uint_as_float(r0[i]), __uint_as_float(r0[i + 1]));
          mx[2] = fmax3(mx[2], __uint_as_float(r1[i]), __uint_as_float(r1[i + 1]));
          if (i + 2 < 32) {
            mx[1] = fmax3(mx[1], __uint_as_float(r0[i + 2]), __uint_as_float(r0[i + 3]));
            mx[3] = fmax3(mx[3], __uint_as_float(r1[i + 2]), __uint_as_float(r1[i + 3]));
          }
        }
        const float bm = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;  // scale > 0 commutes with max
        // lazy reference maximum; O rows are rescaled only when the reference moves
        float factor = 1.f;
        if ((bm > m_ref + kLazyThreshold || m_ref == -INFINITY) && bm > -INFINITY) {
          factor = m_ref == -INFINITY ? 0.f : fast_exp2(m_ref - bm);
          m_ref = bm;
        }
        const bool rescale = sb > 0 && __any_sync(0xffffffffu, factor != 1.f);
        if (rescale) {
          // no P V of this tile may be accumulating into O: the previous sub-block's must have completed, and
          // the next one cannot start before this thread has arrived on p_full
          ok = __all_sync(0xffffffffu, mbar_wait(&bars.pv_done[u][(gg - 1) & 1], ((gg - 1) >> 1) & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(my_O + lane_addr + c * 32, r);
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
            tmem_st32(my_O + lane_addr + c * 32, r);
          }
        }
        l_sum *= factor;
        const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
        // P = exp2(scale*S - m), packed to 16 bits over the first half of this stream's S columns
        uint32_t pk[32];
        const uint64_t scale2 = f2_pack(scale_log2, scale_log2), negm2 = f2_pack(-m_use, -m_use);
        uint64_t ps2[4] = {0ull, 0ull, 0ull, 0ull};  // packed partial sums (bit pattern of +0, +0)
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float a0, a1, a2, a3;
          f2_unpack(f2_fma(f2_pack(__uint_as_float(r0[i]), __uint_as_float(r0[i + 1])), scale2, negm2), a0, a1);
          f2_unpack(f2_fma(f2_pack(__uint_as_float(r1[i]), __uint_as_float(r1[i + 1])), scale2, negm2), a2, a3);
          const float p0 = fast_exp2(a0), p1 = fast_exp2(a1), p2 = fast_exp2(a2);
          const float p3 = fast_exp2(a3);
          ps2[(i >> 1) & 1] = f2_add(ps2[(i >> 1) & 1], f2_pack(p0, p1));
          ps2[2 + ((i >> 1) & 1)] = f2_add(ps2[2 + ((i >> 1) & 1)], f2_pack(p2, p3));
          pk[i >> 1] = pack2<DT>(p0, p1);
          pk[16 + (i >> 1)] = pack2<DT>(p2, p3);
        }
        {
          float lo, hi;
          f2_unpack(f2_add(f2_add(ps2[0], ps2[1]), f2_add(ps2[2], ps2[3])), lo, hi);
          l_sum += lo + hi;
        }
        tmem_st32(s_addr, pk);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars.p_full[u][x]);
      }
      if (!ok) break;
      // epilogue: O / l leaves TMEM as packed 16-bit rows; O is then handed back to the MMA thread
      ok = __all_sync(0xffffffffu, mbar_wait(&bars.o_full[u], n & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
      const TileInfo ti = s_tiles[slot];
      mbar_arrive(&bars.tile_empty[slot]);
      const int i_row = ti.i_base + u * TOK + row / rep;
      const bool live_row = i_row < ti.n_sel;
      uint8_t* orow = ti.out + (((size_t)ti.l * ti.sel_capacity + i_row) * m.Hq + ti.hk * rep + row % rep) * (kD * 2);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(my_O + lane_addr + c * 32, r);
        if (c == 3) {  // O has left TMEM: the MMA thread may start the next pair's P V
          tc_fence_before();
          mbar_arrive(&bars.o_empty[u]);
        }
        if (live_row) {
#pragma unroll
          for (int i = 0; i < 32; i += 16) {
            uint32_t w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = pack2<DT>(__uint_as_float(r[i + 2 * j]) * inv, __uint_as_float(r[i + 2 * j + 1]) * inv);
            st_global_256(orow + (c * 32 + i) * 2, w);
          }
        }
      }
      g += nsb;
    }  // pairs
  }

  // ------------------------------------------------------------------ teardown (all roles)
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (tid == 0 && s_abort) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
}

constexpr size_t kSmemBytes = 2 * kTileBytes + 2 * kStages * kSubBytes + 1024;  // two Q tiles, kStages buffers of K and of V

}  // namespace

cudaError_t attention_dual_configure() {
  const void* fns[2] = {(const void*)attn_dual_kernel<KVB_DT_BF16>, (const void*)attn_dual_kernel<KVB_DT_F16>};
  for (const void* f : fns) {
    cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// total_pairs: pairs of neighbouring tiles over all requests (a request with an odd number of tiles ends in
// a pair whose second tile has no rows); the tensor maps are the one-tile kernel's
cudaError_t launch_attention_dual(const ReqDesc* reqs, const void* maps, int n_req, int total_pairs, const ModelDims& m, float scale,
                                  uint32_t* status, unsigned int* tile_counter, int n_sm, bool pdl, cudaStream_t st) {
  const long long work = (long long)total_pairs * m.Hkv * m.L;
  const float scale_log2 = scale * 1.4426950408889634f;
  const CUtensorMap* mp = static_cast<const CUtensorMap*>(maps);
  const unsigned grid = (unsigned)(work < (long long)n_sm ? work : (long long)n_sm);  // one CTA per SM
  if (m.dtype == KVB_DT_BF16)
    return launch_pdl(pdl, attn_dual_kernel<KVB_DT_BF16>, dim3(grid), dim3(kThreads), kSmemBytes, st, reqs, mp, n_req, total_pairs, m, scale_log2, status, tile_counter);
  return launch_pdl(pdl, attn_dual_kernel<KVB_DT_F16>, dim3(grid), dim3(kThreads), kSmemBytes, st, reqs, mp, n_req, total_pairs, m, scale_log2, status, tile_counter);
}

}  // namespace kvb
