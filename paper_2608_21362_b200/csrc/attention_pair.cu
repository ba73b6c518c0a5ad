// Selected-row causal attention (Eq. 2) on the 5th-generation tensor cores, two SMs per MMA.
//
// Work unit: a tile = (layer, KV head, TOK = 128/rep selected tokens) x the rep = Hq/Hkv query
// heads sharing the KV head = 128 rows.  Two neighbouring tiles of one (layer, KV head) plane are
// processed by a pair of CTAs on two SMs (a thread-block cluster of 2) with tcgen05.mma
// .cta_group::2 (M = 256: 128 rows per CTA).  Keys go by sub-blocks of 128:
//     S = Q K^T   each CTA holds its own Q tile and HALF of the sub-block's keys (64) in shared
//                 memory; the tensor cores of both SMs read both halves, so every K byte crosses
//                 L2 -> shared memory once for 256 rows, and an MMA step reads 6 KB of operands per
//                 SM for 64 cycles of work (the unpaired N = 64 form needs 6 KB per 32 cycles,
//                 more than the shared-memory path delivers)
//     P = exp2(scale*S - m)   by 256 threads per CTA, two per row (64 columns each; the row maximum
//                 is exchanged through shared memory), written back over S as bf16 / fp16
//     O += P V    P from TMEM, V from shared memory: each CTA holds all 128 keys of the sub-block
//                 for HALF of the head dimension (64)
// One thread of the pair's first CTA issues all MMAs; tcgen05.commit with a cluster multicast
// signals the mbarriers of both CTAs.  Each CTA fetches its own operands with its own (non-
// multicast) TMA loads, whose completion bytes go to the first CTA's barriers.  Three S/P buffers
// and one O accumulator fill the 512 TMEM columns; three K and three V stages and two Q buffers
// sit in shared memory, so a tile's first Q K^T steps run under the previous tile's last P V.
// Tile pairs are dealt to the CTA pairs round-robin in the order: request, then groups of (layer,
// KV head) planes whose K/V fit L2 together, inside a group from the longest pair down -- both CTAs
// of a pair decode the same sequence on their own, no counter and no hand-over between them.
//
// The running maximum is lazy: the reference m only moves when a block's maximum exceeds it by
// more than 8 (a factor 256), in which case the O rows in TMEM are rescaled.
// Every wait is bounded; a wait that runs out raises an abort flag, all roles fall through to the
// common teardown (TMEM is released) and the context's status word records it.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kvb_internal.h"
#include "pdl.cuh"

namespace kvb {
namespace {

constexpr int kThreads = 320;                        // warp 0: TMA, warp 1: MMA, warps 2-9: softmax
constexpr int kRows = 128;
constexpr int kSubKeys = 128;                        // keys per sub-block (the pair's MMA N for S)
constexpr int kD = 128;
constexpr int kStages = 3;                           // K stages = V stages = S/P buffers
constexpr uint32_t kQBytes = kRows * kD * 2;         // 32 KB: a Q tile (two 64-wide boxes of 16 KB)
constexpr uint32_t kQHalf = kQBytes / 2;
constexpr uint32_t kKStage = (kSubKeys / 2) * kD * 2;  // 16 KB: this CTA's 64 keys, two 64-wide boxes of 8 KB
constexpr uint32_t kVStage = kSubKeys * (kD / 2) * 2;  // 16 KB: 128 keys x this CTA's 64 channels
constexpr uint32_t kTmemCols = 512;                  // S/P: 3 x 128 columns, O: columns 384..511
constexpr uint32_t kWaitHintNs = 20000;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // a wait that lasts two seconds gives up
constexpr float kLazyThreshold = 8.0f;
constexpr int kTileSlots = 4;                        // published tile records in flight

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}

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
// arrival on a barrier of another CTA of the cluster (address from map_to_rank)
// (the default release at CTA scope: what the arrival publishes -- tcgen05 stores and loads -- is ordered by
// the tcgen05 fences on both sides; a cluster-scope release costs over a thousand cycles per arrival)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
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
// Bounded wait; also gives up as soon as another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > kWaitLimitNs) break;
  }
  *abort_flag = 1;
  return false;
}

// ---- TMA: a load of this CTA's own operands whose completion bytes go to a barrier of the pair's
//      first CTA (bar_cluster: that barrier's cluster address).  No multicast.
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* map) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---- tcgen05, two CTAs per MMA
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// completion of all MMAs issued so far arrives on the barrier at this offset in BOTH CTAs of the pair
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  asm volatile(
      "{\n .reg .pred e;\n .reg .b16 m;\n mov.b16 m, 3;\n elect.sync _|e, 0xffffffff;\n"
      " @e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n}" ::"r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Load 32 columns of this thread's TMEM lane and wait for them (the wait sits in the same asm
// statement so that no use of the registers can be scheduled before it).
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

// Instruction descriptor: float32 accumulate, A/B bf16 or fp16, M = 256 over the pair, N = n.
template <int DT>
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, bool b_mn_major) {
  const uint32_t fmt = DT == KVB_DT_BF16 ? 1u : 0u;
  uint32_t d = 0;
  d |= 1u << 4;                      // D format f32
  d |= fmt << 7;                     // A format
  d |= fmt << 10;                    // B format
  d |= (b_mn_major ? 1u : 0u) << 16; // B major: 0 = K, 1 = MN
  d |= (n >> 3) << 17;               // N
  d |= (256u >> 4) << 24;            // M
  return d;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
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

// The barriers sit at the same offsets in both CTAs.  "first": waited on by the MMA thread, which
// lives in the pair's first CTA; the other CTA's copies of those are unused.
struct __align__(8) Barriers {
  uint64_t tile_full[kTileSlots], tile_empty[kTileSlots];  // local: a tile record is published / has been read
  uint64_t q_full[2];            // first: both CTAs' Q tiles have landed (transaction bytes of both)
  uint64_t q_empty[2];           // both (commit): the tile's S steps have read Q
  uint64_t k_full[kStages];      // first: both halves of the sub-block's keys have landed
  uint64_t v_full[kStages];      // first: both halves of the sub-block's values have landed
  uint64_t s_full[kStages];      // both (commit): S is in TMEM; the K stage is free again
  uint64_t pv_done[kStages];     // both (commit): P V has been accumulated; the V stage and the S/P buffer are free
  uint64_t p_full[kStages];      // first: all 16 softmax warps of the pair have written P
  uint64_t o_full;               // both (commit): the tile pair's last P V is done
  uint64_t o_empty;              // first: all 16 softmax warps of the pair have read O
  uint64_t xchg[4];              // local, per TMEM lane quarter: the two warps that share its rows have both arrived
};

// What a CTA's producer publishes for one tile pair.
struct TileInfo {
  const int32_t* sel;
  uint8_t* out;
  const CUtensorMap *map_q, *map_kv;
  int32_t n_sel, i_base, l, hk, nsb, sel_capacity;  // i_base: this CTA's tile; nsb: sub-blocks of the pair, 0 = no more tiles
};

// Tile pair number `lin` of the call -> this CTA's tile of it.  Order: request, then groups of
// rq.lhk_group (layer, KV head) planes, inside a group pair-major from the longest pair down with
// the group's planes interleaved.  false: the pair has no rows (both tiles lie past n_sel).
__device__ __forceinline__ bool decode_pair(long long lin, uint32_t rank, const ReqDesc* __restrict__ reqs, const CUtensorMap* maps,
                                            int n_req, int per_tile, int TOK, int Hkv, TileInfo& ti) {
  int lo = 0, hi = n_req - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((long long)reqs[mid].tile_offset * per_tile <= lin) lo = mid; else hi = mid - 1;
  }
  const ReqDesc& rq = reqs[lo];
  const int cap = rq.sel_capacity;
  const int pairs_r = ((cap + TOK - 1) / TOK + 1) >> 1;
  const int idx = (int)(lin - (long long)rq.tile_offset * per_tile);
  const int G = rq.lhk_group;
  const int grp = idx / (G * pairs_r);
  const int rem = idx - grp * G * pairs_r;
  const int g_eff = min(G, per_tile - grp * G);
  const int lhk = grp * G + rem % g_eff;
  const int pair = pairs_r - 1 - rem / g_eff;
  const int n_sel = min(*rq.n_sel, cap);
  const int first_row = 2 * pair * TOK;  // of the pair's first tile
  if (first_row >= n_sel) return false;
  const int t_max = min(rq.sel[min(first_row + 2 * TOK, n_sel) - 1], rq.T - 1);
  ti.sel = rq.sel;
  ti.out = rq.out;
  ti.n_sel = n_sel;
  ti.i_base = first_row + (int)rank * TOK;
  ti.l = lhk / Hkv;
  ti.hk = lhk % Hkv;
  ti.nsb = max(t_max, 0) / kSubKeys + 1;
  ti.sel_capacity = cap;
  ti.map_q = maps + 2 * lo;
  ti.map_kv = maps + 2 * lo + 1;
  return true;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 1)
    attn_pair_kernel(const ReqDesc* __restrict__ reqs, const CUtensorMap* __restrict__ maps, int n_req, long long total_pairs,
                     ModelDims m, float scale_log2, uint32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ Barriers bars;
  __shared__ TileInfo s_tiles[kTileSlots];
  __shared__ float s_max[2][2][kRows];   // [sub-block parity][column half][row]: the half-row maxima
  __shared__ float s_lsum[2][kRows];     // [column half][row]: the half-row sums at the end of a tile
  __shared__ uint32_t s_tmem_base;
  __shared__ uint32_t s_abort;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = cluster_rank();   // 0: the pair's first CTA (issues the MMAs, owns the "first" barriers)
  const bool first = rank == 0;
  const int per_tile = m.Hkv * m.L;
  const int rep = m.Hq / m.Hkv;
  const int TOK = kRows / rep;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                                   // 2 buffers of 32 KB
  uint8_t* sK = smem + 2 * kQBytes;                     // kStages x 16 KB
  uint8_t* sV = sK + kStages * kKStage;                 // kStages x 16 KB
  volatile uint32_t* abort_flag = &s_abort;

  if (tid == 64) {
    for (int i = 0; i < kTileSlots; ++i) {
      mbar_init(&bars.tile_full[i], 1);
      mbar_init(&bars.tile_empty[i], first ? 9 : 8);  // the 8 softmax warps, and the MMA warp where it runs
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.q_full[i], 1);
      mbar_init(&bars.q_empty[i], 1);
    }
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&bars.k_full[i], 1);
      mbar_init(&bars.v_full[i], 1);
      mbar_init(&bars.s_full[i], 1);
      mbar_init(&bars.pv_done[i], 1);
      mbar_init(&bars.p_full[i], 16);
    }
    mbar_init(&bars.o_full, 1);
    mbar_init(&bars.o_empty, 16);
    for (int i = 0; i < 4; ++i) mbar_init(&bars.xchg[i], 2);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // TMEM allocation: one warp of each CTA of the pair, together
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  // both CTAs' barriers exist before either CTA signals the other's
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
  tc_fence_after();
  const uint32_t tmem_base = s_tmem_base;
  const uint32_t tmem_O = tmem_base + kStages * kSubKeys;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      pdl_wait();  // descriptors, tensor maps and the selection come from the kernels before this one
      const long long n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;
      // barriers of the first CTA that this CTA's loads complete on
      const uint32_t q_full_c[2] = {map_to_rank(smem_u32(&bars.q_full[0]), 0), map_to_rank(smem_u32(&bars.q_full[1]), 0)};
      uint32_t k_full_c[kStages], v_full_c[kStages];
#pragma unroll
      for (int i = 0; i < kStages; ++i) {
        k_full_c[i] = map_to_rank(smem_u32(&bars.k_full[i]), 0);
        v_full_c[i] = map_to_rank(smem_u32(&bars.v_full[i]), 0);
      }
      bool ok = true;
      long long next_lin = cluster_id;  // this pair's tiles: cluster_id, cluster_id + n_clusters, ...
      int n_pub = 0;                    // tile records published
      bool stream_end = false;
      // decodes and publishes the pair's next tile record (nsb = 0 when there is none)
      auto publish_next = [&]() {
        TileInfo ti;
        ti.nsb = 0;
        while (next_lin < total_pairs) {
          const long long lin = next_lin;
          next_lin += n_clusters;
          if (decode_pair(lin, rank, reqs, maps, n_req, per_tile, TOK, m.Hkv, ti)) break;
          ti.nsb = 0;
        }
        const int slot = n_pub % kTileSlots;
        if (n_pub >= kTileSlots) ok = ok && mbar_wait(&bars.tile_empty[slot], ((n_pub / kTileSlots) & 1) ^ 1, abort_flag);
        if (!ok) return;
        s_tiles[slot] = ti;
        mbar_arrive(&bars.tile_full[slot]);
        if (ti.nsb == 0) stream_end = true;
        ++n_pub;
      };
      // two cursors over the same sequence of (tile, sub-block): the keys run kStages sub-blocks ahead of the values
      int kt = 0, ksb = 0, vt = 0, vsb = 0;  // tile number (of this pair), sub-block in it
      uint32_t gk = 0, gv = 0;               // sub-blocks issued so far
      bool k_end = false;
      auto next_k = [&]() {
        if (kt >= n_pub) publish_next();
        if (!ok) return;
        const TileInfo& ti = s_tiles[kt % kTileSlots];
        if (ti.nsb == 0) {
          k_end = true;
          return;
        }
        if (ksb == 0) {  // the tile's Q, into buffer kt & 1
          const int b = kt & 1;
          if (kt >= 2) ok = mbar_wait(&bars.q_empty[b], ((kt >> 1) & 1) ^ 1, abort_flag);  // tile kt - 2 has been read
          if (!ok) return;
          tensormap_acquire(ti.map_q);
          tensormap_acquire(ti.map_kv);
          if (first) mbar_expect_tx(&bars.q_full[b], 2 * kQBytes);
          tma_load_4d(sQ + b * kQBytes, ti.map_q, 0, ti.hk * rep, ti.i_base, ti.l, q_full_c[b]);
          tma_load_4d(sQ + b * kQBytes + kQHalf, ti.map_q, 64, ti.hk * rep, ti.i_base, ti.l, q_full_c[b]);
        }
        const int st = gk % kStages;
        if (gk >= kStages) ok = mbar_wait(&bars.s_full[st], ((gk / kStages) & 1) ^ 1, abort_flag);  // S(gk - 3) has read the stage
        if (!ok) return;
        if (first) mbar_expect_tx(&bars.k_full[st], 2 * kKStage);
        const int key0 = ksb * kSubKeys + (int)rank * (kSubKeys / 2);  // this CTA's half of the sub-block's keys
        tma_load_5d(sK + st * kKStage, ti.map_kv, 0, ti.hk, key0, 0, ti.l, k_full_c[st]);
        tma_load_5d(sK + st * kKStage + kKStage / 2, ti.map_kv, 64, ti.hk, key0, 0, ti.l, k_full_c[st]);
        ++gk;
        if (++ksb == ti.nsb) ksb = 0, ++kt;
      };
      auto next_v = [&]() {  // false: the stream has ended
        const TileInfo& ti = s_tiles[vt % kTileSlots];  // published: the key cursor is ahead (or at the end record)
        if (ti.nsb == 0) return false;
        const int st = gv % kStages;
        if (gv >= kStages) ok = mbar_wait(&bars.pv_done[st], ((gv / kStages) & 1) ^ 1, abort_flag);  // P V(gv - 3) is done
        if (!ok) return false;
        if (first) mbar_expect_tx(&bars.v_full[st], 2 * kVStage);
        // all 128 keys of the sub-block, this CTA's half of the head dimension: two 64-key boxes, one above the other
        const int d0 = (int)rank * (kD / 2);
        tma_load_5d(sV + st * kVStage, ti.map_kv, d0, ti.hk, vsb * kSubKeys, 1, ti.l, v_full_c[st]);
        tma_load_5d(sV + st * kVStage + kVStage / 2, ti.map_kv, d0, ti.hk, vsb * kSubKeys + 64, 1, ti.l, v_full_c[st]);
        ++gv;
        if (++vsb == ti.nsb) vsb = 0, ++vt;
        return true;
      };
      while (ok) {
        while (ok && !k_end && gk < gv + kStages) next_k();
        if (!ok) break;
        if (vt >= n_pub) publish_next();  // only at the very start of an empty stream
        if (!ok || !next_v()) break;
      }
      // every published record must include the end record, for the other roles to stop
      while (ok && !stream_end) publish_next();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (first CTA of the pair)
    if (first) {  // the whole warp runs the loop (its address arithmetic stays warp-uniform); one elected lane issues
      const uint32_t idesc_s = instr_desc<DT>(kSubKeys, false);
      const uint32_t idesc_pv = instr_desc<DT>(kD, true);
      const uint64_t q_desc = smem_desc(smem_u32(sQ), 16, 1024);
      const uint64_t k_desc = smem_desc(smem_u32(sK), 16, 1024);
      const uint64_t v_desc = smem_desc(smem_u32(sV), kVStage / 2, 1024);
      bool ok = true;
      // S(g) = Q K^T into S buffer g % 3: 8 steps of 16 channels
      auto issue_s = [&](uint32_t g, int q_buf) {
        const int st = g % kStages;
        if (!mbar_wait(&bars.k_full[st], (g / kStages) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint64_t qd = q_desc + (uint64_t)(q_buf * (kQBytes >> 4));
        const uint64_t kd = k_desc + (uint64_t)(st * (kKStage >> 4));
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {  // 4 steps per 64-wide box
          const uint32_t qo = (ks >> 2) * kQHalf + (ks & 3) * 32;
          const uint32_t ko = (ks >> 2) * (kKStage / 2) + (ks & 3) * 32;
          mma_ss(tmem_base + st * kSubKeys, qd + (qo >> 4), kd + (ko >> 4), idesc_s, ks > 0);
        }
        tc_commit_pair(&bars.s_full[st]);
        return true;
      };
      // O (+)= P(g) V(g): 8 steps of 16 keys; P sits in the first 32 columns of each half of the S buffer
      auto issue_pv = [&](uint32_t g, bool first_of_tile) {
        const int st = g % kStages;
        const uint32_t ph = (g / kStages) & 1;
        if (!mbar_wait(&bars.p_full[st], ph, abort_flag) || !mbar_wait(&bars.v_full[st], ph, abort_flag)) return false;
        tc_fence_after();
        const uint64_t vd = v_desc + (uint64_t)(st * (kVStage >> 4));
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {  // 16 keys = 2048 bytes of this CTA's V half
          const uint32_t p_col = (ks >> 2) * 64 + (ks & 3) * 8;
          mma_ts(tmem_O, tmem_base + st * kSubKeys + p_col, vd + (uint64_t)((ks * 2048) >> 4), idesc_pv, !(first_of_tile && ks == 0));
        }
        tc_commit_pair(&bars.pv_done[st]);
        return true;
      };
      // Two cursors over the sequence of sub-blocks: S runs up to kStages ahead of P V, across tile boundaries.
      int st_tile = 0, s_sb = 0, s_nsb = -1;  // S cursor: tile, sub-block, the tile's sub-blocks (-1: not read yet)
      int pv_tile = 0, pv_sb = 0;
      int nsb_of[kTileSlots];                 // sub-blocks of the tiles between the cursors
      uint32_t gs = 0, gp = 0;
      bool s_end = false;
      for (;;) {
        while (ok && !s_end && gs < gp + kStages) {
          if (s_nsb < 0) {  // the next tile's record
            const int slot = st_tile % kTileSlots;
            ok = mbar_wait(&bars.tile_full[slot], (st_tile / kTileSlots) & 1, abort_flag);
            if (!ok) break;
            s_nsb = s_tiles[slot].nsb;
            nsb_of[slot] = s_nsb;
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.tile_empty[slot]);
            if (s_nsb == 0) {
              s_end = true;
              break;
            }
            ok = mbar_wait(&bars.q_full[st_tile & 1], (st_tile >> 1) & 1, abort_flag);
            if (!ok) break;
          }
          ok = issue_s(gs, st_tile & 1);
          if (!ok) break;
          ++gs;
          if (++s_sb == s_nsb) {
            tc_commit_pair(&bars.q_empty[st_tile & 1]);  // the tile's S steps are issued: Q is free once they complete
            s_sb = 0, s_nsb = -1, ++st_tile;
          }
        }
        if (!ok || gp == gs) break;  // nothing left to accumulate: the stream has ended
        if (pv_sb == 0 && pv_tile > 0) {  // the tile's first P V overwrites O: the previous tile's epilogue must have read it
          ok = mbar_wait(&bars.o_empty, (pv_tile - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
        }
        ok = issue_pv(gp, pv_sb == 0);
        if (!ok) break;
        ++gp;
        if (++pv_sb == nsb_of[pv_tile % kTileSlots]) {
          tc_commit_pair(&bars.o_full);
          pv_sb = 0, ++pv_tile;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (warps 2..9)
    const int quarter = warp & 3;              // TMEM lanes this warp may touch
    const int half = warp >= 6 ? 1 : 0;        // which 64 columns of a sub-block (and of O) this thread handles
    const int row = quarter * 32 + lane;       // row of the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const uint32_t p_full_c = map_to_rank(smem_u32(&bars.p_full[0]), 0);  // + 8 * stage
    const uint32_t o_empty_c = map_to_rank(smem_u32(&bars.o_empty), 0);
    bool ok = true;
    uint32_t g = 0;   // sub-blocks of the tiles before this one
    uint32_t xc = 0;  // meetings with the warp that handles the other half of this quarter's rows
    // The two warps of a quarter meet (a bounded wait, like every other): what each wrote to shared
    // memory before is visible to the other afterwards.
    auto meet = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.xchg[quarter]);
      const bool done = __all_sync(0xffffffffu, mbar_wait(&bars.xchg[quarter], xc & 1, abort_flag));
      ++xc;
      return done;
    };
    for (int n = 0; ok; ++n) {
      const int slot = n % kTileSlots;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars.tile_full[slot], (n / kTileSlots) & 1, abort_flag));
      if (!ok) break;
      const int nsb = s_tiles[slot].nsb;
      if (nsb == 0) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.tile_empty[slot]);
        break;
      }
      int t_row;
      {
        const int i_row = s_tiles[slot].i_base + row / rep;
        t_row = i_row < s_tiles[slot].n_sel ? s_tiles[slot].sel[i_row] : -1;
      }
      int warp_tmin = t_row;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) warp_tmin = min(warp_tmin, __shfl_xor_sync(0xffffffffu, warp_tmin, o));
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int sb = 0; sb < nsb; ++sb) {
        const uint32_t gg = g + sb;
        const int st = gg % kStages;
        ok = __all_sync(0xffffffffu, mbar_wait(&bars.s_full[st], (gg / kStages) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        const int key0 = sb * kSubKeys + half * 64;
        const bool need_mask = key0 + 63 > warp_tmin;
        const uint32_t s_addr = tmem_base + lane_addr + st * kSubKeys + half * 64;
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
        // the row's maximum over all 128 columns: the two threads of a row exchange their halves
        const float my_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        s_max[gg & 1][half][row] = my_max;
        ok = meet();
        if (!ok) break;
        const float bm = fmaxf(my_max, s_max[gg & 1][half ^ 1][row]) * scale_log2;  // scale > 0 commutes with max
        // lazy reference maximum (both threads of a row take the same decision); O rows are rescaled only when it moves
        float factor = 1.f;
        if ((bm > m_ref + kLazyThreshold || m_ref == -INFINITY) && bm > -INFINITY) {
          factor = m_ref == -INFINITY ? 0.f : fast_exp2(m_ref - bm);
          m_ref = bm;
        }
        const bool rescale = sb > 0 && __any_sync(0xffffffffu, factor != 1.f);
        if (rescale) {
          // no P V may be accumulating into O: the previous sub-block's must have completed, and the
          // next one cannot start before this thread has arrived on p_full
          const uint32_t gp = gg - 1;
          ok = __all_sync(0xffffffffu, mbar_wait(&bars.pv_done[gp % kStages], (gp / kStages) & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < 2; ++c) {  // this thread's 64 columns of the O row
            uint32_t r[32];
            tmem_ld32(tmem_O + lane_addr + half * 64 + c * 32, r);
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * factor);
            tmem_st32(tmem_O + lane_addr + half * 64 + c * 32, r);
          }
        }
        l_sum *= factor;
        const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
        // P = exp2(scale*S - m), packed to 16 bits over the first 32 of this thread's 64 columns
        uint32_t pk[32];
        const uint64_t scale2 = f2_pack(scale_log2, scale_log2), negm2 = f2_pack(-m_use, -m_use);
        uint64_t ps2[4] = {0ull, 0ull, 0ull, 0ull};
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
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(p_full_c + 8u * st);
      }
      if (!ok) break;
      // epilogue: this thread's 64 columns of O / l leave TMEM as packed 16-bit values; O is then handed back
      // to the MMA thread, whose next tile's first P V overwrites it
      s_lsum[half][row] = l_sum;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars.o_full, n & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      ok = meet();
      if (!ok) break;
      const float l_row = s_lsum[0][row] + s_lsum[1][row];
      const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
      const TileInfo ti = s_tiles[slot];
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.tile_empty[slot]);
      const int i_row = ti.i_base + row / rep;
      const bool live_row = i_row < ti.n_sel;
      uint8_t* orow = ti.out + (((size_t)ti.l * ti.sel_capacity + i_row) * m.Hq + ti.hk * rep + row % rep) * (kD * 2) + half * 128;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_O + lane_addr + half * 64 + c * 32, r);
        if (c == 1) {  // O has left TMEM: the MMA thread may start the next tile's P V
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(o_empty_c);
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
      ok = meet();  // s_lsum has been read before the next tile overwrites it
      g += nsb;
    }  // tiles
  }

  // ------------------------------------------------------------------ teardown (all roles)
  tc_fence_before();
  __syncthreads();
  // neither CTA frees its TMEM or leaves while the other may still signal its barriers or run MMAs on it
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
  if (tid == 0 && s_abort) atomicOr(status, DEV_STATUS_WAIT_TIMEOUT);
}

constexpr size_t kSmemBytes = 2 * kQBytes + kStages * (kKStage + kVStage) + 1024;

}  // namespace

cudaError_t attention_pair_configure() {
  const void* fns[2] = {(const void*)attn_pair_kernel<KVB_DT_BF16>, (const void*)attn_pair_kernel<KVB_DT_F16>};
  for (const void* f : fns) {
    cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// total_pairs: tile pairs of the call over all requests, (layer, KV head) planes included
// (ReqDesc::tile_offset counts a request's tile pairs per plane).
cudaError_t launch_attention_pair(const ReqDesc* reqs, const void* maps, int n_req, long long total_pairs, const ModelDims& m,
                                  float scale, uint32_t* status, int n_sm, bool pdl, cudaStream_t st) {
  const float scale_log2 = scale * 1.4426950408889634f;
  const CUtensorMap* mp = static_cast<const CUtensorMap*>(maps);
  const long long clusters = total_pairs < n_sm / 2 ? total_pairs : n_sm / 2;
  if (clusters <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * clusters));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  if (m.dtype == KVB_DT_BF16) return cudaLaunchKernelEx(&cfg, attn_pair_kernel<KVB_DT_BF16>, reqs, mp, n_req, total_pairs, m, scale_log2, status);
  return cudaLaunchKernelEx(&cfg, attn_pair_kernel<KVB_DT_F16>, reqs, mp, n_req, total_pairs, m, scale_log2, status);
}

}  // namespace kvb
