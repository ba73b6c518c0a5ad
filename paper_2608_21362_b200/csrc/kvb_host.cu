// Host side of libkvb: context, table validation, descriptor packing, launches.
// Nothing here computes on the data path; every step of the path runs in the kernels.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <limits.h>
#include <string.h>

#include <new>
#include <vector>

#include "kvb_internal.h"
#include "pdl.cuh"

using namespace kvb;

namespace {
constexpr int kSlots = 4;  // pinned staging ring: a slot is reused only after its copy has completed
}

struct kvb_ctx {
  int device = 0;
  kvb_model_desc model{};
  kvb_limits limits{};
  ModelDims dims{};
  // device memory
  double* inv_freq = nullptr;            // [d/2]
  float2* cs_table = nullptr;            // [max_chunks][d/2] cos/sin of the chunk's rotation
  uint8_t* arena_dev = nullptr;          // descriptors of the current call
  unsigned long long* acc = nullptr;     // [max_tokens] fixed-point deviation sums (kept zero between calls)
  double* norm_sums = nullptr;           // [max_chunks][L][parts] key-norm sums of the stitch (importance by-product)
  uint32_t* status_dev = nullptr;
  // pinned staging ring
  uint8_t* staging = nullptr;
  cudaEvent_t slot_done[kSlots]{};
  bool slot_used[kSlots]{};
  int next_slot = 0;
  size_t arena_bytes = 0;
  bool acc_dirty = false;
  int n_sm = 0;
  // debug options (kvb_set_debug_option); the defaults are the product path
  bool attn_one_tile = false;  // one tile per attention CTA instead of persistent CTAs (cross-check)
  bool force_copy = false;     // descriptors always go by cudaMemcpyAsync (cross-check)
  bool pdl = true;             // programmatic dependent launch along the kernel chain
  bool attn_pair = false;      // attention on CTA pairs (tcgen05 cta_group::2) instead of single CTAs
  bool attn_dual = false;      // attention with two tiles per CTA sharing K/V, one CTA per SM
  cudaStream_t last_stream = nullptr;
  int64_t launches = 0;
  char err[512] = {0};
};

namespace {

int fail(kvb_ctx* c, int code, const char* fmt, ...) {
  if (c) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c->err, sizeof(c->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

int cuda_fail(kvb_ctx* c, cudaError_t e, const char* what) {
  return fail(c, KVB_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define KVB_CUDA(ctx, call)                                     \
  do {                                                          \
    cudaError_t e_ = (call);                                    \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call);    \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Takes the next staging slot (waiting for its previous copy if needed).
int take_slot(kvb_ctx* c, uint8_t** host) {
  const int s = c->next_slot;
  c->next_slot = (s + 1) % kSlots;
  if (c->slot_used[s]) KVB_CUDA(c, cudaEventSynchronize(c->slot_done[s]));
  *host = c->staging + (size_t)s * c->arena_bytes;
  return -(s + 1);  // negative = success, encodes the slot
}

// Sends the call's packed tables to the device arena.  Small tables ride in a kernel argument (the
// launch reads the host bytes before it returns, so the staging slot is free again at once) and, when
// rope_chunks > 0, the same kernel fills the rotation table: *rope_done tells the caller.  Larger
// tables are copied from the pinned slot, guarded by the slot's event.
int upload(kvb_ctx* c, int slot, const uint8_t* host, size_t bytes, cudaStream_t st, int rope_chunks = 0, bool* rope_done = nullptr) {
  if (rope_done) *rope_done = false;
  if (bytes <= kDescBlobBytes && !c->force_copy) {
    KVB_CUDA(c, launch_store_blob(host, bytes, c->arena_dev, rope_chunks, c->inv_freq, c->model.d / 2, c->cs_table, c->pdl, st));
    c->slot_used[slot] = false;
    c->launches += 1;
    if (rope_done) *rope_done = rope_chunks > 0;
    return KVB_OK;
  }
  KVB_CUDA(c, cudaMemcpyAsync(c->arena_dev, host, bytes, cudaMemcpyHostToDevice, st));
  KVB_CUDA(c, cudaEventRecord(c->slot_done[slot], st));
  c->slot_used[slot] = true;
  return KVB_OK;
}

// Checks one request's table: chunks in prompt order tiling [0, T) exactly, enums and pointers sane.
// need_fresh: the call reads the request's fresh tensor (the attention and the importance score do not).
int check_request(kvb_ctx* c, const kvb_request& r, int ri, bool need_payload, bool need_fresh) {
  const int C = c->model.chunk_tokens;
  if (r.T <= 0 || r.n_chunks <= 0 || !r.chunks) return fail(c, KVB_ERR_INVALID_ARG, "request %d: empty or NULL chunk table", ri);
  if (r.T % C != 0 || r.n_chunks != r.T / C)
    return fail(c, KVB_ERR_BAD_TABLE, "request %d: T=%d is not n_chunks=%d x chunk_tokens=%d", ri, r.T, r.n_chunks, C);
  if (!r.kv_buf || (need_fresh && !r.fresh)) return fail(c, KVB_ERR_INVALID_ARG, "request %d: NULL kv_buf or fresh", ri);
  if (!aligned16(r.kv_buf) || (need_fresh && !aligned16(r.fresh)))
    return fail(c, KVB_ERR_BAD_TABLE, "request %d: kv_buf / fresh must be 16-byte aligned", ri);
  for (int i = 0; i < r.n_chunks; ++i) {
    const kvb_chunk& k = r.chunks[i];
    if (k.n_tokens != C) return fail(c, KVB_ERR_BAD_TABLE, "request %d chunk %d: n_tokens=%d, expected %d", ri, i, k.n_tokens, C);
    if (k.new_pos != i * C)
      return fail(c, KVB_ERR_BAD_TABLE, "request %d chunk %d: new_pos=%d leaves a gap or overlap (expected %d)", ri, i, k.new_pos, i * C);
    if (k.mode < KVB_MODE_FRESH || k.mode > KVB_MODE_INT4) return fail(c, KVB_ERR_INVALID_ARG, "request %d chunk %d: bad mode %d", ri, i, k.mode);
    if (k.meta_fp16 != 0 && k.meta_fp16 != 1) return fail(c, KVB_ERR_INVALID_ARG, "request %d chunk %d: bad meta_fp16 %d", ri, i, k.meta_fp16);
    if (k.match < KVB_MATCH_MISS || k.match > KVB_MATCH_APPROX) return fail(c, KVB_ERR_INVALID_ARG, "request %d chunk %d: bad match %d", ri, i, k.match);
    if (k.mode == KVB_MODE_FRESH) continue;
    if (k.orig_pos < 0 || k.orig_pos >= (1 << 24) || k.new_pos >= (1 << 24))
      return fail(c, KVB_ERR_BAD_TABLE, "request %d chunk %d: position out of range [0, 2^24)", ri, i);
    if (k.match == KVB_MATCH_EXACT && k.orig_pos != k.new_pos)
      return fail(c, KVB_ERR_BAD_TABLE, "request %d chunk %d: EXACT match must keep its position (%d -> %d)", ri, i, k.orig_pos, k.new_pos);
    if (!need_payload) continue;
    if (!k.k_codes || !k.v_codes) return fail(c, KVB_ERR_INVALID_ARG, "request %d chunk %d: NULL codes", ri, i);
    if (!aligned16(k.k_codes) || !aligned16(k.v_codes)) return fail(c, KVB_ERR_BAD_TABLE, "request %d chunk %d: codes must be 16-byte aligned", ri, i);
    if (k.mode != KVB_MODE_FP16) {
      if (!k.k_meta || !k.v_meta) return fail(c, KVB_ERR_INVALID_ARG, "request %d chunk %d: NULL metadata", ri, i);
      if (!aligned16(k.k_meta) || !aligned16(k.v_meta)) return fail(c, KVB_ERR_BAD_TABLE, "request %d chunk %d: metadata must be 16-byte aligned", ri, i);
    }
  }
  return KVB_OK;
}

int check_batch(kvb_ctx* c, const kvb_request* reqs, int n_req, bool need_payload, int* chunks_total, int64_t* tokens_total,
                bool need_fresh = true) {
  if (!c) return KVB_ERR_INVALID_ARG;
  if (n_req < 0 || (n_req > 0 && !reqs)) return fail(c, KVB_ERR_INVALID_ARG, "bad request array");
  if (n_req > c->limits.max_requests) return fail(c, KVB_ERR_WORKSPACE, "%d requests > max_requests=%d", n_req, c->limits.max_requests);
  int ch = 0;
  int64_t tk = 0;
  for (int r = 0; r < n_req; ++r) {
    const int st = check_request(c, reqs[r], r, need_payload, need_fresh);
    if (st != KVB_OK) return st;
    ch += reqs[r].n_chunks;
    tk += reqs[r].T;
  }
  if (ch > c->limits.max_chunks_total) return fail(c, KVB_ERR_WORKSPACE, "%d chunks > max_chunks_total=%d", ch, c->limits.max_chunks_total);
  if (tk > c->limits.max_tokens_total) return fail(c, KVB_ERR_WORKSPACE, "%lld tokens > max_tokens_total=%lld", (long long)tk, (long long)c->limits.max_tokens_total);
  *chunks_total = ch;
  *tokens_total = tk;
  return KVB_OK;
}

}  // namespace

extern "C" {

const char* kvb_status_string(int s) {
  switch (s) {
    case KVB_OK: return "ok";
    case KVB_ERR_INVALID_ARG: return "invalid argument";
    case KVB_ERR_BAD_TABLE: return "bad chunk table";
    case KVB_ERR_UNSUPPORTED: return "unsupported shape or size";
    case KVB_ERR_WORKSPACE: return "call exceeds the context's limits";
    case KVB_ERR_CUDA: return "CUDA error";
    case KVB_ERR_DEVICE_STATUS: return "device-side status set";
    case KVB_ERR_NO_DEVICE: return "no usable GPU";
    default: return "unknown status";
  }
}

int kvb_select_count(int T, double ratio) {
  if (T <= 0 || !(ratio > 0.0)) return 0;
  const double k = floor(ratio * (double)T);
  return k >= (double)T ? T : (int)k;
}

int kvb_validate(const kvb_model_desc* model, const kvb_limits* limits, const kvb_request* reqs, int n_req,
                 int need_payload, char* err, size_t err_len) {
  if (!model || !limits) return KVB_ERR_INVALID_ARG;
  kvb_ctx tmp;  // no device resources: only the fields the checks read
  tmp.model = *model;
  tmp.limits = *limits;
  int ch = 0;
  int64_t tk = 0;
  const int st = check_batch(&tmp, reqs, n_req, need_payload != 0, &ch, &tk);
  if (err && err_len) snprintf(err, err_len, "%s", tmp.err);
  return st;
}

const char* kvb_last_error(kvb_ctx* c) { return c ? c->err : "NULL context"; }
int64_t kvb_launch_count(kvb_ctx* c) { return c ? c->launches : 0; }

int kvb_selftest_wait_timeout(kvb_ctx* c, int limit_ms, void* cuda_stream) {
  if (!c) return KVB_ERR_INVALID_ARG;
  if (limit_ms < 1 || limit_ms > 1000) return fail(c, KVB_ERR_INVALID_ARG, "limit_ms must be in 1..1000");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));
  KVB_CUDA(c, launch_wait_selftest(c->status_dev, (unsigned long long)limit_ms * 1000000ull, st));
  c->last_stream = st;
  c->launches += 1;
  return KVB_OK;
}

int kvb_create(kvb_ctx** out, int device, const kvb_model_desc* model, const kvb_limits* limits) {
  if (!out || !model || !limits) return KVB_ERR_INVALID_ARG;
  *out = nullptr;
  const kvb_model_desc& m = *model;
  if (m.L <= 0 || m.Hq <= 0 || m.Hkv <= 0 || m.Hq % m.Hkv != 0 || !(m.rope_theta > 1.0) ||
      (m.kv_dtype != KVB_DT_F16 && m.kv_dtype != KVB_DT_BF16) || limits->max_requests <= 0 ||
      limits->max_chunks_total <= 0 || limits->max_tokens_total <= 0)
    return KVB_ERR_INVALID_ARG;
  const int rep = m.Hq / m.Hkv;
  const bool pow2_h = (m.Hkv & (m.Hkv - 1)) == 0 && m.Hkv <= 16;
  const bool pow2_rep = (rep & (rep - 1)) == 0 && rep <= 16;
  if (m.d != 128 || m.chunk_tokens != 128 || m.int4_group != 32 || !pow2_h || !pow2_rep) return KVB_ERR_UNSUPPORTED;
  // the kernels index tokens, tiles and grid dimensions with 32 bits: a batch stays below 2^31 tokens
  // (and chunk-layers), L below the grid's y limit
  if (m.L > 65535 || limits->max_tokens_total > (int64_t)INT32_MAX || (int64_t)limits->max_chunks_total * m.L * 2 * m.Hkv > (int64_t)INT32_MAX)
    return KVB_ERR_UNSUPPORTED;

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return KVB_ERR_NO_DEVICE;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess || prop.major != 10) return KVB_ERR_NO_DEVICE;

  kvb_ctx* c = new (std::nothrow) kvb_ctx();
  if (!c) return KVB_ERR_CUDA;
  c->device = device;
  c->n_sm = prop.multiProcessorCount;
  c->model = m;
  c->limits = *limits;
  c->dims = ModelDims{m.L, m.Hq, m.Hkv, m.d, m.chunk_tokens, m.kv_dtype, m.int4_group};
  *out = c;  // handed out even on failure so the caller can read the error text and destroy it

  KVB_CUDA(c, cudaSetDevice(device));
  size_t smem_max = 0;
  for (int mode = KVB_MODE_FP16; mode <= KVB_MODE_INT4; ++mode) {
    const size_t s = assemble_smem_bytes(c->dims, mode);
    if (s > smem_max) smem_max = s;
  }
  if (smem_max > 200 * 1024) return fail(c, KVB_ERR_UNSUPPORTED, "chunk-layer block of %zu bytes does not fit shared memory", smem_max);
  KVB_CUDA(c, assemble_configure(smem_max));
  KVB_CUDA(c, topk_configure());
  KVB_CUDA(c, attention_tc_configure());
  KVB_CUDA(c, attention_pair_configure());
  KVB_CUDA(c, attention_dual_configure());
  KVB_CUDA(c, quantize_configure());

  const int half = m.d / 2;
  std::vector<double> inv(half);
  for (int j = 0; j < half; ++j) inv[j] = pow(m.rope_theta, -2.0 * (double)j / (double)m.d);
  KVB_CUDA(c, cudaMalloc(&c->inv_freq, half * sizeof(double)));
  KVB_CUDA(c, cudaMemcpy(c->inv_freq, inv.data(), half * sizeof(double), cudaMemcpyHostToDevice));
  KVB_CUDA(c, cudaMalloc(&c->cs_table, (size_t)limits->max_chunks_total * half * sizeof(float2)));

  const size_t a1 = sizeof(ChunkDesc) * (size_t)limits->max_chunks_total;
  const size_t a2 = (sizeof(ReqDesc) + 256) * (size_t)limits->max_requests + 384 + sizeof(SeamWindow) * (size_t)limits->max_chunks_total;
  c->arena_bytes = ((a1 + 255) & ~(size_t)255) + ((a2 + 255) & ~(size_t)255);  // the fused call uploads both tables
  static_assert(sizeof(QuantJob) <= sizeof(ChunkDesc), "a quantise job per chunk fits the chunk table's space");
  KVB_CUDA(c, cudaMalloc(&c->arena_dev, c->arena_bytes));
  KVB_CUDA(c, cudaMallocHost(&c->staging, c->arena_bytes * kSlots));
  for (int s = 0; s < kSlots; ++s) KVB_CUDA(c, cudaEventCreateWithFlags(&c->slot_done[s], cudaEventDisableTiming));
  KVB_CUDA(c, cudaMalloc(&c->acc, (size_t)limits->max_tokens_total * sizeof(unsigned long long)));
  KVB_CUDA(c, cudaMemset(c->acc, 0, (size_t)limits->max_tokens_total * sizeof(unsigned long long)));
  KVB_CUDA(c, cudaMalloc(&c->norm_sums, (size_t)limits->max_chunks_total * m.L * assemble_parts_per_layer(m.Hkv) * sizeof(double)));
  KVB_CUDA(c, cudaMalloc(&c->status_dev, sizeof(uint32_t)));
  KVB_CUDA(c, cudaMemset(c->status_dev, 0, sizeof(uint32_t)));
  KVB_CUDA(c, cudaDeviceSynchronize());
  return KVB_OK;
}

int kvb_set_debug_option(kvb_ctx* c, const char* key, int value) {
  if (!c || !key) return KVB_ERR_INVALID_ARG;
  if (value != 0 && value != 1) return fail(c, KVB_ERR_INVALID_ARG, "debug option values are 0 or 1");
  if (strcmp(key, "dependent_launch") == 0) c->pdl = value != 0;
  else if (strcmp(key, "descriptor_copy") == 0) c->force_copy = value != 0;
  else if (strcmp(key, "attention_one_tile_per_cta") == 0) c->attn_one_tile = value != 0;
  else if (strcmp(key, "attention_cta_pairs") == 0) c->attn_pair = value != 0;
  else if (strcmp(key, "attention_two_tiles") == 0) c->attn_dual = value != 0;
  else return fail(c, KVB_ERR_INVALID_ARG, "unknown debug option '%s'", key);
  return KVB_OK;
}

int kvb_destroy(kvb_ctx* c) {
  if (!c) return KVB_ERR_INVALID_ARG;
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  cudaFree(c->inv_freq);
  cudaFree(c->cs_table);
  cudaFree(c->arena_dev);
  cudaFree(c->acc);
  cudaFree(c->norm_sums);
  cudaFree(c->status_dev);
  if (c->staging) cudaFreeHost(c->staging);
  for (int s = 0; s < kSlots; ++s)
    if (c->slot_done[s]) cudaEventDestroy(c->slot_done[s]);
  delete c;
  return KVB_OK;
}

int kvb_last_status(kvb_ctx* c) {
  if (!c) return KVB_ERR_INVALID_ARG;
  KVB_CUDA(c, cudaSetDevice(c->device));
  KVB_CUDA(c, cudaStreamSynchronize(c->last_stream));
  uint32_t st = 0;
  KVB_CUDA(c, cudaMemcpy(&st, c->status_dev, sizeof(st), cudaMemcpyDeviceToHost));
  if (st) {
    KVB_CUDA(c, cudaMemset(c->status_dev, 0, sizeof(st)));  // reported once; the context stays usable
    return fail(c, KVB_ERR_DEVICE_STATUS, "device status word 0x%x%s%s%s", st, (st & DEV_STATUS_WAIT_TIMEOUT) ? " (a bounded wait ran out)" : "",
                (st & DEV_STATUS_BAD_DESC) ? " (a descriptor failed a device-side check)" : "",
                (st & DEV_STATUS_SEL_OVERFLOW) ? " (a selection did not fit sel_capacity)" : "");
  }
  return KVB_OK;
}

}  // extern "C"

namespace {

// One ChunkDesc per chunk of the batch; returns the largest shared-memory need.  The stitch kernel's
// CTAs start in descriptor order.  A small batch (a few waves of CTAs) puts its cached chunks
// (decode, rotate, compare) first and its FRESH chunks (plain copies, the cheapest CTAs) last, so that
// the kernel's last wave is made of short CTAs (cfg1: -6 % on the call).  A large batch keeps the
// request order: there the tail is nothing and copy CTAs running among the decoding ones balance the
// load/store and issue pipes better (cfg4: +3 % when sorted).
size_t pack_chunks(kvb_ctx* c, const kvb_request* reqs, int n_req, ChunkDesc* cd, bool* any_importance) {
  size_t smem = 0;
  *any_importance = false;
  int n = 0;
  long long n_chunks = 0;
  for (int r = 0; r < n_req; ++r) n_chunks += reqs[r].n_chunks;
  const bool fresh_last = n_chunks * c->model.L * 2 <= 16LL * 3 * c->n_sm;  // up to about 16 waves of 3 CTAs per SM
  for (int pass = 0; pass < 2; ++pass) {
    int tok = 0;
    for (int r = 0; r < n_req; ++r) {
      for (int i = 0; i < reqs[r].n_chunks; ++i) {
        const kvb_chunk& k = reqs[r].chunks[i];
        if (fresh_last ? (k.mode == KVB_MODE_FRESH) != (pass == 1) : pass == 1) continue;
        ChunkDesc d{};
        d.k_src = static_cast<const uint8_t*>(k.k_codes);
        d.v_src = static_cast<const uint8_t*>(k.v_codes);
        d.k_meta = static_cast<const float*>(k.k_meta);
        d.v_meta = static_cast<const float*>(k.v_meta);
        d.kv_buf = static_cast<uint8_t*>(reqs[r].kv_buf);
        d.fresh = static_cast<const uint8_t*>(reqs[r].fresh);
        d.T = reqs[r].T;
        d.new_pos = k.new_pos;
        d.delta_pos = k.mode == KVB_MODE_FRESH ? 0 : k.new_pos - k.orig_pos;
        d.mode = k.mode;
        d.tok_offset = tok;
        d.meta16 = k.meta_fp16;
        d.imp_out = reqs[r].importance ? reqs[r].importance + i : nullptr;
        if (d.imp_out) *any_importance = true;
        cd[n++] = d;
        const size_t s = assemble_smem_bytes(c->dims, k.mode);
        if (s > smem) smem = s;
      }
      tok += reqs[r].T;
    }
  }
  return smem;
}

int check_select_args(kvb_ctx* c, const kvb_select_params* p, const kvb_selection* out) {
  if (!p || !out) return fail(c, KVB_ERR_INVALID_ARG, "NULL select params or outputs");
  if ((p->which & 3) == 0 || (p->which & ~3) || p->seam_before < 0 || p->seam_after < 0 || p->sink_tokens < 0 ||
      (p->k_override < 0 && !(p->ratio >= 0.0 && p->ratio <= 1.0)))
    return fail(c, KVB_ERR_INVALID_ARG, "bad select params");
  return KVB_OK;
}

struct SelectExtent {
  int tiles = 0, n_seams = 0, max_T = 0, max_k = 0;
};

// One ReqDesc per request plus the batch's window list (seams, then the sink window, per request).
int pack_selection(kvb_ctx* c, const kvb_request* reqs, int n_req, const kvb_select_params* p, const kvb_selection* out,
                   ReqDesc* rd, SeamWindow* sw, SelectExtent* ext) {
  const int tile_tok = deviation_tile_tokens();
  int tiles = 0, tok = 0, n_seams = 0, max_T = 0, max_k = 0;
  for (int r = 0; r < n_req; ++r) {
    const kvb_request& q = reqs[r];
    const kvb_selection& o = out[r];
    if (!o.delta || !o.rank || !o.sel || !o.n_sel) return fail(c, KVB_ERR_INVALID_ARG, "request %d: NULL selection output", r);
    const int k = p->k_override >= 0 ? p->k_override : kvb_select_count(q.T, p->ratio);
    if (k > q.T) return fail(c, KVB_ERR_INVALID_ARG, "request %d: k=%d > T=%d", r, k, q.T);
    if (q.T > topk_max_T() || k > topk_max_k())
      return fail(c, KVB_ERR_UNSUPPORTED, "request %d: T=%d or k=%d beyond the selection kernel's limits (%d, %d)", r, q.T, k, topk_max_T(), topk_max_k());
    if (o.sel_capacity < k) return fail(c, KVB_ERR_INVALID_ARG, "request %d: sel_capacity=%d < k=%d", r, o.sel_capacity, k);
    ReqDesc d{};
    d.kv_buf = static_cast<const uint8_t*>(q.kv_buf);
    d.fresh = static_cast<const uint8_t*>(q.fresh);
    d.delta = o.delta;
    d.rank = o.rank;
    d.sel = o.sel;
    d.n_sel = o.n_sel;
    d.T = q.T;
    d.k = k;
    d.sel_capacity = o.sel_capacity;
    d.tok_offset = tok;
    d.tile_offset = tiles;
    d.seam_offset = n_seams;
    // seams: interior boundaries with a cached chunk on either side (Algorithm 1 works on cached chunks)
    for (int i = 1; i < q.n_chunks; ++i) {
      if (q.chunks[i].mode == KVB_MODE_FRESH && q.chunks[i - 1].mode == KVB_MODE_FRESH) continue;
      if (p->seam_before == 0 && p->seam_after == 0) continue;
      const int pos = q.chunks[i].new_pos;
      SeamWindow w;
      w.lo = pos - p->seam_before < 0 ? 0 : pos - p->seam_before;
      w.hi = pos + p->seam_after > q.T ? q.T : pos + p->seam_after;
      sw[n_seams++] = w;
    }
    if (p->sink_tokens > 0) {  // attention sinks: the first s positions, one more window
      SeamWindow w;
      w.lo = 0;
      w.hi = p->sink_tokens > q.T ? q.T : p->sink_tokens;
      sw[n_seams++] = w;
    }
    d.n_seams = n_seams - d.seam_offset;
    rd[r] = d;
    tok += q.T;
    tiles += (q.T + tile_tok - 1) / tile_tok;
    if (q.T > max_T) max_T = q.T;
    if (k > max_k) max_k = k;
  }
  ext->tiles = tiles, ext->n_seams = n_seams, ext->max_T = max_T, ext->max_k = max_k;
  return KVB_OK;
}

int clear_acc_if_dirty(kvb_ctx* c, cudaStream_t st) {
  if (c->acc_dirty) {
    KVB_CUDA(c, cudaMemsetAsync(c->acc, 0, (size_t)c->limits.max_tokens_total * sizeof(unsigned long long), st));
    c->acc_dirty = false;
  }
  return KVB_OK;
}

int n_deviation_terms(const kvb_ctx* c, int which) { return c->model.L * c->model.Hkv * ((which & 1) + ((which >> 1) & 1)); }

}  // namespace

extern "C" {

int kvb_assemble(kvb_ctx* c, const kvb_request* reqs, int n_req, void* cuda_stream) {
  int n_chunks = 0;
  int64_t n_tok = 0;
  const int st0 = check_batch(c, reqs, n_req, true, &n_chunks, &n_tok);
  if (st0 != KVB_OK) return st0;
  if (n_req == 0) return KVB_OK;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));

  uint8_t* host = nullptr;
  const int slot_code = take_slot(c, &host);
  if (slot_code >= 0) return slot_code;
  const int slot = -slot_code - 1;
  bool want_importance = false;
  const size_t smem = pack_chunks(c, reqs, n_req, reinterpret_cast<ChunkDesc*>(host), &want_importance);
  bool rope_done = false;
  const int up = upload(c, slot, host, sizeof(ChunkDesc) * (size_t)n_chunks, st, n_chunks, &rope_done);
  if (up != KVB_OK) return up;
  c->last_stream = st;
  const ChunkDesc* cd_dev = reinterpret_cast<const ChunkDesc*>(c->arena_dev);
  if (!rope_done) {
    KVB_CUDA(c, launch_rope_table(cd_dev, n_chunks, c->inv_freq, c->model.d / 2, c->cs_table, st));
    c->launches += 1;
  }
  KVB_CUDA(c, launch_assemble(cd_dev, n_chunks, c->cs_table, c->dims, smem, c->status_dev, 0, nullptr,
                              want_importance ? c->norm_sums : nullptr, c->pdl, st));
  c->launches += 1;
  if (want_importance) {
    KVB_CUDA(c, launch_importance_finalize(cd_dev, n_chunks, c->dims, c->norm_sums, st));
    c->launches += 1;
  }
  return KVB_OK;
}

int kvb_deviation_topk(kvb_ctx* c, const kvb_request* reqs, int n_req, const kvb_select_params* p,
                       const kvb_selection* out, void* cuda_stream) {
  int n_chunks = 0;
  int64_t n_tok = 0;
  const int st0 = check_batch(c, reqs, n_req, false, &n_chunks, &n_tok);
  if (st0 != KVB_OK) return st0;
  if (n_req == 0) return KVB_OK;
  const int st1 = check_select_args(c, p, out);
  if (st1 != KVB_OK) return st1;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));

  uint8_t* host = nullptr;
  const int slot_code = take_slot(c, &host);
  if (slot_code >= 0) return slot_code;
  const int slot = -slot_code - 1;
  ReqDesc* rd = reinterpret_cast<ReqDesc*>(host);
  SeamWindow* sw = reinterpret_cast<SeamWindow*>(host + sizeof(ReqDesc) * (size_t)n_req);
  SelectExtent ext;
  const int st2 = pack_selection(c, reqs, n_req, p, out, rd, sw, &ext);
  if (st2 != KVB_OK) return st2;
  const int st3 = clear_acc_if_dirty(c, st);
  if (st3 != KVB_OK) return st3;
  const int up = upload(c, slot, host, sizeof(ReqDesc) * (size_t)n_req + sizeof(SeamWindow) * (size_t)ext.n_seams, st);
  if (up != KVB_OK) return up;
  c->last_stream = st;
  const ReqDesc* rd_dev = reinterpret_cast<const ReqDesc*>(c->arena_dev);
  const SeamWindow* sw_dev = reinterpret_cast<const SeamWindow*>(c->arena_dev + sizeof(ReqDesc) * (size_t)n_req);
  c->acc_dirty = true;  // cleared again once both kernels are in the stream
  KVB_CUDA(c, launch_deviation(rd_dev, n_req, ext.tiles, c->dims, p->which, c->acc, st));
  KVB_CUDA(c, launch_topk(rd_dev, n_req, sw_dev, c->dims, n_deviation_terms(c, p->which), ext.max_T, ext.max_k, c->acc,
                          c->status_dev, c->pdl, st));
  c->acc_dirty = false;
  c->launches += 2;
  return KVB_OK;
}

int kvb_assemble_select(kvb_ctx* c, const kvb_request* reqs, int n_req, const kvb_select_params* p,
                        const kvb_selection* out, void* cuda_stream) {
  int n_chunks = 0;
  int64_t n_tok = 0;
  const int st0 = check_batch(c, reqs, n_req, true, &n_chunks, &n_tok);
  if (st0 != KVB_OK) return st0;
  if (n_req == 0) return KVB_OK;
  const int st1 = check_select_args(c, p, out);
  if (st1 != KVB_OK) return st1;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));

  uint8_t* host = nullptr;
  const int slot_code = take_slot(c, &host);
  if (slot_code >= 0) return slot_code;
  const int slot = -slot_code - 1;
  // arena: chunk descriptors, then (256-byte aligned) request descriptors and the window list
  const size_t rd_off = (sizeof(ChunkDesc) * (size_t)n_chunks + 255) & ~(size_t)255;
  const size_t sw_off = rd_off + sizeof(ReqDesc) * (size_t)n_req;
  bool want_importance = false;
  const size_t smem = pack_chunks(c, reqs, n_req, reinterpret_cast<ChunkDesc*>(host), &want_importance);
  SelectExtent ext;
  const int st2 = pack_selection(c, reqs, n_req, p, out, reinterpret_cast<ReqDesc*>(host + rd_off),
                                 reinterpret_cast<SeamWindow*>(host + sw_off), &ext);
  if (st2 != KVB_OK) return st2;
  const int st3 = clear_acc_if_dirty(c, st);
  if (st3 != KVB_OK) return st3;
  bool rope_done = false;
  const int up = upload(c, slot, host, sw_off + sizeof(SeamWindow) * (size_t)ext.n_seams, st, n_chunks, &rope_done);
  if (up != KVB_OK) return up;
  c->last_stream = st;
  const ChunkDesc* cd_dev = reinterpret_cast<const ChunkDesc*>(c->arena_dev);
  const ReqDesc* rd_dev = reinterpret_cast<const ReqDesc*>(c->arena_dev + rd_off);
  const SeamWindow* sw_dev = reinterpret_cast<const SeamWindow*>(c->arena_dev + sw_off);
  if (!rope_done) {
    KVB_CUDA(c, launch_rope_table(cd_dev, n_chunks, c->inv_freq, c->model.d / 2, c->cs_table, st));
    c->launches += 1;
  }
  c->acc_dirty = true;  // cleared again once both kernels are in the stream
  KVB_CUDA(c, launch_assemble(cd_dev, n_chunks, c->cs_table, c->dims, smem, c->status_dev, p->which, c->acc,
                              want_importance ? c->norm_sums : nullptr, c->pdl, st));
  KVB_CUDA(c, launch_topk(rd_dev, n_req, sw_dev, c->dims, n_deviation_terms(c, p->which), ext.max_T, ext.max_k, c->acc,
                          c->status_dev, c->pdl, st));
  c->acc_dirty = false;
  c->launches += 2;
  if (want_importance) {  // after the selection, so the dependent-launch chain stitch -> selection stays as it is
    KVB_CUDA(c, launch_importance_finalize(cd_dev, n_chunks, c->dims, c->norm_sums, st));
    c->launches += 1;
  }
  return KVB_OK;
}

int kvb_selective_attn(kvb_ctx* c, const kvb_request* reqs, int n_req, const kvb_selection* sel, const void* const* q,
                       void* const* out, float softmax_scale, void* cuda_stream) {
  int n_chunks = 0;
  int64_t n_tok = 0;
  const int st0 = check_batch(c, reqs, n_req, false, &n_chunks, &n_tok, false);
  if (st0 != KVB_OK) return st0;
  if (n_req == 0) return KVB_OK;
  if (!sel || !q || !out) return fail(c, KVB_ERR_INVALID_ARG, "NULL selection, q or out array");
  if (!(softmax_scale > 0.f)) return fail(c, KVB_ERR_INVALID_ARG, "softmax_scale must be positive");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));

  uint8_t* host = nullptr;
  const int slot_code = take_slot(c, &host);
  if (slot_code >= 0) return slot_code;
  const int slot = -slot_code - 1;
  ReqDesc* rd = reinterpret_cast<ReqDesc*>(host);
  const size_t maps_off = (sizeof(ReqDesc) * (size_t)n_req + 127) & ~(size_t)127;  // tensor maps: 2 x 128 bytes per request
  const int tok_per_tile = 128 / (c->model.Hq / c->model.Hkv);
  int tiles = 0;
  for (int r = 0; r < n_req; ++r) {
    const kvb_selection& s = sel[r];
    if (!s.sel || !s.n_sel || s.sel_capacity <= 0 || !q[r] || !out[r])
      return fail(c, KVB_ERR_INVALID_ARG, "request %d: NULL sel / n_sel / q / out or empty capacity", r);
    if (!aligned16(q[r]) || (reinterpret_cast<uintptr_t>(out[r]) & 31u) != 0)  // the output rows leave as 32-byte stores
      return fail(c, KVB_ERR_BAD_TABLE, "request %d: q must be 16-byte aligned, out 32-byte aligned", r);
    ReqDesc d{};
    d.kv_buf = static_cast<const uint8_t*>(reqs[r].kv_buf);
    d.sel = s.sel;
    d.n_sel = s.n_sel;
    d.q = static_cast<const uint8_t*>(q[r]);
    d.out = static_cast<uint8_t*>(out[r]);
    d.T = reqs[r].T;
    d.sel_capacity = s.sel_capacity;
    d.tile_offset = tiles;
    {  // (layer, head) pairs whose K and V planes (T * d * 2 * 2 bytes each) fit in about 48 MB of L2 together
      const int lh = c->model.L * c->model.Hkv;
      const double pair_bytes = (double)reqs[r].T * c->model.d * 4.0;
      int g0 = (int)(48.0e6 / pair_bytes);
      g0 = g0 < 1 ? 1 : (g0 > lh ? lh : g0);
      const int n_groups = (lh + g0 - 1) / g0;
      d.lhk_group = (lh + n_groups - 1) / n_groups;
    }
    rd[r] = d;
    const int tiles_r = (s.sel_capacity + tok_per_tile - 1) / tok_per_tile;
    tiles += (c->attn_pair || c->attn_dual) ? (tiles_r + 1) / 2 : tiles_r;  // these kernels count pairs of neighbouring tiles
    const int e = attention_tc_encode_maps(c->dims, q[r], s.sel_capacity, reqs[r].kv_buf, reqs[r].T, host + maps_off + 256 * (size_t)r);
    if (e != 0) return fail(c, KVB_ERR_CUDA, "request %d: tensor map encoding failed (%d)", r, e);
  }
  const size_t counter_off = maps_off + 256 * (size_t)n_req;  // the attention kernel's tile counter, uploaded as zero
  memset(host + counter_off, 0, 128);
  const int up = upload(c, slot, host, counter_off + 128, st);
  if (up != KVB_OK) return up;
  c->last_stream = st;
  const ReqDesc* rd_dev = reinterpret_cast<const ReqDesc*>(c->arena_dev);
  // persistent CTAs measured faster at every prompt length (most for short prompts, whose tiles are a
  // few sub-blocks long); the debug option selects one tile per CTA (cross-check)
  if (c->attn_pair)
    KVB_CUDA(c, launch_attention_pair(rd_dev, c->arena_dev + maps_off, n_req, (long long)tiles * c->model.Hkv * c->model.L, c->dims,
                                      softmax_scale, c->status_dev, c->n_sm, c->pdl, st));
  else if (c->attn_dual)
    KVB_CUDA(c, launch_attention_dual(rd_dev, c->arena_dev + maps_off, n_req, tiles, c->dims, softmax_scale, c->status_dev,
                                      reinterpret_cast<unsigned int*>(c->arena_dev + counter_off), c->n_sm, c->pdl, st));
  else
    KVB_CUDA(c, launch_attention_tc(rd_dev, c->arena_dev + maps_off, n_req, tiles, c->dims, softmax_scale, c->status_dev,
                                    reinterpret_cast<unsigned int*>(c->arena_dev + counter_off), c->n_sm, !c->attn_one_tile, c->pdl, st));
  c->launches += 1;
  return KVB_OK;
}

int kvb_patch(kvb_ctx* c, const kvb_request* reqs, int n_req, const kvb_selection* sel, void* cuda_stream) {
  int n_chunks = 0;
  int64_t n_tok = 0;
  const int st0 = check_batch(c, reqs, n_req, false, &n_chunks, &n_tok);
  if (st0 != KVB_OK) return st0;
  if (n_req == 0) return KVB_OK;
  if (!sel) return fail(c, KVB_ERR_INVALID_ARG, "NULL selection array");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));
  auto fill = [&](PatchDesc* out) -> int {
    for (int r = 0; r < n_req; ++r) {
      const kvb_selection& s = sel[r];
      if (!s.sel || !s.n_sel || s.sel_capacity <= 0) return fail(c, KVB_ERR_INVALID_ARG, "request %d: NULL sel / n_sel or empty capacity", r);
      out[r] = PatchDesc{static_cast<uint8_t*>(reqs[r].kv_buf), static_cast<const uint8_t*>(reqs[r].fresh), s.sel, s.n_sel, reqs[r].T, s.sel_capacity};
    }
    return KVB_OK;
  };
  if (n_req <= kPatchInline && !c->force_copy) {  // the descriptors travel as the kernel's argument
    PatchInline descs{};
    const int f = fill(descs.d);
    if (f != KVB_OK) return f;
    c->last_stream = st;
    KVB_CUDA(c, launch_patch_inline(descs, n_req, c->n_sm, c->dims, c->pdl, st));
  } else {
    uint8_t* host = nullptr;
    const int slot_code = take_slot(c, &host);
    if (slot_code >= 0) return slot_code;
    const int slot = -slot_code - 1;
    const int f = fill(reinterpret_cast<PatchDesc*>(host));
    if (f != KVB_OK) return f;
    const int up = upload(c, slot, host, sizeof(PatchDesc) * (size_t)n_req, st);
    if (up != KVB_OK) return up;
    c->last_stream = st;
    KVB_CUDA(c, launch_patch_table(reinterpret_cast<const PatchDesc*>(c->arena_dev), n_req, c->n_sm, c->dims, c->pdl, st));
  }
  c->launches += 1;
  return KVB_OK;
}

int kvb_chunk_importance(kvb_ctx* c, const kvb_request* reqs, int n_req, float* const* importance, void* cuda_stream) {
  int n_chunks = 0;
  int64_t n_tok = 0;
  const int st0 = check_batch(c, reqs, n_req, false, &n_chunks, &n_tok, false);
  if (st0 != KVB_OK) return st0;
  if (n_req == 0) return KVB_OK;
  if (!importance) return fail(c, KVB_ERR_INVALID_ARG, "NULL importance array");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));
  uint8_t* host = nullptr;
  const int slot_code = take_slot(c, &host);
  if (slot_code >= 0) return slot_code;
  const int slot = -slot_code - 1;
  ReqDesc* rd = reinterpret_cast<ReqDesc*>(host);
  int chunks = 0;
  for (int r = 0; r < n_req; ++r) {
    if (!importance[r]) return fail(c, KVB_ERR_INVALID_ARG, "request %d: NULL importance output", r);
    ReqDesc d{};
    d.kv_buf = static_cast<const uint8_t*>(reqs[r].kv_buf);
    d.delta = importance[r];  // the descriptor's float output slot
    d.T = reqs[r].T;
    d.tile_offset = chunks;
    rd[r] = d;
    chunks += reqs[r].n_chunks;
  }
  const int up = upload(c, slot, host, sizeof(ReqDesc) * (size_t)n_req, st);
  if (up != KVB_OK) return up;
  c->last_stream = st;
  KVB_CUDA(c, launch_importance(reinterpret_cast<const ReqDesc*>(c->arena_dev), n_req, chunks, c->dims, c->norm_sums, c->pdl, st));
  c->launches += 2;
  return KVB_OK;
}

int kvb_quantize_chunks(kvb_ctx* c, const kvb_quantize_job* jobs, int n_jobs, void* cuda_stream) {
  if (!c) return KVB_ERR_INVALID_ARG;
  if (n_jobs < 0 || (n_jobs > 0 && !jobs)) return fail(c, KVB_ERR_INVALID_ARG, "bad job array");
  if (n_jobs == 0) return KVB_OK;
  if ((size_t)n_jobs * sizeof(QuantJob) > c->arena_bytes)
    return fail(c, KVB_ERR_WORKSPACE, "%d jobs exceed the context's descriptor arena (%zu bytes)", n_jobs, c->arena_bytes);
  for (int i = 0; i < n_jobs; ++i) {
    const kvb_quantize_job& j = jobs[i];
    if ((!j.k && !j.v) || (j.bits != 4 && j.bits != 8) || (j.meta_fp16 != 0 && j.meta_fp16 != 1))
      return fail(c, KVB_ERR_INVALID_ARG, "job %d: bad quantize arguments", i);
    if (j.unrotate_from >= (1 << 24)) return fail(c, KVB_ERR_INVALID_ARG, "job %d: position %d out of range [0, 2^24)", i, j.unrotate_from);
    if ((j.k && (!j.k_codes || !j.k_meta)) || (j.v && (!j.v_codes || !j.v_meta)))
      return fail(c, KVB_ERR_INVALID_ARG, "job %d: NULL output", i);
    const void* ptrs[6] = {j.k, j.v, j.k_codes, j.v_codes, j.k_meta, j.v_meta};
    for (const void* p : ptrs)
      if (p && !aligned16(p)) return fail(c, KVB_ERR_BAD_TABLE, "job %d: quantize buffers must be 16-byte aligned", i);
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  KVB_CUDA(c, cudaSetDevice(c->device));
  uint8_t* host = nullptr;
  const int slot_code = take_slot(c, &host);
  if (slot_code >= 0) return slot_code;
  const int slot = -slot_code - 1;
  QuantJob* qj = reinterpret_cast<QuantJob*>(host);
  for (int i = 0; i < n_jobs; ++i) {
    const kvb_quantize_job& j = jobs[i];
    qj[i] = QuantJob{j.k, j.v, j.k_codes, j.v_codes, j.k_meta, j.v_meta, j.bits, j.unrotate_from, j.meta_fp16, 0};
  }
  const int up = upload(c, slot, host, sizeof(QuantJob) * (size_t)n_jobs, st);
  if (up != KVB_OK) return up;
  c->last_stream = st;
  KVB_CUDA(c, launch_quantize_batch(reinterpret_cast<const QuantJob*>(c->arena_dev), n_jobs, c->dims, c->inv_freq, c->status_dev, c->pdl, st));
  c->launches += 1;
  return KVB_OK;
}

int kvb_quantize_chunk_ex(kvb_ctx* c, const void* x, int is_value, int bits, int unrotate_from, int meta_fp16, void* codes,
                          void* meta, void* cuda_stream) {
  if (!c) return KVB_ERR_INVALID_ARG;
  if (!x || !codes || !meta) return fail(c, KVB_ERR_INVALID_ARG, "bad quantize arguments");
  if (unrotate_from >= 0 && is_value) return fail(c, KVB_ERR_INVALID_ARG, "values are never rotated");
  kvb_quantize_job j{};
  (is_value ? j.v : j.k) = x;
  (is_value ? j.v_codes : j.k_codes) = codes;
  (is_value ? j.v_meta : j.k_meta) = meta;
  j.bits = bits;
  j.unrotate_from = unrotate_from;
  j.meta_fp16 = meta_fp16;
  return kvb_quantize_chunks(c, &j, 1, cuda_stream);
}

int kvb_quantize_chunk(kvb_ctx* c, const void* x, int is_value, int bits, void* codes, void* meta, void* cuda_stream) {
  return kvb_quantize_chunk_ex(c, x, is_value, bits, -1, 0, codes, meta, cuda_stream);
}

int kvb_quantize_keys_at(kvb_ctx* c, const void* x, int orig_pos, int bits, void* codes, void* meta, void* cuda_stream) {
  if (c && orig_pos < 0) return fail(c, KVB_ERR_INVALID_ARG, "orig_pos=%d out of range [0, 2^24)", orig_pos);
  return kvb_quantize_chunk_ex(c, x, 0, bits, orig_pos, 0, codes, meta, cuda_stream);
}

}  // extern "C"
