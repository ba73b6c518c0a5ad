// Internal declarations shared by the host side of libkvb and its kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "kvb.h"

namespace kvb {

// Sticky device status bits (ORed into the context's status word by kernels).
enum : uint32_t {
  DEV_STATUS_WAIT_TIMEOUT = 1u << 0,  // a bounded mbarrier wait gave up
  DEV_STATUS_BAD_DESC = 1u << 1,      // a descriptor failed a device-side range check
  DEV_STATUS_SEL_OVERFLOW = 1u << 2,  // selection did not fit sel_capacity
};

// One chunk of one request, as the assemble kernel sees it (device memory).
struct ChunkDesc {
  const uint8_t* k_src;  // codes of all layers; unused for FRESH
  const uint8_t* v_src;
  const float* k_meta;
  const float* v_meta;
  uint8_t* kv_buf;       // request's [L][2][T][H][d] buffer
  const uint8_t* fresh;  // request's fresh tensor
  int32_t T;
  int32_t new_pos;
  int32_t delta_pos;     // new_pos - orig_pos
  int32_t mode;
  int32_t tok_offset;    // first token of the request in the call's flat token space
  int32_t meta16;        // (scale, min) pairs are binary16 instead of float32
  float* imp_out;        // where this chunk's importance score goes (NULL: not wanted)
};

// One request, as the deviation / top-k / attention kernels see it.
struct ReqDesc {
  const uint8_t* kv_buf;
  const uint8_t* fresh;
  float* delta;
  int32_t* rank;
  int32_t* sel;
  int32_t* n_sel;
  const uint8_t* q;
  uint8_t* out;
  int32_t T;
  int32_t k;             // number of top-k entries
  int32_t sel_capacity;
  int32_t tok_offset;    // first token of this request in the call's flat token space
  int32_t tile_offset;   // first tile of this request in a kernel's flat tile space
  int32_t seam_offset;   // first entry of this request in the seam window list
  int32_t n_seams;
  int32_t lhk_group;     // attention: (layer, head) pairs per scheduling group
};

struct PatchDesc {
  uint8_t* kv_buf;
  const uint8_t* fresh;
  const int32_t* sel;
  const int32_t* n_sel;
  int32_t T;
  int32_t sel_capacity;
};
constexpr int kPatchInline = 64;
struct PatchInline {
  PatchDesc d[kPatchInline];
};

struct SeamWindow {
  int32_t lo, hi;  // [lo, hi)
};

struct ModelDims {
  int L, Hq, Hkv, d, C, dtype, int4_group;
};

// ---- launchers (each defined next to its kernel) ----
// pdl: launch with the programmatic-dependent-launch attribute (csrc/pdl.cuh); a context option.
// Tables of at most kDescBlobBytes go to the arena as a kernel argument (csrc/desc_store.cu; two
// argument sizes, 3840 and 16384 bytes, so a small call does not pay for a large argument); the
// chunk descriptors, if any, must be at the start of the bytes, and n_rope_chunks > 0 also fills
// cs_table[n_rope_chunks][half_d] from their delta_pos.
constexpr size_t kDescBlobSmall = 3840;
constexpr size_t kDescBlobBytes = 16384;
cudaError_t launch_store_blob(const void* host_bytes, size_t bytes, uint8_t* dst, int n_rope_chunks, const double* inv_freq,
                              int half_d, float2* cs_table, bool pdl, cudaStream_t st);
// launch_assemble: acc != NULL fuses the deviation sums (which: bit 0 keys, bit 1 values) into the stitch;
// norm_sums != NULL ([n_chunks][L][assemble_parts_per_layer] doubles) also takes the key rows' norm sums,
// which launch_importance_finalize turns into the chunks' importance scores (ChunkDesc::imp_out).
cudaError_t launch_rope_table(const ChunkDesc* chunks, int n_chunks, const double* inv_freq, int half_d,
                              float2* cs_table, cudaStream_t st);
cudaError_t launch_assemble(const ChunkDesc* chunks, int n_chunks, const float2* cs_table, const ModelDims& m,
                            size_t smem_bytes, uint32_t* status, int which, unsigned long long* acc, double* norm_sums,
                            bool pdl, cudaStream_t st);
int assemble_parts_per_layer(int Hkv);
cudaError_t launch_importance_finalize(const ChunkDesc* chunks, int n_chunks, const ModelDims& m, const double* norm_sums,
                                       cudaStream_t st);
size_t assemble_smem_bytes(const ModelDims& m, int mode);
cudaError_t assemble_configure(size_t max_smem);

cudaError_t launch_deviation(const ReqDesc* reqs, int n_req, int total_tiles, const ModelDims& m, int which,
                             unsigned long long* acc, cudaStream_t st);
int deviation_tile_tokens();

cudaError_t launch_topk(const ReqDesc* reqs, int n_req, const SeamWindow* seams, const ModelDims& m, int n_terms,
                        int max_T, int max_k, unsigned long long* acc, uint32_t* status, bool pdl, cudaStream_t st);
cudaError_t topk_configure();
int topk_max_T();
int topk_max_k();

cudaError_t attention_tc_configure();
// One warp waits on a barrier nothing completes; gives up after limit_ns and raises DEV_STATUS_WAIT_TIMEOUT.
cudaError_t launch_wait_selftest(uint32_t* status, unsigned long long limit_ns, cudaStream_t st);
// Encodes the request's two TMA tensor maps (Q, KV) into out[0..255]; returns 0 on success.
int attention_tc_encode_maps(const ModelDims& m, const void* q, int sel_capacity, const void* kv_buf, int T, void* out);
// persistent: 2 CTAs per SM drawing tiles from *tile_counter (a zeroed device word), else one tile per CTA;
// n_sm: SMs of the device
cudaError_t launch_attention_tc(const ReqDesc* reqs, const void* maps, int n_req, int total_tiles, const ModelDims& m,
                                float scale, uint32_t* status, unsigned int* tile_counter, int n_sm, bool persistent,
                                bool pdl, cudaStream_t st);

// The paired form (csrc/attention_pair.cu): two tiles of one plane on two SMs per MMA.  total_pairs counts the
// call's tile pairs over all requests and planes; ReqDesc::tile_offset counts a request's tile pairs per plane.
// two neighbouring tiles per CTA, one CTA per SM (csrc/attention_dual.cu); tensor maps and tile counter as for the one-tile kernel
cudaError_t attention_dual_configure();
cudaError_t launch_attention_dual(const ReqDesc* reqs, const void* maps, int n_req, int total_pairs, const ModelDims& m, float scale,
                                  uint32_t* status, unsigned int* tile_counter, int n_sm, bool pdl, cudaStream_t st);
cudaError_t attention_pair_configure();
cudaError_t launch_attention_pair(const ReqDesc* reqs, const void* maps, int n_req, long long total_pairs, const ModelDims& m,
                                  float scale, uint32_t* status, int n_sm, bool pdl, cudaStream_t st);

// kvb_patch: one request's descriptor; up to kPatchInline of them travel as the kernel's own argument
cudaError_t launch_patch_inline(const PatchInline& descs, int n_req, int n_sm, const ModelDims& m, bool pdl, cudaStream_t st);
cudaError_t launch_patch_table(const PatchDesc* table, int n_req, int n_sm, const ModelDims& m, bool pdl, cudaStream_t st);
// part: [total_chunks][L] doubles of scratch (the per-layer sums); two launches
cudaError_t launch_importance(const ReqDesc* reqs, int n_req, int total_chunks, const ModelDims& m, double* part, bool pdl, cudaStream_t st);

// One chunk to quantise (device memory).  k / v NULL: that side is not wanted.
struct QuantJob {
  const void* k;
  const void* v;
  void* k_codes;
  void* v_codes;
  void* k_meta;
  void* v_meta;
  int32_t bits;
  int32_t unrotate_from;  // >= 0 (keys only): rotate back by R^(-unrotate_from) before quantising
  int32_t meta16;
  int32_t reserved;
};
// inv_freq: [d/2] doubles, device
cudaError_t launch_quantize_batch(const QuantJob* jobs, int n_jobs, const ModelDims& m, const double* inv_freq,
                                  uint32_t* status, bool pdl, cudaStream_t st);
cudaError_t quantize_configure();

}  // namespace kvb
