/*
 * kvb.h -- C ABI of libkvb: stitching independently cached KV chunks into one
 * request's KV buffer, and choosing and attending the tokens to recompute.
 *
 * All entry points are plain C.  "device" pointers are CUDA global-memory
 * addresses on the context's GPU and are owned by the caller; "host" pointers
 * are ordinary process memory.  Tables passed by host pointer are consumed
 * (copied) before the call returns.  The three data-path calls are
 * asynchronous on the CUDA stream given (a cudaStream_t passed as void*), do
 * not synchronise, and allocate nothing: the only allocations happen in
 * kvb_create.  All calls on one context must be issued to one stream (or be
 * ordered by the caller), because they share the context's descriptor arena
 * and scratch.
 *
 * Errors: every call returns a kvb_status.  Tables are checked on the host
 * before anything is launched; a rejected call launches nothing.  Device code
 * never traps: a kernel that meets something it cannot process skips it and
 * sets a sticky status word that kvb_last_status reads back.
 *
 * Tensor layouts (row-major, last index fastest; L layers, H = Hkv KV heads,
 * d head_dim, T prompt tokens, C chunk_tokens):
 *   KV buffer / fresh tensor  [L][2][T][H][d]  16-bit (bf16 or fp16), 0 = keys, 1 = values
 *                             -- the prefill KV tensor shape of the paper's
 *                             "Transformer KV Cache" section
 *   cached chunk, keys/values INT8: [L][C][H][d] u8 codes
 *                             INT4: [L][C][H][d/2] bytes, channel 2i in the low
 *                                   nibble and 2i+1 in the high nibble of byte i
 *                             FP16: [L][C][H][d] in the buffer's 16-bit dtype
 *   key metadata              [L][G_k][H][d][2] float32 (scale, min); statistics per
 *                             channel over a token group: G_k = 1 for INT8 (the whole
 *                             chunk), C/int4_group for INT4
 *   value metadata            [L][C][H][G_v][2] float32 (scale, min); statistics per token
 *                             over a channel group: G_v = 1 for INT8, d/int4_group for INT4
 *   compact metadata          the same two layouts with IEEE binary16 (scale, min) pairs
 *                             (4 bytes per pair), chunk flag meta_fp16 = 1: min rounded
 *                             down and scale rounded up to binary16 when the chunk is
 *                             quantised, codes taken against the rounded pair
 * Cached keys are stored already rotated (RoPE) at absolute positions
 * orig_pos .. orig_pos+C-1, as a prefill pass leaves them.
 */
#ifndef KVB_H_
#define KVB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvb_ctx kvb_ctx; /* opaque */

typedef enum {
  KVB_OK = 0,
  KVB_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, bad enum */
  KVB_ERR_BAD_TABLE = 2,     /* chunk table does not tile [0,T), misaligned pointer, bad position */
  KVB_ERR_UNSUPPORTED = 3,   /* shape or size outside what the kernels are built for */
  KVB_ERR_WORKSPACE = 4,     /* call exceeds the limits given to kvb_create */
  KVB_ERR_CUDA = 5,          /* a CUDA runtime call failed (kvb_last_error has the text) */
  KVB_ERR_DEVICE_STATUS = 6, /* a kernel reported a problem (sticky) */
  KVB_ERR_NO_DEVICE = 7      /* no usable sm_100 GPU */
} kvb_status;

typedef enum {
  KVB_MODE_FRESH = 0, /* not cached: rows are taken bit for bit from the request's fresh tensor */
  KVB_MODE_FP16 = 1,  /* cached, unquantised, in the buffer's 16-bit dtype */
  KVB_MODE_INT8 = 2,
  KVB_MODE_INT4 = 3
} kvb_mode;

/* Outcome of the lookup cascade (EXACT via prefix hash, APPROX via content hash, MISS). */
typedef enum { KVB_MATCH_MISS = 0, KVB_MATCH_EXACT = 1, KVB_MATCH_APPROX = 2 } kvb_match;

typedef enum { KVB_DT_F16 = 0, KVB_DT_BF16 = 1 } kvb_dtype;

/* One row of a request's chunk table (host memory).  Mirrors the cached-chunk
 * record of the paper's implementation section: both hashes, the absolute
 * position the chunk was cached at, and where it goes in this prompt. */
typedef struct {
  uint8_t content_hash[32]; /* SHA-256 of the token ids (Dual-Hash Keying, Eq. 5); opaque here */
  uint8_t prefix_hash[32];  /* chained SHA-256 (Eq. 4); opaque here */
  int32_t orig_pos;         /* absolute position of the chunk's first token when it was cached */
  int32_t new_pos;          /* position of its first token in this prompt */
  int32_t n_tokens;         /* must equal the model's chunk_tokens */
  int32_t mode;             /* kvb_mode */
  int32_t match;            /* kvb_match; EXACT requires orig_pos == new_pos */
  int32_t meta_fp16;        /* 0: float32 (scale, min) pairs; 1: binary16 pairs (INT8 / INT4 chunks) */
  const void* k_codes;      /* device; NULL for FRESH */
  const void* v_codes;      /* device; NULL for FRESH */
  const void* k_meta;       /* device; INT8 / INT4 only */
  const void* v_meta;       /* device; INT8 / INT4 only */
} kvb_chunk;

/* One request.  Its chunks, sorted by new_pos, must tile [0, T) exactly. */
typedef struct {
  int32_t T;
  int32_t n_chunks;
  const kvb_chunk* chunks; /* host */
  void* kv_buf;            /* device, [L][2][T][H][d], written by kvb_assemble */
  const void* fresh;       /* device, same shape and dtype: freshly projected K~, V~ of every position */
  float* importance;       /* device, optional (NULL: not wanted): [n_chunks] float32.  kvb_assemble and
                              kvb_assemble_select write every chunk's importance score (KV Cache Manager,
                              Eq. 7: mean L2 norm of the chunk's stitched keys over layers, KV heads and
                              tokens) from the key rows they hold while stitching; other calls ignore it */
} kvb_request;

typedef struct {
  int32_t L, Hq, Hkv, d;
  int32_t chunk_tokens;    /* C */
  int32_t kv_dtype;        /* kvb_dtype of the KV buffer, the fresh tensor, FP16-mode chunks, Q and O */
  int32_t int4_group;      /* tokens per key group and channels per value group in INT4 mode */
  int32_t reserved;
  double rope_theta;
} kvb_model_desc;

/* Upper bounds for ONE call; they size what kvb_create allocates. */
typedef struct {
  int32_t max_requests;
  int32_t max_chunks_total;
  int64_t max_tokens_total;
} kvb_limits;

typedef struct {
  double ratio;        /* rho: k = floor(ratio * T) */
  int32_t k_override;  /* >= 0: use this k instead */
  int32_t seam_before; /* R of Algorithm 1: window [p-before, p+after) around each seam p */
  int32_t seam_after;
  int32_t which;       /* bit 0: keys (the printed deviation formula); bit 1: values */
  int32_t sink_tokens; /* attention-sink tokens (Tokenization and Chunking): the first s positions of the
                          prompt are always selected; 0 = off */
  int32_t reserved;
} kvb_select_params;

/* Per-request outputs of the selection (device memory, caller-owned). */
typedef struct {
  float* delta;         /* [T]  cosine deviation of every position */
  int32_t* rank;        /* [k]  the k most deviated positions, most deviated first (ties: lower index) */
  int32_t* sel;         /* [sel_capacity] ascending union of rank[0..k) and the seam windows */
  int32_t* n_sel;       /* [1]  number of valid entries of sel */
  int32_t sel_capacity; /* >= k + seam tokens, or T */
  int32_t reserved;
} kvb_selection;

/* Creates a context on `device` (a CUDA ordinal).  Allocates the descriptor
 * arena (pinned host + device) and the deviation scratch for the given limits.
 * KVB_ERR_UNSUPPORTED for shapes the kernels are not built for (d, chunk_tokens
 * other than 128, int4_group other than 32, head counts that are not powers of
 * two up to 16, L > 65535) and for limits beyond 2^31-1 tokens per call. */
int kvb_create(kvb_ctx** out, int device, const kvb_model_desc* model, const kvb_limits* limits);
int kvb_destroy(kvb_ctx* ctx);

/* Prompt Assembly, CHUNK_REUSE mode, with the steps the paper places before it
 * fused in: for every cached chunk, dequantise (inverse of KV Quantization
 * Eq. 6: x = code*scale + min; keys per channel, values per token), rotate the
 * keys by R_theta^(new_pos - orig_pos) (the correction the Rotary Positional
 * Embeddings section calls for; values are not rotated), and write rows
 * new_pos .. new_pos+C-1 of every layer of kv_buf.  FRESH chunks copy the
 * rows of `fresh`.  reqs: host array of n_req requests. */
int kvb_assemble(kvb_ctx* ctx, const kvb_request* reqs, int n_req, void* cuda_stream);

/* CacheBlendRecompute (Algorithm 2) steps 2 and 3 plus the token set of
 * SelectiveRecompute (Algorithm 1):
 *   delta_t = 1 - mean over layers, KV heads (and K/V per `which`) of
 *             cos(kv_buf row, fresh row);
 *   rank    = the floor(ratio*T) largest delta_t, ties broken by lower index;
 *   sel     = ascending union of rank and [p-before, p+after) for every seam p
 *             (an interior chunk boundary with a cached chunk on either side).
 * out: host array of n_req kvb_selection (device pointers inside). */
int kvb_deviation_topk(kvb_ctx* ctx, const kvb_request* reqs, int n_req, const kvb_select_params* params,
                       const kvb_selection* out, void* cuda_stream);

/* kvb_assemble followed by kvb_deviation_topk, with the deviation sums taken
 * while the stitched rows are still in registers, so kv_buf is written once and
 * never read back and `fresh` is read once (Prompt Assembly + Algorithm 2 steps
 * 2-3 + the token set of Algorithm 1 in one pass over the chunk store).
 * Writes the same kv_buf as kvb_assemble; delta agrees with the two-call
 * path to float32 rounding of the per-row sums (a few 1e-7), and rank / sel
 * are the selection of this call's delta.  Arguments and errors as for the
 * two calls; chunks need their payload pointers. */
int kvb_assemble_select(kvb_ctx* ctx, const kvb_request* reqs, int n_req, const kvb_select_params* params,
                        const kvb_selection* out, void* cuda_stream);

/* Causal attention (Eq. 2) of the selected rows only.  q[r], out[r]: device,
 * [L][sel_capacity][Hq][d] in kv_dtype; row i belongs to position sel[i] and
 * attends keys 0..sel[i] of kv_buf; query head hq reads KV head hq/(Hq/Hkv).
 * Rows >= *n_sel are left untouched.  softmax in float32.  q[r] must be
 * 16-byte aligned, out[r] 32-byte aligned (KVB_ERR_BAD_TABLE otherwise).
 * reqs[r].fresh is not read and may be NULL. */
int kvb_selective_attn(kvb_ctx* ctx, const kvb_request* reqs, int n_req, const kvb_selection* sel,
                       const void* const* q, void* const* out, float softmax_scale, void* cuda_stream);

/* CacheBlendRecompute (Algorithm 2) step 4, which is also the splice of
 * SelectiveRecompute (Algorithm 1): for every request and every i < *n_sel,
 * the K and V rows of position sel[i] in every layer of kv_buf are replaced
 * by the rows of `fresh` (K~, V~).  sel: host array of n_req kvb_selection
 * (only sel, n_sel, sel_capacity are read).  Other rows are not touched; an
 * entry of sel outside [0, T) is skipped. */
int kvb_patch(kvb_ctx* ctx, const kvb_request* reqs, int n_req, const kvb_selection* sel, void* cuda_stream);

/* Importance score of the cache manager's eviction policy (KV Cache Manager,
 * Eq. 7): importance[r][c] = 1/(L*H*C) * sum over layers, KV heads and the C
 * tokens of chunk c of ||k||_2, read from the stitched kv_buf (a rotation
 * leaves the norms unchanged).  importance: host array of n_req device
 * pointers, each to n_chunks float32 values.  reqs[r].fresh is not read and
 * may be NULL.  For callers that only hold a stitched buffer: a stitching call
 * delivers the same scores without this second read of the keys when
 * kvb_request.importance is set. */
int kvb_chunk_importance(kvb_ctx* ctx, const kvb_request* reqs, int n_req, float* const* importance,
                         void* cuda_stream);

/* KV Quantization, Eq. 6 (cache-population side), for one chunk: x [L][C][H][d]
 * in kv_dtype (device) -> codes and (scale, min) metadata in the layouts above.
 * is_value = 0: keys, per channel; 1: values, per token.  bits: 4 or 8. */
int kvb_quantize_chunk(kvb_ctx* ctx, const void* x, int is_value, int bits, void* codes, void* meta,
                       void* cuda_stream);

/* Position-free cache population for keys: x [L][C][H][d] are the keys of a
 * chunk encoded at positions orig_pos .. orig_pos+C-1.  Every key is rotated
 * back by R_theta^(-orig_pos) (Rotary Positional Embeddings, Eq. 3 -- the
 * inverse of the correction a key "cached at one position and reused at
 * another" needs) and then quantised as in kvb_quantize_chunk (Eq. 6, per
 * channel).  The stored chunk is the one a prompt starting at position 0 would
 * produce: list it in a chunk table with orig_pos = 0 and kvb_assemble applies
 * the single rotation by new_pos.  The rotation runs in float32 in a fixed
 * order (u = fma(x, cos, +-(x_partner * sin)), cos and sin from a double
 * angle), which is what makes the codes reproducible bit for bit.
 * orig_pos in [0, 2^24); bits: 4 or 8; buffers device, 16-byte aligned. */
int kvb_quantize_keys_at(kvb_ctx* ctx, const void* x, int orig_pos, int bits, void* codes, void* meta,
                         void* cuda_stream);

/* The general form of the two calls above.  unrotate_from < 0: no rotation
 * (kvb_quantize_chunk); >= 0: keys only, rotated back from that position
 * (kvb_quantize_keys_at).  meta_fp16 = 1 writes compact metadata: per group,
 * min is rounded down and scale = (max - min_rounded)/(2^b - 1) is rounded up
 * to binary16 (so every value still falls inside the code range), and the
 * codes are rint((x - min16)/scale16) in float32 against those rounded values;
 * the chunk's statistics must lie in binary16's finite range (|x| < 65504,
 * scale >= 2^-24).  List such a chunk with kvb_chunk.meta_fp16 = 1. */
int kvb_quantize_chunk_ex(kvb_ctx* ctx, const void* x, int is_value, int bits, int unrotate_from, int meta_fp16,
                          void* codes, void* meta, void* cuda_stream);

/* One chunk of a batched quantisation (host memory; all pointers device, 16-byte
 * aligned).  k / v: the chunk's keys / values [L][C][H][d] in kv_dtype, NULL for
 * a side that is not wanted; the outputs of a wanted side are required. */
typedef struct {
  const void* k;
  const void* v;
  void* k_codes;
  void* v_codes;
  void* k_meta;
  void* v_meta;
  int32_t bits;          /* 4 or 8 */
  int32_t unrotate_from; /* < 0: keys as they are; >= 0: keys rotated back from that position first */
  int32_t meta_fp16;     /* 1: compact (binary16) metadata */
  int32_t reserved;
} kvb_quantize_job;

/* KV Quantization, Eq. 6, for a batch of chunks in one launch (cache population
 * after a prefill: the Inference Engine's warm step stores every chunk of the
 * prompt).  Each job is kvb_quantize_chunk_ex for the keys and / or the values of
 * one chunk, with the same bit-exact code decision.  A context takes at least
 * max_chunks_total jobs per call (KVB_ERR_WORKSPACE beyond its descriptor arena). */
int kvb_quantize_chunks(kvb_ctx* ctx, const kvb_quantize_job* jobs, int n_jobs, void* cuda_stream);

/* Cosine deviation of ONE request for callers that cannot allocate GPU memory:
 * a server that gave the whole GPU to its own block pool at start-up, or a
 * latency-critical thread that may not take the device-wide synchronisation an
 * allocation implies.  (The paper has no counterpart; the arithmetic is that of
 * kvb_deviation_topk's deviation step, Algorithm 2 step 2.)  Needs no context
 * and calls no cudaMalloc / cudaFree: its scratch (fixed-point sums and one
 * descriptor) is a static device array of 128 KiB + 256 bytes that every GPU
 * loading this library holds until the process exits.
 *   kv_buf, fresh  device, [L][2][T][H][d] in model->kv_dtype, 16-byte aligned
 *   delta          device, [T] float32, written
 *   T              1 .. 16384; larger returns KVB_ERR_WORKSPACE (use a context)
 *   which          bit 0 keys, bit 1 values
 *   model          L <= 65535 (KVB_ERR_UNSUPPORTED beyond), d = 128
 * Asynchronous on cuda_stream.  The call makes `device` current while it
 * launches and restores the caller's current device before it returns.  The
 * first call on a device resolves the array's device address
 * (cudaGetSymbolAddress) and should come before any stream capture; first
 * calls from several host threads at once are safe.  All calls share the one array, which keeps the previous call's
 * contents (this call clears what it sums into): two calls whose GPU work
 * overlaps, e.g. on different streams, race on it. */
int kvb_deviation_static(int device, const kvb_model_desc* model, const void* kv_buf, const void* fresh, int T,
                         int which, float* delta, void* cuda_stream);

/* Host-only: runs the table checks the data-path calls run before launching
 * (chunks in prompt order tiling [0,T), enums, positions, pointer alignment,
 * the limits) without touching a GPU.  need_payload != 0 also requires the
 * code / metadata pointers, as kvb_assemble does.  err (optional) receives
 * the message.  No counterpart in the paper: it is the guard that keeps a bad
 * table from ever reaching a kernel. */
int kvb_validate(const kvb_model_desc* model, const kvb_limits* limits, const kvb_request* reqs, int n_req,
                 int need_payload, char* err, size_t err_len);

/* floor(ratio * T), the k of Algorithm 2 step 3. */
int kvb_select_count(int T, double ratio);

/* Synchronises the context's last stream and reports the device status word:
 * KVB_OK if no kernel flagged anything since the last report, else
 * KVB_ERR_DEVICE_STATUS with the bits in kvb_last_error's text (0x1 a bounded
 * wait ran out, 0x2 a descriptor failed a device-side check, 0x4 a selection
 * did not fit sel_capacity and was cut to its first sel_capacity entries).
 * Reporting clears the word, so the context stays usable. */
int kvb_last_status(kvb_ctx* ctx);
/* Text of the last host-side error of this context (valid until the next call). */
const char* kvb_last_error(kvb_ctx* ctx);
const char* kvb_status_string(int status);
/* Number of kernels this context has launched so far. */
int64_t kvb_launch_count(kvb_ctx* ctx);

/* Test hook (the paper has no counterpart): switches one of the context's
 * cross-check paths on (1) or off (0) for its later calls.  Keys:
 *   "dependent_launch"            default 1; 0 launches the kernel chain without
 *                                 programmatic dependent launch
 *   "descriptor_copy"             default 0; 1 sends every descriptor table through
 *                                 the pinned staging ring and cudaMemcpyAsync
 *   "attention_one_tile_per_cta"  default 0; 1 runs kvb_selective_attn with one tile
 *                                 per CTA instead of persistent CTAs
 *   "attention_cta_pairs"         default 0; 1 runs kvb_selective_attn on pairs of CTAs
 *                                 (two neighbouring tiles on two SMs per MMA, keys by
 *                                 sub-blocks of 128): measured slower than the default
 *                                 form, kept as a cross-check; same result to the
 *                                 attention tolerance, not bit for bit
 *   "attention_two_tiles"         default 0; 1 runs kvb_selective_attn with two
 *                                 neighbouring tiles per CTA that share every K/V
 *                                 sub-block in shared memory, one CTA per SM; same
 *                                 result to the attention tolerance
 * The first three settings compute the same bits; the tests compare them.
 * Unknown key or value: KVB_ERR_INVALID_ARG. */
int kvb_set_debug_option(kvb_ctx* ctx, const char* key, int value);

/* Self-test of the error path of a stuck barrier wait: launches one warp that
 * waits, with the attention kernel's own bounded wait, on a barrier that
 * nothing ever completes.  After limit_ms (1..1000) the wait gives up, the
 * kernel returns and sets status bit 0x1; the next kvb_last_status reports
 * KVB_ERR_DEVICE_STATUS and the context stays usable.  Asynchronous on the
 * stream like the data-path calls. */
int kvb_selftest_wait_timeout(kvb_ctx* ctx, int limit_ms, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* KVB_H_ */
