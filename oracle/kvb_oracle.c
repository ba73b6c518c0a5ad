/*
 * kvb_oracle.c -- plain, slow CPU statement of the KV-chunk stitching path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA library is
 * compared against; it is never part of the product path and shares no code,
 * header, table or helper with it.  Everything is written out in the order and
 * notation of the paper, in double precision, with no blocking or fusion.  The
 * only parallelism is an OpenMP loop over independent (layer, chunk) or
 * (layer, row) items, which changes no arithmetic.
 *
 * What is computed, and the passage each part follows:
 *   kvo_quantize_k / kvo_quantize_v   KV Quantization, Eq. 6 (per-channel keys,
 *                                     per-token values), test-data side
 *   kvo_dequant_k / kvo_dequant_v     inverse of Eq. 6:  x^ = q*s + min
 *   kvo_rope_rotate                   Rotary Positional Embeddings, Eq. 3: the
 *                                     correction R_theta^{delta} that a key cached
 *                                     at one position needs at another
 *   kvo_unrotate_keys_f32             the same rotation by -orig_pos ahead of Eq. 6
 *                                     (position-free cache population), in float32
 *   kvo_assemble                      Prompt Assembly (CHUNK_REUSE): cached chunks
 *                                     concatenated in prompt order into the
 *                                     [L,2,T,H,d] KV tensor of the Background section
 *   kvo_deviation                     Algorithm 2 step 2 (cosine deviation delta_t)
 *   kvo_topk                          Algorithm 2 step 3 (top floor(rho*T))
 *   kvo_seam_select                   Algorithm 1 window [max(0,p-R), p) per seam,
 *                                     united with the top-k set
 *   kvo_attention                     Eq. 2 (causal softmax attention) for the
 *                                     selected query rows, GQA head mapping
 *   kvo_patch                         Algorithm 2 step 4 / Algorithm 1 splice
 *   kvo_importance                    Eq. 7 (mean key norm of a chunk)
 *
 * Pins (tests/test_oracle_*.py): every function above is pinned to closed
 * forms, invariants, brute force or a library routine; the three format
 * choices that the paper leaves open (packed byte layout, seam definition,
 * K+V averaging) are design readings -- "parity unpinned" against the authors'
 * own code, which is not available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define KVO_MODE_FRESH 0
#define KVO_MODE_FP16 1 /* cached, unquantised, in the buffer's 16-bit dtype */
#define KVO_MODE_INT8 2
#define KVO_MODE_INT4 3

#define KVO_DT_F16 0
#define KVO_DT_BF16 1

/* ------------------------------------------------------------------ */
/* 16-bit storage formats: decode to double, round double to nearest-even */
/* ------------------------------------------------------------------ */

/* Round x to a binary format with p significand bits (hidden bit included),
 * minimum normal exponent emin and largest finite value maxfinite.
 * Round-to-nearest, ties-to-even, done once from the double (no intermediate
 * float rounding). */
static double round_to_format(double x, int p, int emin, double maxfinite) {
  if (x == 0.0 || isnan(x) || isinf(x)) return x;
  int e;
  (void)frexp(fabs(x), &e); /* |x| = m * 2^e, m in [0.5,1)  =>  exponent of 1.f form is e-1 */
  int ex = e - 1;
  if (ex < emin) ex = emin; /* subnormal range: fixed quantum */
  double quantum = ldexp(1.0, ex - (p - 1));
  double r = nearbyint(fabs(x) / quantum) * quantum; /* default rounding mode = ties-to-even */
  if (r > maxfinite) r = INFINITY;
  return copysign(r, x);
}

double kvo_bf16_to_f64(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

uint16_t kvo_f64_to_bf16(double x) {
  if (isnan(x)) return 0x7FC0;
  double r = round_to_format(x, 8, -126, 3.3895313892515355e38);
  float f = (float)r; /* exact: r is representable */
  uint32_t u;
  memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}

double kvo_f16_to_f64(uint16_t h) {
  int s = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
  double v;
  if (e == 0)
    v = ldexp((double)m, -24);
  else if (e == 31)
    v = m ? NAN : INFINITY;
  else
    v = ldexp(1.0 + m / 1024.0, e - 15);
  return s ? -v : v;
}

uint16_t kvo_f64_to_f16(double x) {
  if (isnan(x)) return 0x7E00;
  double r = round_to_format(x, 11, -14, 65504.0);
  uint16_t s = signbit(r) ? 0x8000 : 0;
  double a = fabs(r);
  if (isinf(a)) return s | 0x7C00;
  if (a == 0.0) return s;
  int e;
  double m = frexp(a, &e); /* a = m*2^e, m in [0.5,1) */
  int ex = e - 1;
  if (ex < -14) { /* subnormal: a = k * 2^-24 */
    return s | (uint16_t)(a * 16777216.0);
  }
  int mant = (int)((m * 2.0 - 1.0) * 1024.0);
  return s | (uint16_t)((ex + 15) << 10) | (uint16_t)mant;
}

static double load16(const uint16_t* p, int dtype) {
  return dtype == KVO_DT_BF16 ? kvo_bf16_to_f64(*p) : kvo_f16_to_f64(*p);
}
static uint16_t store16(double x, int dtype) {
  return dtype == KVO_DT_BF16 ? kvo_f64_to_bf16(x) : kvo_f64_to_f16(x);
}

void kvo_round_array(const double* x, int64_t n, int dtype, uint16_t* out) {
  for (int64_t i = 0; i < n; i++) out[i] = store16(x[i], dtype);
}
void kvo_decode_array(const uint16_t* x, int64_t n, int dtype, double* out) {
  for (int64_t i = 0; i < n; i++) out[i] = load16(x + i, dtype);
}

/* ------------------------------------------------------------------ */
/* Eq. 6: asymmetric min/max quantisation, b in {4, 8}                 */
/* ------------------------------------------------------------------ */

/* One group of n values at stride `stride`.  scale = (max-min)/(2^b-1) and min
 * are STORED as float32, and the code is decided in float32 arithmetic
 * (subtract, divide, round-half-even, clamp) so that a float32 quantiser on
 * any IEEE machine takes the same decisions.  A group with max == min gets
 * scale 1 and all-zero codes, so it dequantises to min exactly. */
/* Largest binary16 value <= x (up = 0) or smallest one >= x (up = 1); x finite, inside binary16's range. */
static float f16_directed(float x, int up) {
  if (x == 0.0f) return x;
  int e;
  (void)frexp(fabs((double)x), &e);
  int ex = e - 1;
  if (ex < -14) ex = -14;
  double quantum = ldexp(1.0, ex - 10);
  double q = (double)x / quantum; /* exact: a power-of-two scaling */
  return (float)((up ? ceil(q) : floor(q)) * quantum);
}

/* meta16: compact metadata -- the minimum is rounded DOWN to binary16, the scale is taken against
 * the rounded minimum and rounded UP to binary16 (so that no value leaves the code range), and the
 * codes are decided against that rounded pair. */
static void quantize_group(const double* x, int n, int64_t stride, int bits, int meta16, uint8_t* q /* n codes */,
                           float* scale_out, float* min_out) {
  float mn = (float)x[0], mx = (float)x[0];
  for (int i = 1; i < n; i++) {
    float v = (float)x[i * stride];
    if (v < mn) mn = v;
    if (v > mx) mx = v;
  }
  float levels = (float)((1 << bits) - 1);
  if (meta16) mn = f16_directed(mn, 0);
  float s = (mx > mn) ? (mx - mn) / levels : 1.0f;
  if (meta16) s = f16_directed(s, 1);
  for (int i = 0; i < n; i++) {
    float v = (float)x[i * stride];
    float c = rintf((v - mn) / s);
    if (c < 0.0f) c = 0.0f;
    if (c > levels) c = levels;
    q[i] = (uint8_t)c;
  }
  *scale_out = s;
  *min_out = mn;
}

/* int4 packing: element 2i along the head dimension in the low nibble of byte
 * i, element 2i+1 in the high nibble. */
static void put_code(uint8_t* codes, int bits, int64_t elem, uint8_t q) {
  if (bits == 8) {
    codes[elem] = q;
  } else {
    uint8_t* b = codes + (elem >> 1);
    if (elem & 1)
      *b = (uint8_t)((*b & 0x0F) | (q << 4));
    else
      *b = (uint8_t)((*b & 0xF0) | (q & 0x0F));
  }
}
static int get_code(const uint8_t* codes, int bits, int64_t elem) {
  if (bits == 8) return codes[elem];
  uint8_t b = codes[elem >> 1];
  return (elem & 1) ? (b >> 4) : (b & 0x0F);
}

/* Keys, per channel: for each (head h, channel j) the statistics run over the
 * tokens of one group (group_tokens consecutive tokens of the chunk).
 *   x     [C][H][d] doubles (the cached, already-rotated keys of one layer)
 *   codes [C][H][d] u8, or [C][H][d/2] packed nibbles
 *   meta  [C/group_tokens][H][d][2] float32 (scale, min) */
void kvo_quantize_k_ex(const double* x, int C, int H, int d, int bits, int group_tokens, int meta16, uint8_t* codes,
                       float* meta) {
  int G = C / group_tokens;
  uint8_t* tmp = (uint8_t*)malloc((size_t)group_tokens);
  if (bits == 4) memset(codes, 0, (size_t)C * H * d / 2);
  for (int g = 0; g < G; g++)
    for (int h = 0; h < H; h++)
      for (int j = 0; j < d; j++) {
        const double* base = x + ((int64_t)(g * group_tokens) * H + h) * d + j;
        float* m = meta + (((int64_t)g * H + h) * d + j) * 2;
        quantize_group(base, group_tokens, (int64_t)H * d, bits, meta16, tmp, &m[0], &m[1]);
        for (int i = 0; i < group_tokens; i++)
          put_code(codes, bits, ((int64_t)(g * group_tokens + i) * H + h) * d + j, tmp[i]);
      }
  free(tmp);
}

/* Values, per token: for each (token t, head h) the statistics run over the
 * channels of one group (group_ch consecutive channels).
 *   meta [C][H][d/group_ch][2] float32 (scale, min) */
void kvo_quantize_v_ex(const double* x, int C, int H, int d, int bits, int group_ch, int meta16, uint8_t* codes,
                       float* meta) {
  int G = d / group_ch;
  uint8_t* tmp = (uint8_t*)malloc((size_t)group_ch);
  if (bits == 4) memset(codes, 0, (size_t)C * H * d / 2);
  for (int t = 0; t < C; t++)
    for (int h = 0; h < H; h++)
      for (int g = 0; g < G; g++) {
        int64_t e0 = ((int64_t)t * H + h) * d + g * group_ch;
        float* m = meta + (((int64_t)t * H + h) * G + g) * 2;
        quantize_group(x + e0, group_ch, 1, bits, meta16, tmp, &m[0], &m[1]);
        for (int i = 0; i < group_ch; i++) put_code(codes, bits, e0 + i, tmp[i]);
      }
  free(tmp);
}

void kvo_quantize_k(const double* x, int C, int H, int d, int bits, int group_tokens, uint8_t* codes, float* meta) {
  kvo_quantize_k_ex(x, C, H, d, bits, group_tokens, 0, codes, meta);
}
void kvo_quantize_v(const double* x, int C, int H, int d, int bits, int group_ch, uint8_t* codes, float* meta) {
  kvo_quantize_v_ex(x, C, H, d, bits, group_ch, 0, codes, meta);
}

/* Inverse of Eq. 6:  x^ = q * scale + min, in double. */
void kvo_dequant_k(const uint8_t* codes, const float* meta, int C, int H, int d, int bits,
                   int group_tokens, double* out) {
  for (int t = 0; t < C; t++)
    for (int h = 0; h < H; h++)
      for (int j = 0; j < d; j++) {
        int64_t e = ((int64_t)t * H + h) * d + j;
        const float* m = meta + (((int64_t)(t / group_tokens) * H + h) * d + j) * 2;
        out[e] = (double)get_code(codes, bits, e) * (double)m[0] + (double)m[1];
      }
}

void kvo_dequant_v(const uint8_t* codes, const float* meta, int C, int H, int d, int bits,
                   int group_ch, double* out) {
  int G = d / group_ch;
  for (int t = 0; t < C; t++)
    for (int h = 0; h < H; h++)
      for (int j = 0; j < d; j++) {
        int64_t e = ((int64_t)t * H + h) * d + j;
        const float* m = meta + (((int64_t)t * H + h) * G + j / group_ch) * 2;
        out[e] = (double)get_code(codes, bits, e) * (double)m[0] + (double)m[1];
      }
}

/* ------------------------------------------------------------------ */
/* Eq. 3: rotary embedding as a rotation by `delta` positions           */
/* ------------------------------------------------------------------ */

/* rows [n][H][d], rotated in place by R_theta^{delta}.  Channel j pairs with
 * j + d/2 (rotate-half pairing of the Qwen2 family), frequency
 * f_j = theta^(-2j/d), angle delta * f_j, all in double. */
void kvo_rope_rotate(double* rows, int64_t n, int H, int d, double theta, double delta) {
  int half = d / 2;
  for (int j = 0; j < half; j++) {
    double f = pow(theta, -2.0 * (double)j / (double)d);
    double a = delta * f;
    double c = cos(a), s = sin(a);
    for (int64_t t = 0; t < n; t++)
      for (int h = 0; h < H; h++) {
        double* v = rows + (t * H + h) * d;
        double lo = v[j], hi = v[j + half];
        v[j] = lo * c - hi * s;
        v[j + half] = hi * c + lo * s;
      }
  }
}

/* Position-free cache population: the keys of a chunk that was encoded at
 * positions orig_pos.. are rotated back by R_theta^{-orig_pos} before they are
 * quantised (Eq. 6), so the stored chunk is the one a prompt starting at
 * position 0 would produce and re-use at new_pos needs the single rotation
 * R_theta^{new_pos} (Rotary Positional Embeddings, Eq. 3).  The result feeds a
 * quantiser whose code decision is taken in float32, so this step is float32
 * too, with one fixed operation order (cos and sin evaluated in double and
 * rounded to float32; one rounded product, one fused multiply-add):
 *   u_lo = fma(x_lo, c, x_hi * s)      u_hi = fma(x_hi, c, -(x_lo * s))
 * rows: [n][H][d] 16-bit; out: [n][H][d] doubles holding float32 values. */
void kvo_unrotate_keys_f32(const uint16_t* rows, int64_t n, int H, int d, int dtype, double theta, int orig_pos,
                           double* out) {
  int half = d / 2;
  for (int j = 0; j < half; j++) {
    double f = pow(theta, -2.0 * (double)j / (double)d);
    double a = (double)orig_pos * f;
    float c = (float)cos(a), s = (float)sin(a);
    for (int64_t t = 0; t < n; t++)
      for (int h = 0; h < H; h++) {
        int64_t base = (t * H + h) * d;
        float lo = (float)load16(rows + base + j, dtype), hi = (float)load16(rows + base + j + half, dtype);
        float p_hi = hi * s, p_lo = lo * s;
        out[base + j] = (double)fmaf(lo, c, p_hi);
        out[base + j + half] = (double)fmaf(hi, c, -p_lo);
      }
  }
}

/* ------------------------------------------------------------------ */
/* Prompt assembly                                                      */
/* ------------------------------------------------------------------ */

typedef struct {
  int32_t orig_pos, new_pos, n_tokens, mode;
  const void* k_codes; /* [L][C][H][d] u8 | [L][C][H][d/2] nibbles | [L][C][H][d] 16-bit */
  const void* v_codes;
  const float* k_meta; /* [L][G_k][H][d][2], G_k = 1 (int8) or C/int4_group (int4) */
  const float* v_meta; /* [L][C][H][G_v][2], G_v = 1 (int8) or d/int4_group (int4) */
} kvo_chunk;

/* kv_buf and fresh: [L][2][T][H][d] 16-bit.  exact (optional, may be NULL):
 * same shape in double, the un-rounded values (used to state tolerances
 * against the true result rather than against one rounding of it).
 * Steps per cached chunk and layer, in the paper's order: dequantise
 * (KV Quantization), rotate keys by new_pos - orig_pos (Rotary Positional
 * Embeddings), write at rows new_pos.. (Prompt Assembly).  Values are never
 * rotated.  FRESH chunks copy the caller's fresh rows bit for bit. */
void kvo_assemble(const kvo_chunk* chunks, int n_chunks, int L, int H, int d, int T, double theta,
                  int dtype, int int4_group, const uint16_t* fresh, uint16_t* kv_buf, double* exact) {
  int64_t plane = (int64_t)T * H * d;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int l = 0; l < L; l++)
    for (int c = 0; c < n_chunks; c++) {
      const kvo_chunk* ck = &chunks[c];
      int C = ck->n_tokens;
      int64_t n = (int64_t)C * H * d;
      uint16_t* kout = kv_buf + ((int64_t)l * 2 + 0) * plane + (int64_t)ck->new_pos * H * d;
      uint16_t* vout = kv_buf + ((int64_t)l * 2 + 1) * plane + (int64_t)ck->new_pos * H * d;
      double* kex = exact ? exact + (kout - kv_buf) : NULL;
      double* vex = exact ? exact + (vout - kv_buf) : NULL;
      if (ck->mode == KVO_MODE_FRESH) {
        const uint16_t* kin = fresh + (kout - kv_buf);
        const uint16_t* vin = fresh + (vout - kv_buf);
        memcpy(kout, kin, (size_t)n * 2);
        memcpy(vout, vin, (size_t)n * 2);
        if (exact) {
          kvo_decode_array(kin, n, dtype, kex);
          kvo_decode_array(vin, n, dtype, vex);
        }
        continue;
      }
      double* k = (double*)malloc((size_t)n * sizeof(double));
      double* v = (double*)malloc((size_t)n * sizeof(double));
      if (ck->mode == KVO_MODE_FP16) {
        kvo_decode_array((const uint16_t*)ck->k_codes + (int64_t)l * n, n, dtype, k);
        kvo_decode_array((const uint16_t*)ck->v_codes + (int64_t)l * n, n, dtype, v);
      } else {
        int bits = ck->mode == KVO_MODE_INT8 ? 8 : 4;
        int gk = bits == 8 ? C : int4_group; /* tokens per key group */
        int gv = bits == 8 ? d : int4_group; /* channels per value group */
        int64_t code_bytes = n * bits / 8;
        const uint8_t* kc = (const uint8_t*)ck->k_codes + (int64_t)l * code_bytes;
        const uint8_t* vc = (const uint8_t*)ck->v_codes + (int64_t)l * code_bytes;
        const float* km = ck->k_meta + (int64_t)l * (C / gk) * H * d * 2;
        const float* vm = ck->v_meta + (int64_t)l * C * H * (d / gv) * 2;
        kvo_dequant_k(kc, km, C, H, d, bits, gk, k);
        kvo_dequant_v(vc, vm, C, H, d, bits, gv, v);
      }
      kvo_rope_rotate(k, C, H, d, theta, (double)(ck->new_pos - ck->orig_pos));
      kvo_round_array(k, n, dtype, kout);
      kvo_round_array(v, n, dtype, vout);
      if (exact) {
        memcpy(kex, k, (size_t)n * sizeof(double));
        memcpy(vex, v, (size_t)n * sizeof(double));
      }
      free(k);
      free(v);
    }
}

/* ------------------------------------------------------------------ */
/* Algorithm 2, step 2: per-token cosine deviation                      */
/* ------------------------------------------------------------------ */

/* cos(a, b) over d elements, with the two degenerate cases fixed:
 * a == b element-wise -> 1 (also for zero vectors); otherwise a zero norm -> 0. */
static double cosine(const uint16_t* a, const uint16_t* b, int d, int dtype) {
  double ab = 0, aa = 0, bb = 0;
  int same = 1;
  for (int j = 0; j < d; j++) {
    double x = load16(a + j, dtype), y = load16(b + j, dtype);
    ab += x * y;
    aa += x * x;
    bb += y * y;
    if (x != y) same = 0;
  }
  if (same) return 1.0;
  if (aa == 0.0 || bb == 0.0) return 0.0;
  return ab / (sqrt(aa) * sqrt(bb));
}

/* delta_t = 1 - mean over (layer, head[, K and V]) of cos(stored, fresh).
 * which: bit 0 = keys (the printed formula), bit 1 = values; both bits set
 * averages over 2*L*H cosines.  delta64 (may be NULL) gets the double,
 * delta32 the float32 rounding that the selection step orders by. */
void kvo_deviation(const uint16_t* kv_buf, const uint16_t* fresh, int L, int H, int d, int T, int dtype,
                   int which, double* delta64, float* delta32) {
  int64_t plane = (int64_t)T * H * d;
  int nw = ((which & 1) ? 1 : 0) + ((which & 2) ? 1 : 0);
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; t++) {
    double sum = 0;
    for (int l = 0; l < L; l++)
      for (int kv = 0; kv < 2; kv++) {
        if (!((which >> kv) & 1)) continue;
        for (int h = 0; h < H; h++) {
          int64_t off = ((int64_t)l * 2 + kv) * plane + ((int64_t)t * H + h) * d;
          sum += cosine(kv_buf + off, fresh + off, d, dtype);
        }
      }
    double dl = 1.0 - sum / ((double)L * H * nw);
    if (delta64) delta64[t] = dl;
    delta32[t] = (float)dl;
  }
}

/* ------------------------------------------------------------------ */
/* Algorithm 2, step 3, and Algorithm 1's windows                       */
/* ------------------------------------------------------------------ */

int kvo_select_count(int T, double ratio) { return (int)floor(ratio * (double)T); }

typedef struct {
  float v;
  int32_t i;
} kvo_item;

/* larger delta first; equal deltas: lower index first.  NaN ranks as +inf,
 * -0 as +0, so the order is total. */
static int item_cmp(const void* pa, const void* pb) {
  const kvo_item* a = (const kvo_item*)pa;
  const kvo_item* b = (const kvo_item*)pb;
  if (a->v > b->v) return -1;
  if (a->v < b->v) return 1;
  return (a->i > b->i) - (a->i < b->i);
}

/* rank[0..k): indices of the k largest delta, most deviated first. */
void kvo_topk(const float* delta, int T, int k, int32_t* rank) {
  kvo_item* it = (kvo_item*)malloc((size_t)(T > 0 ? T : 1) * sizeof(kvo_item));
  for (int t = 0; t < T; t++) {
    float v = delta[t];
    if (isnan(v)) v = INFINITY;
    if (v == 0.0f) v = 0.0f; /* folds -0 into +0 */
    it[t].v = v;
    it[t].i = t;
  }
  qsort(it, (size_t)T, sizeof(kvo_item), item_cmp);
  for (int i = 0; i < k && i < T; i++) rank[i] = it[i].i;
  free(it);
}

/* A seam is an interior chunk boundary p = new_pos of chunk i >= 1 (chunks in
 * prompt order) where chunk i or chunk i-1 is cached (not FRESH).  Its window
 * is [max(0, p-before), min(T, p+after)); Algorithm 1 is (before, after) =
 * (R, 0).  The first `sinks` positions (attention-sink tokens of the Tokenization
 * and Chunking section) are always taken.  sel = ascending, duplicate-free
 * union of rank[0..k), all windows and the sinks; returns n_sel.  sel must hold
 * T entries. */
int kvo_seam_select(const int32_t* rank, int k, const int32_t* chunk_new_pos, const int32_t* chunk_mode,
                    int n_chunks, int T, int before, int after, int sinks, int32_t* sel) {
  uint8_t* mark = (uint8_t*)calloc((size_t)(T > 0 ? T : 1), 1);
  for (int i = 0; i < k; i++) mark[rank[i]] = 1;
  for (int t = 0; t < sinks && t < T; t++) mark[t] = 1;
  for (int c = 1; c < n_chunks; c++) {
    if (chunk_mode[c] == KVO_MODE_FRESH && chunk_mode[c - 1] == KVO_MODE_FRESH) continue;
    int p = chunk_new_pos[c];
    int lo = p - before < 0 ? 0 : p - before;
    int hi = p + after > T ? T : p + after;
    for (int t = lo; t < hi; t++) mark[t] = 1;
  }
  int n = 0;
  for (int t = 0; t < T; t++)
    if (mark[t]) sel[n++] = t;
  free(mark);
  return n;
}

/* ------------------------------------------------------------------ */
/* Eq. 2: causal attention of the selected query rows                   */
/* ------------------------------------------------------------------ */

/* q, out: [L][cap][Hq][d] 16-bit, row i belongs to position sel[i], i < n_sel.
 * kv_buf: [L][2][T][Hkv][d].  Query head hq reads KV head hq / (Hq/Hkv).
 * Keys 0..sel[i] inclusive.  layers[0..n_layers) picks which layers to do and
 * rows[0..n_rows) which selected rows (NULL = all), so that a bounded sample
 * can be computed exactly.  out_exact (may be NULL): un-rounded doubles. */
void kvo_attention(const uint16_t* q, const uint16_t* kv_buf, const int32_t* sel, int n_sel, int cap,
                   int L, int Hq, int Hkv, int d, int T, int dtype, double scale, const int32_t* layers,
                   int n_layers, const int32_t* rows, int n_rows, uint16_t* out, double* out_exact) {
  int64_t plane = (int64_t)T * Hkv * d;
  int rep = Hq / Hkv;
  int nr = rows ? n_rows : n_sel;
  (void)L;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int li = 0; li < n_layers; li++)
    for (int ri = 0; ri < nr; ri++) {
      int l = layers[li];
      int i = rows ? rows[ri] : ri;
      int t = sel[i];
      double* p = (double*)malloc((size_t)(t + 1) * sizeof(double));
      double* acc = (double*)malloc((size_t)d * sizeof(double));
      for (int hq = 0; hq < Hq; hq++) {
        int hk = hq / rep;
        const uint16_t* qv = q + (((int64_t)l * cap + i) * Hq + hq) * d;
        const uint16_t* K = kv_buf + ((int64_t)l * 2 + 0) * plane + (int64_t)hk * d;
        const uint16_t* V = kv_buf + ((int64_t)l * 2 + 1) * plane + (int64_t)hk * d;
        double mx = -INFINITY;
        for (int s = 0; s <= t; s++) {
          double dot = 0;
          for (int j = 0; j < d; j++)
            dot += load16(qv + j, dtype) * load16(K + (int64_t)s * Hkv * d + j, dtype);
          p[s] = dot * scale;
          if (p[s] > mx) mx = p[s];
        }
        double den = 0;
        for (int s = 0; s <= t; s++) {
          p[s] = exp(p[s] - mx);
          den += p[s];
        }
        for (int j = 0; j < d; j++) acc[j] = 0;
        for (int s = 0; s <= t; s++) {
          double w = p[s] / den;
          for (int j = 0; j < d; j++) acc[j] += w * load16(V + (int64_t)s * Hkv * d + j, dtype);
        }
        int64_t o = (((int64_t)l * cap + i) * Hq + hq) * d;
        for (int j = 0; j < d; j++) {
          out[o + j] = store16(acc[j], dtype);
          if (out_exact) out_exact[o + j] = acc[j];
        }
      }
      free(p);
      free(acc);
    }
}

int kvo_max_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Number of threads the parallel loops may use from now on (timing on one core vs all cores). */
void kvo_set_threads(int n) {
#ifdef _OPENMP
  extern void omp_set_num_threads(int);
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* ------------------------------------------------------------------ */
/* Algorithm 2, step 4 (and Algorithm 1's splice): patch                */
/* ------------------------------------------------------------------ */

/* Replaces the K and V rows of every selected position, in every layer, by the
 * freshly projected ones:  KV[l, :, sel[i], :, :] <- fresh[l, :, sel[i], :, :]. */
void kvo_patch(uint16_t* kv_buf, const uint16_t* fresh, const int32_t* sel, int n_sel, int L, int T, int H, int d) {
  int64_t row = (int64_t)H * d;
  for (int l = 0; l < L; l++)
    for (int kv = 0; kv < 2; kv++)
      for (int i = 0; i < n_sel; i++) {
        int64_t off = (((int64_t)l * 2 + kv) * T + sel[i]) * row;
        memcpy(kv_buf + off, fresh + off, (size_t)row * 2);
      }
}

/* ------------------------------------------------------------------ */
/* Eq. 7: importance of a chunk = mean L2 norm of its keys              */
/* ------------------------------------------------------------------ */

/* importance[c] = 1/(L*H*C) * sum over layers, heads and the chunk's C tokens of ||k||_2,
 * for the chunks [c*C, (c+1)*C) of a [L][2][T][H][d] buffer. */
void kvo_importance(const uint16_t* kv_buf, int L, int T, int H, int d, int C, int dtype, double* importance) {
  int n_chunks = T / C;
  for (int c = 0; c < n_chunks; c++) {
    double sum = 0;
    for (int l = 0; l < L; l++)
      for (int t = c * C; t < (c + 1) * C; t++)
        for (int h = 0; h < H; h++) {
          const uint16_t* k = kv_buf + ((((int64_t)l * 2 + 0) * T + t) * H + h) * d;
          double n2 = 0;
          for (int j = 0; j < d; j++) {
            double x = load16(k + j, dtype);
            n2 += x * x;
          }
          sum += sqrt(n2);
        }
    importance[c] = sum / ((double)L * H * C);
  }
}
