/*
 * puzzle_oracle.c -- TEST INFRASTRUCTURE, not part of the product path.
 *
 * A plain, slow, float64 CPU statement of what the decode-step attention path
 * computes, written from the paper's problem statement:
 *
 *   - KV cache held as FP8 (Section "KV Quantization"): E4M3 codes with
 *     max-calibrated scales, optionally rounded up to a power of two.
 *   - Every layer is either full-context or window attention; a window layer
 *     lets the current token see only the most recent W tokens (Section
 *     "Window attention for long-context inference").
 *   - Decode is KV-cache-I/O bound (Section "Optimized Scenarios"), which is why
 *     the product streams the cache; the oracle just walks it.
 *
 * Nothing here is blocked, fused, vectorised or reordered: each function is the
 * textbook definition written out, in double precision, so that it can be
 * checked against the paper by eye.  The only tests, the smoke check and the
 * bench's cpu_baseline leg may call this file.  It shares no code, header,
 * table or constant with the CUDA library.
 *
 * Parity pins (tests marked "not gpu"): the E4M3 codec is pinned by closed-form
 * code values, exhaustive round trip and brute-force nearest search; append by
 * power-of-two-scale closed forms; attention by window>=context == full,
 * sink=-inf == no sink == library softmax attention, identical-key closed form,
 * single-token closed form, permutation invariance and an independent
 * pure-Python triple loop; merge by partition invariance.  Model-level accuracy
 * effects of FP8/scales/window (the paper's accuracy tables) are parity
 * unpinned: they need the trained weights and are outside this path.
 *
 * Layouts (all host memory, caller owned):
 *   cache   [num_blocks][Hkv][block_size][D]   u8 E4M3 codes, or u16 bf16 bits
 *   q       [batch][Hq][D]                     u16 bf16 bits
 *   k_new   [batch][Hkv][D]                    u16 bf16 bits
 *   table   [batch][max_blocks_per_seq] i32, or NULL: block = b*max_blocks+i
 *   seq_lens[batch] i32, length AFTER this step's append
 *   scales  [Hkv] f32 dequantisation scales (x ~= code_value*scale), NULL = 1
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_KV_FP8_E4M3 0
#define ORACLE_KV_BF16 1

/* ---------------------------------------------------------------- bf16 --- */

/* bf16 is the top 16 bits of an IEEE float32, so widening is exact. */
static float bf16_bits_to_float(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

/* ------------------------------------------------------- E4M3 (FP8 KV) --- */

/* Value of one E4M3 code: 1 sign, 4 exponent (bias 7), 3 mantissa bits; the
 * all-ones exponent is an ordinary binade except mantissa 111, which is NaN
 * (no infinities), so the largest finite magnitude is 1.75*2^8 = 448. */
double oracle_e4m3_decode(uint8_t code) {
  int s = code >> 7;
  int e = (code >> 3) & 15;
  int m = code & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0)
    v = ldexp((double)m / 8.0, -6); /* subnormal: 2^-6 * m/8 */
  else
    v = ldexp(1.0 + (double)m / 8.0, e - 7);
  return s ? -v : v;
}

/* Nearest E4M3 code to y: round to nearest, ties to the code whose mantissa
 * LSB is 0, magnitudes above the largest finite value saturate to it, the sign
 * of zero is kept.  Every NaN maps to the one canonical NaN code 0x7F: the
 * sign a NaN carries out of a division is not fixed by IEEE 754 (it differs
 * between processors), so it cannot be part of a bit-exact contract.
 * Done as a search over the codebook. */
uint8_t oracle_e4m3_encode(float y) {
  uint8_t sign = signbit(y) ? 0x80 : 0x00;
  double a = fabs((double)y);
  int lo;
  if (isnan(y)) return (uint8_t)0x7F;
  if (a >= oracle_e4m3_decode(0x7E)) return (uint8_t)(sign | 0x7E);
  /* magnitudes of codes 0x00..0x7E increase strictly with the code */
  lo = 0;
  while (oracle_e4m3_decode((uint8_t)(lo + 1)) <= a) lo++;
  {
    double below = a - oracle_e4m3_decode((uint8_t)lo);
    double above = oracle_e4m3_decode((uint8_t)(lo + 1)) - a;
    int pick;
    if (below < above)
      pick = lo;
    else if (above < below)
      pick = lo + 1;
    else
      pick = (lo & 1) ? lo + 1 : lo; /* tie: even mantissa bit */
    return (uint8_t)(sign | pick);
  }
}

/* Element-wise encode of n floats (a loop over the function above). */
void oracle_e4m3_encode_array(const float* y, int64_t n, uint8_t* codes) {
  for (int64_t i = 0; i < n; i++) codes[i] = oracle_e4m3_encode(y[i]);
}

/* ------------------------------------------------------- calibration ----- */

/* Max calibration (Section "KV Quantization"): scale[h] = amax_h / 448 in
 * float32, amax over every token and channel of KV head h.  pow2 != 0 rounds
 * each scale up to the next power of two, as the paper does.  amax == 0 gives
 * scale 1.   x: float32 [n_tokens][Hkv][D]. */
void oracle_calibrate_scales(const float* x, int64_t n_tokens, int Hkv, int D, int pow2,
                             float* scale_out) {
  for (int h = 0; h < Hkv; h++) {
    float amax = 0.0f;
    for (int64_t t = 0; t < n_tokens; t++)
      for (int d = 0; d < D; d++) {
        float a = fabsf(x[(t * Hkv + h) * D + d]);
        if (a > amax) amax = a;
      }
    if (amax == 0.0f) {
      scale_out[h] = 1.0f;
      continue;
    }
    {
      float s = amax / 448.0f;
      if (pow2) {
        int e;
        float fr = frexpf(s, &e); /* s = fr * 2^e, fr in [0.5, 1) */
        s = (fr == 0.5f) ? s : ldexpf(1.0f, e);
      }
      scale_out[h] = s;
    }
  }
}

/* ------------------------------------------------------- paging ---------- */

static int64_t physical_block(const int32_t* table, int max_blocks_per_seq, int b, int64_t i) {
  if (table == NULL) return (int64_t)b * max_blocks_per_seq + i;
  return table[(int64_t)b * max_blocks_per_seq + i];
}

static int64_t cache_index(int64_t block, int Hkv, int block_size, int D, int h, int slot, int d) {
  return ((block * Hkv + h) * block_size + slot) * (int64_t)D + d;
}

/* ------------------------------------------------------- append ---------- */

/* Quantise-and-append of one new token per sequence.  For FP8: the float32
 * quotient x/scale (the double quotient rounded once to float equals the
 * correctly rounded float quotient, since 53 >= 2*24+2), then the E4M3 encode
 * above.  For bf16 KV: the bits are stored as they are.  The token goes to
 * logical position seq_len-1. Sequences with seq_len <= 0 append nothing. */
void oracle_kv_append(void* k_cache, void* v_cache, int kv_dtype, int Hkv, int D, int block_size,
                      const int32_t* table, int max_blocks_per_seq, const int32_t* seq_lens,
                      const float* k_scale, const float* v_scale, const uint16_t* k_new,
                      const uint16_t* v_new, int batch) {
  for (int b = 0; b < batch; b++) {
    int64_t pos = (int64_t)seq_lens[b] - 1;
    if (pos < 0) continue;
    {
      int64_t block = physical_block(table, max_blocks_per_seq, b, pos / block_size);
      int slot = (int)(pos % block_size);
      for (int h = 0; h < Hkv; h++)
        for (int d = 0; d < D; d++) {
          int64_t src = ((int64_t)b * Hkv + h) * D + d;
          int64_t dst = cache_index(block, Hkv, block_size, D, h, slot, d);
          if (kv_dtype == ORACLE_KV_BF16) {
            ((uint16_t*)k_cache)[dst] = k_new[src];
            ((uint16_t*)v_cache)[dst] = v_new[src];
          } else {
            double ks = k_scale ? (double)k_scale[h] : 1.0;
            double vs = v_scale ? (double)v_scale[h] : 1.0;
            float yk = (float)((double)bf16_bits_to_float(k_new[src]) / ks);
            float yv = (float)((double)bf16_bits_to_float(v_new[src]) / vs);
            ((uint8_t*)k_cache)[dst] = oracle_e4m3_encode(yk);
            ((uint8_t*)v_cache)[dst] = oracle_e4m3_encode(yv);
          }
        }
    }
  }
}

/* ------------------------------------------------------- attention ------- */

typedef struct {
  const void* k_cache;
  const void* v_cache;
  int kv_dtype, Hq, Hkv, D, block_size;
  const int32_t* table;
  int max_blocks_per_seq;
  const int32_t* seq_lens;
  const float* k_scale;
  const float* v_scale;
  const uint16_t* q;
  const float* sinks;
  int window;
  double sm_scale;
  int use_range; /* 0: window rule; 1: keys [t0, t1) exactly, no sink */
  int64_t t0, t1;
  const int32_t* items; /* [n_items][2] = (b, query head) */
  int64_t n_items;
  double* out; /* [n_items][D] */
  double* lse; /* [n_items] */
  int64_t next; /* shared work counter */
  pthread_mutex_t lock;
} attn_job;

static double cache_value(const void* cache, int kv_dtype, int64_t idx, double scale) {
  if (kv_dtype == ORACLE_KV_BF16) return (double)bf16_bits_to_float(((const uint16_t*)cache)[idx]);
  return oracle_e4m3_decode(((const uint8_t*)cache)[idx]) * scale;
}

/* One (sequence, query head): softmax(q.k * sm_scale, with the sink logit as
 * one more column that carries no value) times V, over the visible keys. */
static void attend_one(const attn_job* J, int b, int g, double* out, double* lse_out) {
  int D = J->D;
  int h = g / (J->Hq / J->Hkv); /* grouped-query: consecutive query heads share a KV head */
  int64_t L = J->seq_lens[b];
  int64_t lo, hi;
  double ks = (J->k_scale && J->kv_dtype == ORACLE_KV_FP8_E4M3) ? (double)J->k_scale[h] : 1.0;
  double vs = (J->v_scale && J->kv_dtype == ORACLE_KV_FP8_E4M3) ? (double)J->v_scale[h] : 1.0;
  double sink = -INFINITY;
  double M, Z;
  double* s;
  if (L < 0) L = 0;
  if (J->use_range) {
    lo = J->t0 < 0 ? 0 : J->t0;
    hi = J->t1 > L ? L : J->t1;
  } else {
    /* window W: the most recent W tokens, the current one included */
    lo = (J->window > 0 && L > J->window) ? L - J->window : 0;
    hi = L;
    if (J->sinks) sink = (double)J->sinks[g];
  }
  if (hi < lo) hi = lo;
  s = (double*)malloc(sizeof(double) * (size_t)(hi - lo + 1));
  M = sink;
  for (int64_t j = lo; j < hi; j++) {
    int64_t block = physical_block(J->table, J->max_blocks_per_seq, b, j / J->block_size);
    int slot = (int)(j % J->block_size);
    double dot = 0.0;
    for (int d = 0; d < D; d++) {
      double qd = (double)bf16_bits_to_float(J->q[((int64_t)b * J->Hq + g) * D + d]);
      double kd = cache_value(J->k_cache, J->kv_dtype,
                              cache_index(block, J->Hkv, J->block_size, D, h, slot, d), ks);
      dot += qd * kd;
    }
    s[j - lo] = dot * J->sm_scale;
    if (s[j - lo] > M) M = s[j - lo];
  }
  for (int d = 0; d < D; d++) out[d] = 0.0;
  if (M == -INFINITY) { /* nothing visible and no sink */
    *lse_out = -INFINITY;
    free(s);
    return;
  }
  Z = (sink == -INFINITY) ? 0.0 : exp(sink - M);
  for (int64_t j = lo; j < hi; j++) {
    int64_t block = physical_block(J->table, J->max_blocks_per_seq, b, j / J->block_size);
    int slot = (int)(j % J->block_size);
    double p = exp(s[j - lo] - M);
    Z += p;
    for (int d = 0; d < D; d++)
      out[d] += p * cache_value(J->v_cache, J->kv_dtype,
                                cache_index(block, J->Hkv, J->block_size, D, h, slot, d), vs);
  }
  for (int d = 0; d < D; d++) out[d] /= Z;
  *lse_out = M + log(Z);
  free(s);
}

static void* attn_worker(void* arg) {
  attn_job* J = (attn_job*)arg;
  for (;;) {
    int64_t i;
    pthread_mutex_lock(&J->lock);
    i = J->next++;
    pthread_mutex_unlock(&J->lock);
    if (i >= J->n_items) break;
    attend_one(J, J->items[2 * i], J->items[2 * i + 1], J->out + i * J->D, J->lse + i);
  }
  return NULL;
}

static void run_job(attn_job* J, int threads) {
  pthread_t* tid;
  if (threads < 1) threads = 1;
  if (threads > 1024) threads = 1024;
  J->next = 0;
  pthread_mutex_init(&J->lock, NULL);
  tid = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)threads);
  for (int t = 1; t < threads; t++) pthread_create(&tid[t], NULL, attn_worker, J);
  attn_worker(J);
  for (int t = 1; t < threads; t++) pthread_join(tid[t], NULL);
  pthread_mutex_destroy(&J->lock);
  free(tid);
}

/* Decode-step attention for the listed (sequence, query head) items.
 * window == 0: full context; window == W > 0: keys [L - min(W, L), L).
 * sinks: [Hq] raw logits (not multiplied by sm_scale) or NULL (no sink).
 * An empty context gives out = 0 and lse = sink (or -inf without one). */
void oracle_decode_attn(const void* k_cache, const void* v_cache, int kv_dtype, int Hq, int Hkv,
                        int D, int block_size, const int32_t* table, int max_blocks_per_seq,
                        const int32_t* seq_lens, const float* k_scale, const float* v_scale,
                        const uint16_t* q, const float* sinks, int window, double sm_scale,
                        const int32_t* items, int64_t n_items, double* out, double* lse,
                        int threads) {
  attn_job J;
  memset(&J, 0, sizeof J);
  J.k_cache = k_cache; J.v_cache = v_cache; J.kv_dtype = kv_dtype;
  J.Hq = Hq; J.Hkv = Hkv; J.D = D; J.block_size = block_size;
  J.table = table; J.max_blocks_per_seq = max_blocks_per_seq; J.seq_lens = seq_lens;
  J.k_scale = k_scale; J.v_scale = v_scale; J.q = q; J.sinks = sinks;
  J.window = window; J.sm_scale = sm_scale; J.use_range = 0;
  J.items = items; J.n_items = n_items; J.out = out; J.lse = lse;
  run_job(&J, threads);
}

/* Attention restricted to keys [t0, t1) of every listed item, WITHOUT the
 * sink: the partial (o, lse) that a split of the context produces. */
void oracle_partial_attn(const void* k_cache, const void* v_cache, int kv_dtype, int Hq, int Hkv,
                         int D, int block_size, const int32_t* table, int max_blocks_per_seq,
                         const int32_t* seq_lens, const float* k_scale, const float* v_scale,
                         const uint16_t* q, double sm_scale, int64_t t0, int64_t t1,
                         const int32_t* items, int64_t n_items, double* out, double* lse,
                         int threads) {
  attn_job J;
  memset(&J, 0, sizeof J);
  J.k_cache = k_cache; J.v_cache = v_cache; J.kv_dtype = kv_dtype;
  J.Hq = Hq; J.Hkv = Hkv; J.D = D; J.block_size = block_size;
  J.table = table; J.max_blocks_per_seq = max_blocks_per_seq; J.seq_lens = seq_lens;
  J.k_scale = k_scale; J.v_scale = v_scale; J.q = q; J.sinks = NULL;
  J.window = 0; J.sm_scale = sm_scale; J.use_range = 1; J.t0 = t0; J.t1 = t1;
  J.items = items; J.n_items = n_items; J.out = out; J.lse = lse;
  run_job(&J, threads);
}

/* ------------------------------------------------------- merge ----------- */

/* Log-sum-exp combination of partial results, the sink counted once:
 *   M = max(sink, max_p lse_p);  Z = e^(sink-M) + sum_p e^(lse_p-M);
 *   out = sum_p e^(lse_p-M) o_p / Z;  lse = M + ln Z.
 * part_o [rows][S][D], part_lse [rows][S], num_parts [rows] or NULL (= S),
 * sink [rows] or NULL.  A part with lse = -inf has weight 0. */
void oracle_attn_merge(const double* part_o, const double* part_lse, const int32_t* num_parts,
                       const double* sink, int64_t rows, int S, int D, double* out,
                       double* lse_out) {
  for (int64_t r = 0; r < rows; r++) {
    int n = num_parts ? num_parts[r] : S;
    double sk = sink ? sink[r] : -INFINITY;
    double M = sk, Z;
    for (int p = 0; p < n; p++)
      if (part_lse[r * S + p] > M) M = part_lse[r * S + p];
    for (int d = 0; d < D; d++) out[r * D + d] = 0.0;
    if (M == -INFINITY) {
      if (lse_out) lse_out[r] = -INFINITY;
      continue;
    }
    Z = (sk == -INFINITY) ? 0.0 : exp(sk - M);
    for (int p = 0; p < n; p++) {
      double lp = part_lse[r * S + p];
      double w;
      if (lp == -INFINITY) continue;
      w = exp(lp - M);
      Z += w;
      for (int d = 0; d < D; d++) out[r * D + d] += w * part_o[(r * S + p) * D + d];
    }
    for (int d = 0; d < D; d++) out[r * D + d] /= Z;
    if (lse_out) lse_out[r] = M + log(Z);
  }
}
