/*
 * dt8 oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct CPU statement of the 8-bit optimizer step of
 * Section IV ("Optimizer State Quantization"): the dynamic-tree 8-bit data type,
 * block-wise absmax quantization / dequantization (Eq. quant1, quant2, quant3) and
 * the SGD-with-momentum (Eq. sgd) and Adam/AdamW (Eq. adam) updates wrapped into
 * "dequantize -> update in 32-bit -> quantize back" (Section I, Section IV-B).
 *
 * Only the tests, the smoke check and the benchmark's cpu-baseline leg may call
 * this file.  It shares no code, table, header or helper with the CUDA library and
 * must never be linked or imported by it.
 *
 * Precision: the paper fixes it -- states are dequantized to 32-bit floating point
 * and the weight update is done in 32-bit (Section I, Section IV-B), so every
 * state-path operation below is one IEEE binary32 operation, round-to-nearest-even,
 * in exactly the order written (compile with -ffp-contract=off, no fast-math).
 * The nearest-code decision (Eq. quant2) is taken in binary64, where the differences
 * |Q_j - v| of binary32 numbers are exact, so "nearest" is decided without rounding.
 *
 * Parity pins (see tests): every function here is pinned by invariants, closed forms,
 * brute force or a library special case, EXCEPT
 *   - the numeric VALUES of the code book: parity unpinned against the cited
 *     dynamic-tree data type (its source text is not available); they are pinned
 *     only to the paper's four-part description of the bit format;
 *   - the 100-step quantized trajectory: parity unpinned (the paper's evidence is
 *     recognition accuracy on a speech corpus, not reproducible here).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define DT8O_FLAG_BIAS_CORRECTION 1u
#define DT8O_FLAG_DECOUPLED_WD 2u

static int g_threads = 1;

/* Number of host threads used for the loop over quantization blocks (blocks are
 * independent: each is quantized on its own, Section IV-B "Tensor chunking"). */
void dt8o_set_threads(int t) { g_threads = t < 1 ? 1 : t; }
int dt8o_get_threads(void) {
#ifdef _OPENMP
  return g_threads;
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------------
 * Code book (Section IV-B, "Nearest value searching", Fig. dynamic_tree).
 *
 * The 8-bit pattern is: [sign bit] [E zero bits] [indicator bit 1] [F fraction bits].
 * The magnitude field has W bits (W = 7 after a sign bit, W = 8 for the unsigned
 * variant used for the non-negative second moment).  E, the length of the zero run,
 * is the decimal exponent; the F = W-1-E bits after the indicator hold an integer k
 * that steps linearly through the decade:
 *
 *     value(E,k) = 10^-E * (0.1 + 0.9*(k+1)/2^F) = (2^F + 9(k+1)) / (10^(E+1) * 2^F)
 *
 * evaluated as one binary64 division of two exact integers and rounded once to
 * binary32.  The all-zero field is the value 0.  The stored code is the index into
 * the ASCENDING table (Section IV-B, "Indexing": what is stored is the position i
 * of the chosen value q_i).
 * Signed table: out[127-p] = -value(p), out[128+p] = +value(p) for magnitude pattern
 * p (p = 0 is the value 0, so out[127] = out[128] = 0: the sign bit gives two zeros).
 * Unsigned table: out[p] = value(p).
 * ------------------------------------------------------------------------------ */
static float dt8o_pattern_value(int W, unsigned p) {
  if (p == 0) return 0.0f;
  int E = 0; /* zero bits before the indicator, scanning from the field's top bit */
  while (((p >> (W - 1 - E)) & 1u) == 0u) ++E;
  int F = W - 1 - E;
  unsigned k = p - (1u << F);
  int64_t num = ((int64_t)1 << F) + 9 * ((int64_t)k + 1);
  int64_t den = (int64_t)1 << F;
  for (int i = 0; i <= E; ++i) den *= 10;
  return (float)((double)num / (double)den);
}

int dt8o_codebook(int is_signed, float out[256]) {
  if (!out) return 1;
  if (is_signed) {
    for (unsigned p = 0; p < 128; ++p) {
      float v = dt8o_pattern_value(7, p);
      out[128 + p] = v;
      out[127 - p] = -v;
    }
  } else {
    for (unsigned p = 0; p < 256; ++p) out[p] = dt8o_pattern_value(8, p);
  }
  return 0;
}

/* ------------------------------------------------------------------------------
 * Nearest code, Eq. quant2: argmin_j |Q_j - v|, written out as the definition.
 * Differences are exact in binary64; the lowest index wins a tie (so the value 0 and
 * everything that rounds to it get code 127 in the signed table, never 128).
 * ------------------------------------------------------------------------------ */
uint8_t dt8o_nearest_scan(const float *Q, float v) {
  int best = 0;
  double bestd = fabs((double)Q[0] - (double)v);
  for (int j = 1; j < 256; ++j) {
    double d = fabs((double)Q[j] - (double)v);
    if (d < bestd) { bestd = d; best = j; }
  }
  return (uint8_t)best;
}

/* The same decision by bisection over the sorted table, the search the paper names
 * (Section IV-B, "Nearest value searching").  Finds the last entry <= v,
 * compares it with its upper neighbour, and returns the lowest index holding the
 * chosen value. */
uint8_t dt8o_nearest_bsearch(const float *Q, float v) {
  int j;
  if (!(v > Q[0])) {
    j = 0;
  } else if (!(v < Q[255])) {
    j = 255;
  } else {
    int lo = 0, hi = 255; /* invariant: Q[lo] <= v < Q[hi] */
    while (hi - lo > 1) {
      int mid = (lo + hi) / 2;
      if (Q[mid] <= v) lo = mid; else hi = mid;
    }
    double dlo = (double)v - (double)Q[lo];
    double dhi = (double)Q[hi] - (double)v;
    j = (dhi < dlo) ? hi : lo;
  }
  while (j > 0 && Q[j - 1] == Q[j]) --j;
  return (uint8_t)j;
}

void dt8o_nearest_many(const float *Q, const float *v, int64_t n, int use_scan, uint8_t *out) {
  for (int64_t i = 0; i < n; ++i)
    out[i] = use_scan ? dt8o_nearest_scan(Q, v[i]) : dt8o_nearest_bsearch(Q, v[i]);
}

/* ------------------------------------------------------------------------------
 * One block: Eq. quant1 (absmax, normalise by true division) + Eq. quant2.
 * An all-zero block has N_b = 0; its normalised values are taken as 0.
 * ------------------------------------------------------------------------------ */
static void quantize_block(const float *Q, const float *x, int cnt, int use_scan,
                           uint8_t *codes, float *absmax) {
  float N = 0.0f;
  for (int i = 0; i < cnt; ++i) {
    float a = fabsf(x[i]);
    if (a > N) N = a;
  }
  for (int i = 0; i < cnt; ++i) {
    float v = (N > 0.0f) ? x[i] / N : 0.0f;
    codes[i] = use_scan ? dt8o_nearest_scan(Q, v) : dt8o_nearest_bsearch(Q, v);
  }
  *absmax = N;
}

/* Eq. quant3: T^D = Q(code) * N_b, one binary32 multiply. */
static void dequantize_block(const float *Q, const uint8_t *codes, float N, int cnt, float *out) {
  for (int i = 0; i < cnt; ++i) out[i] = Q[codes[i]] * N;
}

static int block_size_ok(int B) { return B >= 1 && B <= 65536; }

/* Section IV-B "Tensor chunking": flatten, cut into ceil(n/B) blocks (the last one may
 * be short), quantize each block on its own. */
int dt8o_quantize_blockwise(const float *x, int64_t n, int B, int is_signed, int use_scan,
                            uint8_t *codes, float *absmax) {
  if (n < 0 || !block_size_ok(B)) return 1;
  float Q[256];
  dt8o_codebook(is_signed, Q);
  int64_t nb = (n + B - 1) / B;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads)
#endif
  for (int64_t b = 0; b < nb; ++b) {
    int64_t s = b * B;
    int cnt = (int)((n - s < B) ? (n - s) : B);
    quantize_block(Q, x + s, cnt, use_scan, codes + s, absmax + b);
  }
  return 0;
}

int dt8o_dequantize_blockwise(const uint8_t *codes, const float *absmax, int64_t n, int B,
                              int is_signed, float *out) {
  if (n < 0 || !block_size_ok(B)) return 1;
  float Q[256];
  dt8o_codebook(is_signed, Q);
  int64_t nb = (n + B - 1) / B;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads)
#endif
  for (int64_t b = 0; b < nb; ++b) {
    int64_t s = b * B;
    int cnt = (int)((n - s < B) ? (n - s) : B);
    dequantize_block(Q, codes + s, absmax[b], cnt, out + s);
  }
  return 0;
}

/* bfloat16 -> binary32 is exact: the 16 bits are the top half of the binary32 word. */
static float bf16_widen(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
static float grad_at(const void *g, int g_dtype, int64_t i) {
  return g_dtype == 0 ? ((const float *)g)[i] : bf16_widen(((const uint16_t *)g)[i]);
}

/* binary32 -> bfloat16, round to nearest, ties to even: the value is cut after the 8th
 * significand bit; the 16 dropped bits decide (more than half: up; exactly half: to the even
 * neighbour).  A NaN keeps its top bits with the quiet bit set. */
uint16_t dt8o_bf16_round(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x0040u);
  uint32_t kept = u >> 16, dropped = u & 0xFFFFu;
  if (dropped > 0x8000u || (dropped == 0x8000u && (kept & 1u))) kept += 1;
  return (uint16_t)kept;
}

void dt8o_bf16_round_many(const float *x, int64_t n, uint16_t *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = dt8o_bf16_round(x[i]);
}

/* Parameters are binary32 in the paper (Section II: 32-bit floating point).  The bfloat16
 * parameter variant (no 32-bit master copy) is a reading: the stored parameter is widened
 * exactly, the update of Eq. sgd / Eq. adam runs in binary32 as written, and the result is
 * rounded once, to nearest even, when it is stored. */
static float param_at(const void *w, int p_dtype, int64_t i) {
  return p_dtype == 0 ? ((const float *)w)[i] : bf16_widen(((const uint16_t *)w)[i]);
}
static void param_store(void *w, int p_dtype, int64_t i, float v) {
  if (p_dtype == 0) ((float *)w)[i] = v;
  else ((uint16_t *)w)[i] = dt8o_bf16_round(v);
}

/* ------------------------------------------------------------------------------
 * Eq. sgd on exact binary32 state (no quantizer):
 *     g' = g + wd*w      (weight decay as in the training recipe of Section V; skipped
 *                         when wd == 0)
 *     m  = beta*m + g'   (from m = 0 the first step gives m = g', which is m_0 = g_0)
 *     w  = w - lr*m
 * ------------------------------------------------------------------------------ */
void dt8o_sgd_update_fp32(float *w, const float *g, float *m, int64_t n, float lr, float beta,
                          float wd) {
  for (int64_t i = 0; i < n; ++i) {
    float gi = g[i];
    if (wd != 0.0f) gi = gi + wd * w[i];
    float mi = beta * m[i] + gi;
    m[i] = mi;
    w[i] = w[i] - lr * mi;
  }
}

/* Bias-correction factors 1 - beta^t, evaluated in binary64 and rounded to binary32;
 * both are 1 when bias correction is off (the literal Eq. adam). */
static void adam_bias(float beta1, float beta2, int64_t step, uint32_t flags, float *bc1,
                      float *bc2) {
  if (flags & DT8O_FLAG_BIAS_CORRECTION) {
    *bc1 = (float)(1.0 - pow((double)beta1, (double)step));
    *bc2 = (float)(1.0 - pow((double)beta2, (double)step));
  } else {
    *bc1 = 1.0f;
    *bc2 = 1.0f;
  }
}

/* ------------------------------------------------------------------------------
 * Eq. adam on exact binary32 state (no quantizer):
 *     decoupled decay (AdamW): w = w*(1 - lr*wd);   coupled: g = g + wd*w
 *     m = beta1*m + (1-beta1)*g
 *     r = beta2*r + (1-beta2)*(g*g)
 *     w = w - lr * (m/bc1) / (sqrt(r/bc2) + eps)
 * ------------------------------------------------------------------------------ */
void dt8o_adam_update_fp32(float *w, const float *g, float *m, float *r, int64_t n, float lr,
                           float beta1, float beta2, float eps, float wd, int64_t step,
                           uint32_t flags) {
  float bc1, bc2;
  adam_bias(beta1, beta2, step, flags, &bc1, &bc2);
  const float omb1 = 1.0f - beta1;
  const float omb2 = 1.0f - beta2;
  const float decay = 1.0f - lr * wd;
  for (int64_t i = 0; i < n; ++i) {
    float gi = g[i];
    float wi = w[i];
    if (wd != 0.0f) {
      if (flags & DT8O_FLAG_DECOUPLED_WD) wi = wi * decay;
      else gi = gi + wd * wi;
    }
    float mi = beta1 * m[i] + omb1 * gi;
    float ri = beta2 * r[i] + omb2 * (gi * gi);
    m[i] = mi;
    r[i] = ri;
    float mhat = mi / bc1;
    float rhat = ri / bc2;
    float upd = mhat / (sqrtf(rhat) + eps);
    w[i] = wi - lr * upd;
  }
}

/* ------------------------------------------------------------------------------
 * 8-bit SGD step (Section I / IV-B: states 8-bit -> 32-bit, weight update in 32-bit
 * with the 32-bit states, states quantized back with a fresh absmax).
 * ------------------------------------------------------------------------------ */
int dt8o_sgd_step_ex(void *w, int p_dtype, const void *g, int g_dtype, uint8_t *m_codes,
                     float *m_absmax, int64_t n, float lr, float beta, float wd, int64_t step, int B) {
  (void)step;
  if (n < 0 || !block_size_ok(B)) return 1;
  float Qs[256];
  dt8o_codebook(1, Qs);
  int64_t nb = (n + B - 1) / B;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads)
#endif
  for (int64_t b = 0; b < nb; ++b) {
    int64_t s = b * B;
    int cnt = (int)((n - s < B) ? (n - s) : B);
    float *m = (float *)malloc(sizeof(float) * (size_t)cnt);
    float *gb = (float *)malloc(sizeof(float) * (size_t)cnt);
    float *wb = (float *)malloc(sizeof(float) * (size_t)cnt);
    for (int i = 0; i < cnt; ++i) gb[i] = grad_at(g, g_dtype, s + i);
    for (int i = 0; i < cnt; ++i) wb[i] = param_at(w, p_dtype, s + i);
    dequantize_block(Qs, m_codes + s, m_absmax[b], cnt, m);
    dt8o_sgd_update_fp32(wb, gb, m, cnt, lr, beta, wd);
    quantize_block(Qs, m, cnt, 0, m_codes + s, m_absmax + b);
    for (int i = 0; i < cnt; ++i) param_store(w, p_dtype, s + i, wb[i]);
    free(m);
    free(gb);
    free(wb);
  }
  return 0;
}

int dt8o_sgd_step(float *w, const void *g, int g_dtype, uint8_t *m_codes, float *m_absmax,
                  int64_t n, float lr, float beta, float wd, int64_t step, int B) {
  return dt8o_sgd_step_ex(w, 0, g, g_dtype, m_codes, m_absmax, n, lr, beta, wd, step, B);
}

/* 8-bit Adam / AdamW step: first moment on the signed table, second moment on the
 * unsigned table. */
int dt8o_adam_step_ex(void *w, int p_dtype, const void *g, int g_dtype, uint8_t *m_codes,
                      float *m_absmax, uint8_t *r_codes, float *r_absmax, int64_t n, float lr,
                      float beta1, float beta2, float eps, float wd, int64_t step, int B,
                      uint32_t flags) {
  if (n < 0 || !block_size_ok(B) || step < 1) return 1;
  float Qs[256], Qu[256];
  dt8o_codebook(1, Qs);
  dt8o_codebook(0, Qu);
  int64_t nb = (n + B - 1) / B;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(g_threads)
#endif
  for (int64_t b = 0; b < nb; ++b) {
    int64_t s = b * B;
    int cnt = (int)((n - s < B) ? (n - s) : B);
    float *m = (float *)malloc(sizeof(float) * (size_t)cnt);
    float *r = (float *)malloc(sizeof(float) * (size_t)cnt);
    float *gb = (float *)malloc(sizeof(float) * (size_t)cnt);
    float *wb = (float *)malloc(sizeof(float) * (size_t)cnt);
    for (int i = 0; i < cnt; ++i) gb[i] = grad_at(g, g_dtype, s + i);
    for (int i = 0; i < cnt; ++i) wb[i] = param_at(w, p_dtype, s + i);
    dequantize_block(Qs, m_codes + s, m_absmax[b], cnt, m);
    dequantize_block(Qu, r_codes + s, r_absmax[b], cnt, r);
    dt8o_adam_update_fp32(wb, gb, m, r, cnt, lr, beta1, beta2, eps, wd, step, flags);
    quantize_block(Qs, m, cnt, 0, m_codes + s, m_absmax + b);
    quantize_block(Qu, r, cnt, 0, r_codes + s, r_absmax + b);
    for (int i = 0; i < cnt; ++i) param_store(w, p_dtype, s + i, wb[i]);
    free(m);
    free(r);
    free(gb);
    free(wb);
  }
  return 0;
}

int dt8o_adam_step(float *w, const void *g, int g_dtype, uint8_t *m_codes, float *m_absmax,
                   uint8_t *r_codes, float *r_absmax, int64_t n, float lr, float beta1,
                   float beta2, float eps, float wd, int64_t step, int B, uint32_t flags) {
  return dt8o_adam_step_ex(w, 0, g, g_dtype, m_codes, m_absmax, r_codes, r_absmax, n, lr, beta1,
                           beta2, eps, wd, step, B, flags);
}
