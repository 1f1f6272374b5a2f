/*
 * CPU oracle for the QTALE token-adaptive quantised layer forward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, step-by-step
 * definition of what the layer path computes, written from the paper
 * (arXiv 2602.10431): residual layer update (Eq. 1), execute / bypass rule
 * (Eq. 3), softmax-probability threshold rule with one global theta (Eq. 9),
 * gathering of the active tokens into a dense tensor (App. B.2), and b-bit
 * group-quantised weights (Sec. 4.1, implementation details).  It shares no
 * code with the CUDA library and must never be called from the product path.
 *
 * Storage is fp32, every reduction accumulates in fp64 in index order.  The
 * only parallelism is an optional OpenMP "parallel for" over independent
 * output rows, which does not change any arithmetic.
 *
 * Parts the paper leaves open and that this file fixes (so no external pin
 * exists for them -- "parity unpinned"): the attention / KV treatment of
 * bypassed tokens (they produce no Q, K, V at that layer), RoPE using the
 * original position, the min/max quantiser's rounding, top-k selection
 * (an extension; the paper controls the ratio through theta only), the ReLU
 * of the MLP router (Eq. 2 names neither width nor activation), and the
 * rounding k = floor(ratio n + 0.5) of the theta quantile for a target ratio.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 1;
static int g_emulate_bf16 = 0;

void orc_set_threads(int n) {
  g_threads = n < 1 ? 1 : n;
#ifdef _OPENMP
  omp_set_num_threads(g_threads);
#endif
}
int orc_get_threads(void) {
#ifdef _OPENMP
  return g_threads;
#else
  return 1;
#endif
}
/* Diagnostic only: round to bf16 at the tensors a bf16 pipeline materialises. */
void orc_set_emulate_bf16(int on) { g_emulate_bf16 = on; }

/* ---- small format helpers ------------------------------------------------ */

static float half_bits_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) & 1u;
  uint32_t exp = (uint32_t)(h >> 10) & 0x1Fu;
  uint32_t man = (uint32_t)h & 0x3FFu;
  double v;
  if (exp == 0) {
    v = ldexp((double)man, -24); /* subnormal: man * 2^-10 * 2^-14 */
  } else if (exp == 31) {
    v = man ? NAN : INFINITY;
  } else {
    v = ldexp(1.0 + (double)man / 1024.0, (int)exp - 15);
  }
  return (float)(sign ? -v : v);
}

static uint16_t float_to_half_bits(float f) {
  /* round-to-nearest-even conversion of a finite float to IEEE binary16 */
  if (isnan(f)) return 0x7E00u;
  uint16_t sign = signbit(f) ? 0x8000u : 0u;
  double a = fabs((double)f);
  if (a >= 65520.0) return (uint16_t)(sign | 0x7C00u);
  if (a < ldexp(1.0, -25)) return sign;
  int e;
  double m = frexp(a, &e); /* a = m * 2^e, m in [0.5,1) */
  int exp = e - 1;         /* a = (2m) * 2^exp, 2m in [1,2) */
  if (exp < -14) {
    double q = nearbyint(ldexp(a, 24)); /* units of 2^-24 */
    return (uint16_t)(sign | (uint16_t)q);
  }
  double frac = nearbyint(ldexp(2.0 * m - 1.0, 10)); /* 0..1024 */
  uint32_t bits = ((uint32_t)(exp + 15) << 10) + (uint32_t)frac; /* carry bumps exponent */
  return (uint16_t)(sign | (uint16_t)bits);
}

static float round_bf16(float x) {
  uint32_t b;
  memcpy(&b, &x, 4);
  if ((b & 0x7F800000u) == 0x7F800000u) return x;
  b += 0x7FFFu + ((b >> 16) & 1u);
  b &= 0xFFFF0000u;
  memcpy(&x, &b, 4);
  return x;
}
static void maybe_bf16(float* p, size_t n) {
  if (!g_emulate_bf16) return;
  for (size_t i = 0; i < n; ++i) p[i] = round_bf16(p[i]);
}

float orc_half_to_float(uint16_t h) { return half_bits_to_float(h); }
uint16_t orc_float_to_half(float f) { return float_to_half_bits(f); }
float orc_round_bf16(float f) { return round_bf16(f); }

/* ---- router (Eq. 2, Eq. 9) ----------------------------------------------- */

/* Two-class router with logits (g0, g1): p0 = softmax(g)[0].  With a linear
 * router, g0 - g1 = w.x + b, and softmax over two classes is the logistic
 * function of the logit difference.  z_out (optional) receives the fp64 logit
 * difference, p_out the probability rounded to fp32. */
void orc_router_scores(const float* x, int T, int d, const float* w, float bias,
                       float* p_out, double* z_out) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    double z = 0.0;
    for (int k = 0; k < d; ++k) z += (double)x[(size_t)t * d + k] * (double)w[k];
    z += (double)bias;
    if (z_out) z_out[t] = z;
    p_out[t] = (float)(1.0 / (1.0 + exp(-z)));
  }
}

/* Router as a small MLP (Eq. 2: "a lightweight MLP" emits the two class logits):
 * u = W1 x + b1 (hidden units), a = max(u, 0), (g0, g1) = W2 a + b2, and
 * p0 = softmax([g0, g1])[0] (Eq. 9).  The paper gives neither the width nor the
 * activation; ReLU is this library's reading ("parity unpinned" by the paper).
 * w1 [h, d], b1 [h], w2 [2, h] (row 0: execute logit, row 1: bypass logit), b2 [2]. */
void orc_router_mlp_scores(const float* x, int T, int d, const float* w1, const float* b1, int h,
                           const float* w2, const float* b2, float* p_out, double* z_out) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    double g0 = (double)b2[0], g1 = (double)b2[1];
    for (int j = 0; j < h; ++j) {
      double u = 0.0;
      for (int k = 0; k < d; ++k) u += (double)x[(size_t)t * d + k] * (double)w1[(size_t)j * d + k];
      u += (double)b1[j];
      const double a = u > 0.0 ? u : 0.0;
      g0 += (double)w2[j] * a;
      g1 += (double)w2[(size_t)h + j] * a;
    }
    const double m = g0 > g1 ? g0 : g1;
    const double e0 = exp(g0 - m), e1 = exp(g1 - m);
    if (z_out) z_out[t] = g0 - g1;
    p_out[t] = (float)(e0 / (e0 + e1));
  }
}

/* General two-logit form of Eq. 9: p = softmax([g0, g1]); returns p[0]. */
void orc_softmax2_p0(const double* g0, const double* g1, int T, float* p_out) {
  for (int t = 0; t < T; ++t) {
    double m = g0[t] > g1[t] ? g0[t] : g1[t];
    double e0 = exp(g0[t] - m), e1 = exp(g1[t] - m);
    p_out[t] = (float)(e0 / (e0 + e1));
  }
}

/* Eq. 9: execute iff p0 >= theta.  Padding tokens (valid == 0) never execute
 * (App. B.2: padding is skipped by the routing decision). */
void orc_select_threshold(const float* p, const uint8_t* valid, int T, float theta,
                          uint8_t* mask) {
  for (int t = 0; t < T; ++t) {
    int ok = valid ? (valid[t] != 0) : 1;
    mask[t] = (uint8_t)(ok && (p[t] >= theta));
  }
}

/* Extension (not in the paper): number of tokens for a requested ratio. */
int orc_topk_count(double ratio, int n_valid) {
  double k = floor(ratio * (double)n_valid + 0.5);
  if (k < 0) k = 0;
  if (k > n_valid) k = n_valid;
  return (int)k;
}

/* Extension: the k valid tokens with the highest score; equal scores are
 * ordered by lower token index first.  O(T k) selection, no sort library. */
void orc_select_topk(const float* p, const uint8_t* valid, int T, int k, uint8_t* mask) {
  memset(mask, 0, (size_t)T);
  for (int r = 0; r < k; ++r) {
    int best = -1;
    for (int t = 0; t < T; ++t) {
      if (mask[t]) continue;
      if (valid && !valid[t]) continue;
      if (best < 0 || p[t] > p[best]) best = t; /* strict: lower index wins ties */
    }
    if (best < 0) break;
    mask[best] = 1;
  }
}

/* Threshold for a requested execution ratio (Sec. 3.4: one global theta sets the
 * ratio after training; lowering it executes more).  Given pooled router scores
 * of a calibration batch, the theta for which a share `ratio` of the valid
 * scores satisfies p >= theta (Eq. 9) is the k-th largest valid score with
 * k = floor(ratio * n_valid + 0.5): written out as a full descending sort.
 * k = 0: theta = 2, above every probability.  Returns theta, *count = number of
 * valid scores >= theta (more than k only when scores tie at theta). */
static int cmp_float_desc(const void* a, const void* b) {
  const float x = *(const float*)a, y = *(const float*)b;
  return (x < y) - (x > y);
}
float orc_theta_for_ratio(const float* p, const uint8_t* valid, long n, double ratio, long* count) {
  float* v = (float*)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
  long nv = 0;
  for (long i = 0; i < n; ++i)
    if (!valid || valid[i]) v[nv++] = p[i];
  double kd = floor(ratio * (double)nv + 0.5);
  if (kd < 0) kd = 0;
  if (kd > (double)nv) kd = (double)nv;
  const long k = (long)kd;
  float theta = 2.0f;
  long c = 0;
  if (k > 0) {
    qsort(v, (size_t)nv, sizeof(float), cmp_float_desc);
    theta = v[k - 1];
    for (long i = 0; i < nv; ++i) c += v[i] >= theta;
  }
  free(v);
  if (count) *count = c;
  return theta;
}

/* Active-token gather bookkeeping (App. B.2): ascending index list, count,
 * per-sequence offsets of executed tokens and each executed token's position
 * inside its own sequence. */
void orc_compact_indices(const uint8_t* mask, int T, const int32_t* cu_seqlens, int B,
                         int32_t* idx, int32_t* n_exec, int32_t* cu_exec, int32_t* pos) {
  int n = 0;
  int b = 0;
  if (cu_exec) cu_exec[0] = 0;
  for (int t = 0; t < T; ++t) {
    while (b < B && t >= cu_seqlens[b + 1]) {
      ++b;
      if (cu_exec) cu_exec[b] = n;
    }
    if (mask[t]) {
      idx[n] = t;
      if (pos) pos[n] = t - cu_seqlens[b];
      ++n;
    }
  }
  while (b < B) {
    ++b;
    if (cu_exec) cu_exec[b] = n;
  }
  *n_exec = n;
}

/* ---- quantised weights (Sec. 4.1: 4-bit / 3-bit, per-group parameters; the mixed
 * ---- precision appendix interleaves 4-bit and 2-bit layers).  A row of b-bit codes is
 * ---- a little-endian bit stream: code k occupies bits b k .. b k + b - 1. ---- */

static int row_bytes_for(int K, int bits) {
  return (bits * K + 7) / 8;
}
int orc_row_bytes(int K, int bits) { return row_bytes_for(K, bits); }

static unsigned get_code(const uint8_t* row, int k, int bits) {
  if (bits == 4) {
    uint8_t b = row[k >> 1];
    return (k & 1) ? (unsigned)(b >> 4) : (unsigned)(b & 0xF);
  }
  unsigned v = 0;
  for (int j = 0; j < bits; ++j) {
    int bb = bits * k + j;
    v |= (unsigned)((row[bb >> 3] >> (bb & 7)) & 1u) << j;
  }
  return v;
}

static void put_code(uint8_t* row, int k, int bits, unsigned q) {
  if (bits == 4) {
    if (k & 1)
      row[k >> 1] = (uint8_t)((row[k >> 1] & 0x0F) | (q << 4));
    else
      row[k >> 1] = (uint8_t)((row[k >> 1] & 0xF0) | (q & 0xF));
    return;
  }
  for (int j = 0; j < bits; ++j) {
    int bb = bits * k + j;
    uint8_t m = (uint8_t)(1u << (bb & 7));
    if ((q >> j) & 1u)
      row[bb >> 3] |= m;
    else
      row[bb >> 3] &= (uint8_t)~m;
  }
}

void orc_pack_codes(const uint8_t* codes, int N, int K, int bits, uint8_t* packed) {
  int rb = row_bytes_for(K, bits);
  memset(packed, 0, (size_t)N * rb);
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) put_code(packed + (size_t)n * rb, k, bits, codes[(size_t)n * K + k]);
}

void orc_unpack_codes(const uint8_t* packed, int N, int K, int bits, uint8_t* codes) {
  int rb = row_bytes_for(K, bits);
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k)
      codes[(size_t)n * K + k] = (uint8_t)get_code(packed + (size_t)n * rb, k, bits);
}

/* Uniform affine dequantisation: w_hat = (q - zero) * scale, group g = k / G.
 * Every factor is exactly representable and the product is exact in fp32. */
void orc_dequantize(const uint8_t* packed, const uint16_t* scales, const uint16_t* zeros,
                    int N, int K, int bits, int group, float* w_hat) {
  int rb = row_bytes_for(K, bits);
  int ng = (K + group - 1) / group;
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n) {
    for (int k = 0; k < K; ++k) {
      int g = k / group;
      float s = half_bits_to_float(scales[(size_t)n * ng + g]);
      float z = half_bits_to_float(zeros[(size_t)n * ng + g]);
      float q = (float)get_code(packed + (size_t)n * rb, k, bits);
      w_hat[(size_t)n * K + k] = (q - z) * s;
    }
  }
}

/* Min/max asymmetric quantiser used to make synthetic weights and to pin
 * dequantise by a round trip.  Range always contains 0. */
void orc_quantize(const float* w, int N, int K, int bits, int group, uint8_t* codes,
                  uint16_t* scales, uint16_t* zeros) {
  int ng = (K + group - 1) / group;
  float qmax = (float)((1 << bits) - 1);
  for (int n = 0; n < N; ++n) {
    for (int g = 0; g < ng; ++g) {
      int k0 = g * group, k1 = k0 + group < K ? k0 + group : K;
      float lo = 0.f, hi = 0.f;
      for (int k = k0; k < k1; ++k) {
        float v = w[(size_t)n * K + k];
        if (v < lo) lo = v;
        if (v > hi) hi = v;
      }
      uint16_t sb = float_to_half_bits((hi - lo) / qmax);
      float s = half_bits_to_float(sb);
      if (s == 0.f) {
        s = 1.f;
        sb = float_to_half_bits(1.f);
      }
      float z = rintf(-lo / s);
      if (z < 0.f) z = 0.f;
      if (z > qmax) z = qmax;
      scales[(size_t)n * ng + g] = sb;
      zeros[(size_t)n * ng + g] = float_to_half_bits(z);
      for (int k = k0; k < k1; ++k) {
        float q = rintf(w[(size_t)n * K + k] / s) + z;
        if (q < 0.f) q = 0.f;
        if (q > qmax) q = qmax;
        codes[(size_t)n * K + k] = (uint8_t)q;
      }
    }
  }
}

/* Re-quantise already dequantised values with FIXED (scale, zero): used to pin
 * that dequantise -> quantise reproduces the integer codes. */
void orc_requantize_fixed(const float* w_hat, const uint16_t* scales, const uint16_t* zeros,
                          int N, int K, int bits, int group, uint8_t* codes) {
  int ng = (K + group - 1) / group;
  float qmax = (float)((1 << bits) - 1);
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) {
      int g = k / group;
      float s = half_bits_to_float(scales[(size_t)n * ng + g]);
      float z = half_bits_to_float(zeros[(size_t)n * ng + g]);
      float q = rintf(w_hat[(size_t)n * K + k] / s) + z;
      if (q < 0.f) q = 0.f;
      if (q > qmax) q = qmax;
      codes[(size_t)n * K + k] = (uint8_t)q;
    }
}

/* ---- dense building blocks of f_l (Eq. 1) ---------------------------------- */

/* y[t,:] = x[t,:] / sqrt(mean_k x^2 + eps) * gamma */
void orc_rmsnorm(const float* x, int T, int d, const float* gamma, float eps, float* y) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    double ss = 0.0;
    for (int k = 0; k < d; ++k) ss += (double)x[(size_t)t * d + k] * (double)x[(size_t)t * d + k];
    double inv = 1.0 / sqrt(ss / (double)d + (double)eps);
    for (int k = 0; k < d; ++k)
      y[(size_t)t * d + k] = (float)((double)x[(size_t)t * d + k] * inv * (double)gamma[k]);
  }
}

/* y[t,n] = sum_k x[t,k] * w[n,k]   (y = x W^T) */
void orc_linear(const float* x, int T, int K, const float* w, int N, float* y) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int n = 0; n < N; ++n) {
      double acc = 0.0;
      const float* xr = x + (size_t)t * K;
      const float* wr = w + (size_t)n * K;
      for (int k = 0; k < K; ++k) acc += (double)xr[k] * (double)wr[k];
      y[(size_t)t * N + n] = (float)acc;
    }
  }
}

/* Rotary embedding, rotate-half pairing (j, j + hd/2), angle pos * base^(-2j/hd).
 * v is [T, n_heads, hd] with row stride `stride` floats. */
void orc_rope(float* v, int T, int n_heads, int hd, size_t stride, const int32_t* pos,
              float base) {
  int half = hd / 2;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int j = 0; j < half; ++j) {
      double inv_freq = pow((double)base, -2.0 * (double)j / (double)hd);
      double ang = (double)pos[t] * inv_freq;
      double c = cos(ang), s = sin(ang);
      for (int h = 0; h < n_heads; ++h) {
        float* p = v + (size_t)t * stride + (size_t)h * hd;
        double a = p[j], b = p[j + half];
        p[j] = (float)(a * c - b * s);
        p[j + half] = (float)(b * c + a * s);
      }
    }
  }
}

void orc_swiglu(const float* gate, const float* up, size_t n, float* out) {
  for (size_t i = 0; i < n; ++i) {
    double g = gate[i];
    out[i] = (float)(g / (1.0 + exp(-g)) * (double)up[i]);
  }
}

/* Causal softmax attention over the tokens that exist at this layer.
 *
 * Queries: the Te executed tokens of this call (q: [Te, H, hd]).  Keys/values
 * visible to executed token i of sequence s: the kv_len[s] entries already in
 * that sequence's cache for this layer (all from earlier positions), then the
 * executed tokens j of the same sequence in this call with pos[j] <= pos[i].
 * Bypassed tokens contribute nothing (they never produced K or V here).
 * cache_k / cache_v: [B, cap, H_kv, hd] (may be NULL when kv_len is NULL).
 */
void orc_attention(const float* q, const float* k, const float* v, int Te, int H, int Hkv,
                   int hd, const int32_t* seq_of, const int32_t* pos, const float* cache_k,
                   const float* cache_v, const int32_t* kv_len, int cap, float* out) {
  int rep = H / Hkv;
  double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel for schedule(dynamic, 4)
  for (int i = 0; i < Te; ++i) {
    int s = seq_of[i];
    int nc = kv_len ? kv_len[s] : 0;
    /* executed tokens of one sequence are contiguous and ascending in the list */
    int j0 = i;
    while (j0 > 0 && seq_of[j0 - 1] == s) --j0;
    int nk = nc + (i - j0 + 1);
    double* sc = (double*)malloc(sizeof(double) * (size_t)nk);
    for (int h = 0; h < H; ++h) {
      int hk = h / rep;
      const float* qi = q + ((size_t)i * H + h) * hd;
      double mx = -INFINITY;
      for (int c = 0; c < nk; ++c) {
        const float* kc = c < nc ? cache_k + (((size_t)s * cap + c) * Hkv + hk) * hd
                                 : k + ((size_t)(j0 + c - nc) * Hkv + hk) * hd;
        double dot = 0.0;
        for (int e = 0; e < hd; ++e) dot += (double)qi[e] * (double)kc[e];
        sc[c] = dot * scale;
        if (sc[c] > mx) mx = sc[c];
      }
      double den = 0.0;
      for (int c = 0; c < nk; ++c) {
        sc[c] = exp(sc[c] - mx);
        den += sc[c];
      }
      float* o = out + ((size_t)i * H + h) * hd;
      for (int e = 0; e < hd; ++e) {
        double acc = 0.0;
        for (int c = 0; c < nk; ++c) {
          const float* vc = c < nc ? cache_v + (((size_t)s * cap + c) * Hkv + hk) * hd
                                   : v + ((size_t)(j0 + c - nc) * Hkv + hk) * hd;
          acc += sc[c] * (double)vc[e];
        }
        o[e] = (float)(acc / den);
      }
    }
    free(sc);
    (void)pos;
  }
}

/* ---- the token-adaptive layer (Eq. 1, 3, 9; App. B.2) ----------------------- */

typedef struct {
  int d, n_heads, n_kv_heads, head_dim, ffn;
  float rms_eps, rope_theta;
} orc_layer_shape;

typedef struct {
  const float* w_qkv;  /* [(H + 2 Hkv) hd, d]  dequantised */
  const float* w_o;    /* [d, H hd] */
  const float* w_gate_up; /* [2 F, d]: gate rows then up rows */
  const float* w_down; /* [d, F] */
  const float* gamma1; /* [d] */
  const float* gamma2; /* [d] */
} orc_layer_weights;

/* x: [T, d] in, x_out: [T, d] out (may alias).  mask[t] = execute decision.
 * pos0[b]: position of the first token of sequence b in this call (NULL = 0).
 * cache_k / cache_v / kv_len: per-layer KV cache, updated for executed tokens
 * only (NULL = no cache).  Returns the number of executed tokens. */
int orc_layer_forward(const orc_layer_shape* sh, const orc_layer_weights* W, const float* x,
                      int T, const int32_t* cu_seqlens, int B, const uint8_t* mask,
                      const int32_t* pos0, float* cache_k, float* cache_v, int32_t* kv_len,
                      int cap, float* x_out) {
  int d = sh->d, H = sh->n_heads, Hkv = sh->n_kv_heads, hd = sh->head_dim, F = sh->ffn;
  int qd = H * hd, kvd = Hkv * hd, nqkv = qd + 2 * kvd;

  int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T + 1));
  int32_t* pos = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T + 1));
  int32_t* cu_exec = (int32_t*)malloc(sizeof(int32_t) * (size_t)(B + 1));
  int32_t* seq_of = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T + 1));
  int32_t Te = 0;
  orc_compact_indices(mask, T, cu_seqlens, B, idx, &Te, cu_exec, pos);
  for (int b = 0; b < B; ++b)
    for (int i = cu_exec[b]; i < cu_exec[b + 1]; ++i) {
      seq_of[i] = b;
      if (pos0) pos[i] += pos0[b];
    }

  /* bypass: x_{l+1} = x_l (Eq. 3, second case) */
  if (x_out != x) memcpy(x_out, x, sizeof(float) * (size_t)T * d);
  if (Te == 0) {
    free(idx); free(pos); free(cu_exec); free(seq_of);
    return 0;
  }

  size_t te = (size_t)Te;
  float* xc = (float*)malloc(sizeof(float) * te * d);
  float* hn = (float*)malloc(sizeof(float) * te * d);
  float* qkv = (float*)malloc(sizeof(float) * te * nqkv);
  float* qb = (float*)malloc(sizeof(float) * te * qd);
  float* kb = (float*)malloc(sizeof(float) * te * kvd);
  float* vb = (float*)malloc(sizeof(float) * te * kvd);
  float* ao = (float*)malloc(sizeof(float) * te * qd);
  float* a = (float*)malloc(sizeof(float) * te * d);
  float* u = (float*)malloc(sizeof(float) * te * d);
  float* gu = (float*)malloc(sizeof(float) * te * 2 * F);
  float* act = (float*)malloc(sizeof(float) * te * F);
  float* m = (float*)malloc(sizeof(float) * te * d);

  /* gather the active tokens into a dense tensor (App. B.2) */
  for (size_t i = 0; i < te; ++i) memcpy(xc + i * d, x + (size_t)idx[i] * d, sizeof(float) * d);

  orc_rmsnorm(xc, Te, d, W->gamma1, sh->rms_eps, hn);
  maybe_bf16(hn, te * d);
  orc_linear(hn, Te, d, W->w_qkv, nqkv, qkv);
  for (size_t i = 0; i < te; ++i) {
    memcpy(qb + i * qd, qkv + i * nqkv, sizeof(float) * qd);
    memcpy(kb + i * kvd, qkv + i * nqkv + qd, sizeof(float) * kvd);
    memcpy(vb + i * kvd, qkv + i * nqkv + qd + kvd, sizeof(float) * kvd);
  }
  orc_rope(qb, Te, H, hd, (size_t)qd, pos, sh->rope_theta);
  orc_rope(kb, Te, Hkv, hd, (size_t)kvd, pos, sh->rope_theta);
  maybe_bf16(qb, te * qd);
  maybe_bf16(kb, te * kvd);
  maybe_bf16(vb, te * kvd);

  orc_attention(qb, kb, vb, Te, H, Hkv, hd, seq_of, pos, cache_k, cache_v, kv_len, cap, ao);
  maybe_bf16(ao, te * qd);

  /* executed tokens (and only they) enter this layer's KV cache */
  if (kv_len) {
    for (int b = 0; b < B; ++b) {
      for (int i = cu_exec[b]; i < cu_exec[b + 1]; ++i) {
        int slot = kv_len[b] + (i - cu_exec[b]);
        memcpy(cache_k + ((size_t)b * cap + slot) * kvd, kb + (size_t)i * kvd, sizeof(float) * kvd);
        memcpy(cache_v + ((size_t)b * cap + slot) * kvd, vb + (size_t)i * kvd, sizeof(float) * kvd);
      }
    }
    for (int b = 0; b < B; ++b) kv_len[b] += cu_exec[b + 1] - cu_exec[b];
  }

  orc_linear(ao, Te, qd, W->w_o, d, a);
  for (size_t i = 0; i < te * d; ++i) u[i] = xc[i] + a[i];
  orc_rmsnorm(u, Te, d, W->gamma2, sh->rms_eps, hn);
  maybe_bf16(hn, te * d);
  orc_linear(hn, Te, d, W->w_gate_up, 2 * F, gu);
  for (size_t i = 0; i < te; ++i) orc_swiglu(gu + i * 2 * F, gu + i * 2 * F + F, (size_t)F, act + i * F);
  maybe_bf16(act, te * F);
  orc_linear(act, Te, F, W->w_down, d, m);

  /* execute: x_{l+1} = x_l + f_l(x_l), f_l = attention branch + MLP branch (Eq. 1, 3) */
  for (size_t i = 0; i < te; ++i) {
    float* o = x_out + (size_t)idx[i] * d;
    for (int k = 0; k < d; ++k) {
      double f = (double)a[i * d + k] + (double)m[i * d + k];
      o[k] = (float)((double)xc[i * d + k] + f);
    }
    if (g_emulate_bf16)
      for (int k = 0; k < d; ++k) o[k] = round_bf16(o[k]);
  }

  free(xc); free(hn); free(qkv); free(qb); free(kb); free(vb); free(ao); free(a); free(u);
  free(gu); free(act); free(m); free(idx); free(pos); free(cu_exec); free(seq_of);
  return Te;
}

/* Row gather / residual scatter as standalone steps (App. B.2; Eq. 3). */
void orc_gather_rows(const float* x, const int32_t* idx, int n, int d, float* xc) {
  for (int i = 0; i < n; ++i) memcpy(xc + (size_t)i * d, x + (size_t)idx[i] * d, sizeof(float) * d);
}
void orc_scatter_add(float* x, const float* xc, const float* f, const int32_t* idx, int n, int d) {
  for (int i = 0; i < n; ++i)
    for (int k = 0; k < d; ++k)
      x[(size_t)idx[i] * d + k] = (float)((double)xc[(size_t)i * d + k] + (double)f[(size_t)i * d + k]);
}
