/*
 * pq_oracle.c -- plain CPU oracle for the quantized linear layer (W8A8 / W4A8).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the quantized linear layer computes, written from the paper's equations.  It
 * shares no code, header, table or constant with the CUDA library; only tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  The product path
 * never routes through it.
 *
 * What it follows:
 *   - Eq. 1 (integer code = round(X / s)) and Eq. 2 (s = 2*max|X| / (2^n - 1),
 *     clamp to [-2^(n-1), 2^(n-1)-1], round-to-nearest) of the paper's
 *     "Preliminary" section, with n = 8 for activations and W8 weights and n = 4
 *     for W4 weights.
 *   - The granularities named in the same section: one scale per token for
 *     activations, one per output channel for W8 weights, one per fixed-size
 *     group along K for W4 weights.
 *   - Symmetric quantization (no zero point), as the experimental set-up states.
 *   - The "Unified low-bit inference framework" section: integer matrix product of
 *     the codes followed by dequantization back to FP16.
 *   - Eq. 3 (SmoothQuant variant of the W4A8 configurations): Y = (X S^-1)(S W) with
 *     S = diag(s), s_j = max|X_j|^alpha / max|W_j|^(1-alpha), alpha = 0.5.  The column
 *     factors enter the quantizers as an optional per-k multiplier applied in binary32
 *     BEFORE the absolute maximum is taken (the *_smooth entry points).
 *   - Eq. 4 (Hadamard variant): Y = (X H)(H^T W) with H a normalized Hadamard matrix.  With W
 *     stored [N,K] both sides are rotated along K: rows of X and rows of W are multiplied by H
 *     (the *_hadamard entry points), so that (X H)(W H)^T = X W^T.
 *
 * Readings taken where the paper is silent (also listed in the design notes):
 *   - ties in the rounding go to even;
 *   - the quotient X/s of Eq. 1 is evaluated in IEEE binary32 as X * (c / max|X|)
 *     for activations (c = (2^n-1)/2), and as a binary32 division X / s for the
 *     offline weight packers;
 *   - an all-zero row or group has scale 0 and codes 0;
 *   - W4 codes are chosen against the FP16-rounded group scale that is stored;
 *   - dequantization is evaluated in binary64 and rounded once to FP16;
 *   - Eq. 3 with alpha = 0.5 is evaluated literally as sqrtf(max|X_j|) / sqrtf(max|W_j|)
 *     (three correctly rounded binary32 operations), s^-1 as the binary32 quotient 1 / s;
 *     a channel whose activation or weight maximum is 0 gets s = 1;
 *   - the smoothed value X[m,k] * s^-1[k] (or W[n,k] * s[k]) is one binary32 product of the
 *     exact FP16 value and the factor; it is NOT rounded back to FP16;
 *   - Eq. 4 needs a Hadamard matrix of order K.  Where K is a power of two (up to 16384) that is the
 *     Sylvester matrix H_K itself.  For the other widths of the paper's layers (11008 = 2^8 * 43) no
 *     construction is at hand: H is taken block-diagonal, H = I (x) H_B / sqrt(B), with H_B the
 *     Sylvester matrix of order B = the largest power of two that divides K, at most 256.  It is
 *     applied as the textbook in-place butterfly (distances 1, 2, 4, ..., B/2 in this order, each
 *     step a' = a + b, b' = a - b in binary32), then one binary32 product with
 *     1 / sqrtf(B); the rotated values stay in binary32.
 *   - The decoder layer's MLP between the gate/up linears and the down linear (the paper quantizes
 *     "all linear layers" of such a decoder and times whole prefill passes, Table 3, but does not
 *     define the activation): the gated form SwiGLU, h = silu(gate) * up, silu(g) = g / (1 + e^-g).
 *     Its result is the down projection's input and is quantized per token by Eq. 1-2 directly
 *     (pqo_swiglu_quantize).  Because a binary32 value decides an integer code here, the
 *     evaluation is FIXED as a sequence of single binary32 operations (swiglu_f32 below): e^t by
 *     range reduction t = n ln2 + r with ln2 split in two parts, the degree-7 Taylor polynomial
 *     p of e^r in Horner form with fused multiply-adds; then d = fma(p, 2^n, 1) = 1 + e^t, the
 *     IEEE reciprocal 1 / d, the product g * (1 / d) and one product with `up`.  h stays in
 *     binary32.
 *
 * Arithmetic notes: integer dot products accumulate in int64 and are checked to
 * fit int32.  All binary32 steps are single IEEE operations (compile with
 * -ffp-contract=off, no fast-math).  FP16 is handled with the bit-level
 * conversions below; no hardware half type is used.
 *
 * Parity pins live in tests/test_oracle_pins.py (closed forms with power-of-two
 * scales, exact-rational cross-check, brute force, identity / one-hot weights,
 * error bound, overflow bound, exhaustive FP16 round trip).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PQO_OK 0
#define PQO_ERR_OVERFLOW 1 /* an integer accumulator left the int32 range */
#define PQO_ERR_ARG 2

/* ------------------------------------------------------------------ FP16 */

/* FP16 bit pattern -> binary32 value (exact). */
float pqo_half_to_float(uint16_t h) {
  int sign = (h >> 15) & 1;
  int e = (h >> 10) & 0x1f;
  int m = h & 0x3ff;
  double v;
  if (e == 0) {
    v = ldexp((double)m, -24); /* zero and subnormals: m * 2^-24 */
  } else if (e == 31) {
    v = m ? NAN : INFINITY;
  } else {
    v = ldexp((double)(1024 + m), e - 25); /* (1 + m/1024) * 2^(e-15) */
  }
  return (float)(sign ? -v : v);
}

/* binary64 value -> FP16 bit pattern, one rounding, round-to-nearest-even,
 * overflow to infinity, subnormals kept. */
uint16_t pqo_double_to_half_rne(double d) {
  uint16_t sign = signbit(d) ? 0x8000u : 0u;
  double a = fabs(d);
  if (isnan(d)) return (uint16_t)(sign | 0x7e00u);
  if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u); /* >= midpoint(65504, 65536) */
  if (a < ldexp(1.0, -14)) {
    /* subnormal range: spacing 2^-24 */
    double r = nearbyint(ldexp(a, 24)); /* 0 .. 1024; 1024 encodes the smallest normal */
    return (uint16_t)(sign | (uint16_t)r);
  }
  int e2;
  (void)frexp(a, &e2); /* a = f * 2^e2 with f in [0.5, 1) */
  int e = e2 - 1;      /* a in [2^e, 2^(e+1)) */
  double r = nearbyint(ldexp(a, 10 - e)); /* in [1024, 2048] */
  if (r >= 2048.0) {
    r = 1024.0;
    e += 1;
  }
  if (e > 15) return (uint16_t)(sign | 0x7c00u);
  return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | ((uint16_t)r - 1024u));
}

uint16_t pqo_float_to_half_rne(float f) { return pqo_double_to_half_rne((double)f); }

/* ------------------------------------------------------------ quantizers */

static float clampf(float v, float lo, float hi) { return v < lo ? lo : (v > hi ? hi : v); }

/*
 * Per-token activation quantization, Eq. 1-2 with n = 8.
 *   a = max_k |X[m,k]|;  s_tok[m] = a / 127.5  (= 2a / 255)
 *   Q[m,k] = clamp(rne(X[m,k] * (127.5 / a)), -128, 127)
 * x: FP16 bit patterns [M,K] row-major.  q: [M,K].  s_tok: [M].
 */
/* The value a quantizer sees: the FP16 element, times the column factor when there is one
 * (Eq. 3: X S^-1 on the activation side, S W on the weight side). */
static float smoothed(uint16_t h, const float* col, int64_t k) {
  float v = pqo_half_to_float(h);
  return col ? v * col[k] : v;
}

/* Eq. 4: order of the Hadamard blocks for a row of length K (see the readings above). */
int64_t pqo_hadamard_block(int64_t K) {
  if (K >= 1 && K <= 16384 && (K & (K - 1)) == 0) return K;   /* a power of two: H of the row's own order */
  int64_t B = 1;
  while (B < 256 && K % (2 * B) == 0) B *= 2;
  return B;
}

/* v[0..B) <- v H_B (Sylvester order; H_B is symmetric), unnormalized, in place. */
static void butterfly(float* v, int64_t B) {
  for (int64_t h = 1; h < B; h *= 2) {
    for (int64_t i = 0; i < B; i += 2 * h) {
      for (int64_t j = i; j < i + h; ++j) {
        float a = v[j], b = v[j + h];
        v[j] = a + b;
        v[j + h] = a - b;
      }
    }
  }
}

/* out[r,:] = A[r,:] H  for A FP16 [R,K], out binary32 [R,K]. */
int pqo_rotate_rows(const uint16_t* a, int64_t R, int64_t K, float* out) {
  if (R < 0 || K <= 0) return PQO_ERR_ARG;
  int64_t B = pqo_hadamard_block(K);
  float norm = 1.0f / sqrtf((float)B);
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r) {
    float* o = out + r * K;
    for (int64_t k = 0; k < K; ++k) o[k] = pqo_half_to_float(a[r * K + k]);
    for (int64_t k0 = 0; k0 < K; k0 += B) {
      butterfly(o + k0, B);
      for (int64_t k = k0; k < k0 + B; ++k) o[k] = o[k] * norm;
    }
  }
  return PQO_OK;
}

/* Eq. 1-2 per row on values that are already binary32 (the rotated rows of Eq. 4). */
static void quantize_row_f32(const float* t, int64_t K, int as_weight, int8_t* q, float* scale) {
  float a = 0.0f;
  for (int64_t k = 0; k < K; ++k) {
    float v = fabsf(t[k]);
    if (v > a) a = v;
  }
  if (a == 0.0f) {
    *scale = 0.0f;
    for (int64_t k = 0; k < K; ++k) q[k] = 0;
    return;
  }
  float s = a / 127.5f;
  float inv = 127.5f / a;
  *scale = s;
  for (int64_t k = 0; k < K; ++k) {
    float r = nearbyintf(as_weight ? t[k] / s : t[k] * inv);   /* the same two forms as the plain quantizers */
    float c = r < -128.0f ? -128.0f : (r > 127.0f ? 127.0f : r);
    q[k] = (int8_t)c;
  }
}

/* ---------------------------------------------------------------- SwiGLU + per-token quantization
 * silu(g) * u in binary32, as the fixed operation sequence named in the header.  g and u are
 * exact (FP16 values).  The argument of the exponential is clamped to [-87, 88], where e^t and
 * 2^n are normal binary32 numbers; beyond it silu is 0 or g to within 1e-33. */
static float one_plus_exp_f32(float t) {
  const float log2e = 0x1.715476p+0f;                       /* 1 / ln 2, rounded to binary32 */
  const float ln2_hi = 0x1.62e4p-1f, ln2_lo = 0x1.7f7d1cp-20f;   /* ln 2 = hi + lo, hi with 9 trailing zero bits */
  float n = nearbyintf(t * log2e);
  float r = fmaf(n, -ln2_hi, t);
  r = fmaf(n, -ln2_lo, r);
  float p = 0x1.a01a02p-13f;                                /* 1/7! */
  p = fmaf(p, r, 0x1.6c16c2p-10f);                          /* 1/6! */
  p = fmaf(p, r, 0x1.111112p-7f);                           /* 1/5! */
  p = fmaf(p, r, 0x1.555556p-5f);                           /* 1/4! */
  p = fmaf(p, r, 0x1.555556p-3f);                           /* 1/3! */
  p = fmaf(p, r, 0.5f);
  p = fmaf(p, r, 1.0f);
  p = fmaf(p, r, 1.0f);
  union { uint32_t u; float f; } two_n;
  two_n.u = (uint32_t)((int32_t)n + 127) << 23;             /* 2^n, n in [-126, 127] */
  return fmaf(p, two_n.f, 1.0f);                            /* 1 + e^t, one rounding */
}

static float swiglu_f32(float g, float u) {
  float t = -g;
  t = t < -87.0f ? -87.0f : (t > 88.0f ? 88.0f : t);
  float rcp = 1.0f / one_plus_exp_f32(t);
  float silu = g * rcp;
  return silu * u;
}

/* h[m,i] = silu(gate[m,i]) * up[m,i] in binary32 (out may be NULL), then Eq. 1-2 per token on h. */
int pqo_swiglu_quantize(const uint16_t* gate, const uint16_t* up, int64_t M, int64_t I, float* h_out, int8_t* q,
                        float* s_tok) {
  if (M < 0 || I <= 0) return PQO_ERR_ARG;
  int bad = 0;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    float* h = (float*)malloc((size_t)I * sizeof(float));
    if (!h) {
      bad = 1;
      continue;
    }
    for (int64_t i = 0; i < I; ++i)
      h[i] = swiglu_f32(pqo_half_to_float(gate[m * I + i]), pqo_half_to_float(up[m * I + i]));
    if (h_out) {
      for (int64_t i = 0; i < I; ++i) h_out[m * I + i] = h[i];
    }
    if (q && s_tok) quantize_row_f32(h, I, 0, q + m * I, s_tok + m);
    free(h);
  }
  return bad ? PQO_ERR_ARG : PQO_OK;
}

/* Eq. 4, activation side: per-token INT8 quantization of X H. */
int pqo_quantize_act_hadamard(const uint16_t* x, int64_t M, int64_t K, int8_t* q, float* s_tok) {
  if (M < 0 || K <= 0) return PQO_ERR_ARG;
  float* t = (float*)malloc((size_t)(M > 0 ? M : 1) * (size_t)K * sizeof(float));
  if (!t) return PQO_ERR_ARG;
  int rc = pqo_rotate_rows(x, M, K, t);
  if (rc == PQO_OK) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) quantize_row_f32(t + m * K, K, 0, q + m * K, s_tok + m);
  }
  free(t);
  return rc;
}

/* Eq. 4, weight side, W8: per-output-channel INT8 quantization of W H (rows of W rotated). */
int pqo_pack_w8_hadamard(const uint16_t* w, int64_t N, int64_t K, int8_t* wq, float* s_ch) {
  if (N < 0 || K <= 0) return PQO_ERR_ARG;
  float* t = (float*)malloc((size_t)(N > 0 ? N : 1) * (size_t)K * sizeof(float));
  if (!t) return PQO_ERR_ARG;
  int rc = pqo_rotate_rows(w, N, K, t);
  if (rc == PQO_OK) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) quantize_row_f32(t + n * K, K, 1, wq + n * K, s_ch + n);
  }
  free(t);
  return rc;
}

/* Eq. 4, weight side, W4: group-wise INT4 quantization of W H against the stored FP16 scale. */
int pqo_pack_w4_hadamard(const uint16_t* w, int64_t N, int64_t K, int64_t group, int8_t* codes,
                         uint16_t* s_grp) {
  if (N < 0 || K <= 0 || group <= 0 || K % group) return PQO_ERR_ARG;
  float* t = (float*)malloc((size_t)(N > 0 ? N : 1) * (size_t)K * sizeof(float));
  if (!t) return PQO_ERR_ARG;
  int rc = pqo_rotate_rows(w, N, K, t);
  int64_t G = K / group;
  if (rc == PQO_OK) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
      for (int64_t g = 0; g < G; ++g) {
        const float* tr = t + n * K + g * group;
        float a = 0.0f;
        for (int64_t k = 0; k < group; ++k) {
          float v = fabsf(tr[k]);
          if (v > a) a = v;
        }
        uint16_t s16 = pqo_float_to_half_rne(a / 7.5f);
        float sf = pqo_half_to_float(s16);
        s_grp[n * G + g] = s16;
        for (int64_t k = 0; k < group; ++k) {
          int8_t c = 0;
          if (sf != 0.0f) {
            float r = nearbyintf(tr[k] / sf);
            c = (int8_t)(r < -8.0f ? -8.0f : (r > 7.0f ? 7.0f : r));
          }
          codes[n * K + g * group + k] = c;
        }
      }
    }
  }
  free(t);
  return rc;
}

static int quantize_act_impl(const uint16_t* x, const float* col, int64_t M, int64_t K, int8_t* q,
                             float* s_tok) {
  if (M < 0 || K <= 0) return PQO_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    const uint16_t* xr = x + m * K;
    float a = 0.0f;
    for (int64_t k = 0; k < K; ++k) {
      float v = fabsf(smoothed(xr[k], col, k));
      if (v > a) a = v;
    }
    if (a == 0.0f) {
      s_tok[m] = 0.0f;
      for (int64_t k = 0; k < K; ++k) q[m * K + k] = 0;
      continue;
    }
    float s = a / 127.5f;
    float inv = 127.5f / a;
    s_tok[m] = s;
    for (int64_t k = 0; k < K; ++k) {
      float t = smoothed(xr[k], col, k) * inv;
      float r = nearbyintf(t); /* ties to even */
      q[m * K + k] = (int8_t)clampf(r, -128.0f, 127.0f);
    }
  }
  return PQO_OK;
}

int pqo_quantize_act(const uint16_t* x, int64_t M, int64_t K, int8_t* q, float* s_tok) {
  return quantize_act_impl(x, 0, M, K, q, s_tok);
}

/*
 * Static (calibrated) activation scale: Eq. 1 with a scale fixed ahead of time instead of the
 * token's own maximum (the paper's accuracy runs use "calibrated scales"); one scale for the whole
 * tensor.  code = clamp(rne(X * (1 / s)), -128, 127), 1 / s one binary32 division, the product one
 * binary32 multiplication; values beyond the calibrated range saturate.  s <= 0 gives codes 0.
 * s_tok[m] = s for every token, so that the GEMM calls are used unchanged.
 */
int pqo_quantize_act_static(const uint16_t* x, float s, int64_t M, int64_t K, int8_t* q, float* s_tok) {
  if (M < 0 || K <= 0) return PQO_ERR_ARG;
  float inv = s > 0.0f ? 1.0f / s : 0.0f;
  for (int64_t m = 0; m < M; ++m) {
    s_tok[m] = s > 0.0f ? s : 0.0f;
    for (int64_t k = 0; k < K; ++k) {
      float r = nearbyintf(pqo_half_to_float(x[m * K + k]) * inv);
      q[m * K + k] = (int8_t)clampf(r, -128.0f, 127.0f);
    }
  }
  return PQO_OK;
}

/*
 * Static activation scales with one scale per feature channel (the other granularity the paper's
 * "Preliminary" section names for calibrated scales): code = clamp(rne(X[m,k] * inv_s[k])), one
 * binary32 product with the reciprocal of channel k's calibrated scale (given by the caller; a
 * reciprocal that is not positive gives code 0).  A scale that depends on k cannot be taken out of
 * the sum over k, so it is the caller's to fold into the weights (W[n,k] * s[k], as Eq. 3 does):
 * the token scales are set to 1.
 */
int pqo_quantize_act_static_channel(const uint16_t* x, const float* inv_s, int64_t M, int64_t K, int8_t* q,
                                    float* s_tok) {
  if (M < 0 || K <= 0 || !inv_s) return PQO_ERR_ARG;
  for (int64_t m = 0; m < M; ++m) {
    s_tok[m] = 1.0f;
    for (int64_t k = 0; k < K; ++k) {
      float f = inv_s[k] > 0.0f ? inv_s[k] : 0.0f;
      float r = nearbyintf(pqo_half_to_float(x[m * K + k]) * f);
      q[m * K + k] = (int8_t)clampf(r, -128.0f, 127.0f);
    }
  }
  return PQO_OK;
}

/* Eq. 3, activation side: quantize X S^-1.  s_inv: [K] binary32. */
int pqo_quantize_act_smooth(const uint16_t* x, const float* s_inv, int64_t M, int64_t K, int8_t* q,
                            float* s_tok) {
  if (!s_inv) return PQO_ERR_ARG;
  return quantize_act_impl(x, s_inv, M, K, q, s_tok);
}

/*
 * Per-output-channel INT8 weight quantization, Eq. 2 with n = 8.
 *   a = max_k |W[n,k]|;  s_ch[n] = a / 127.5;  Wq = clamp(rne(W / s_ch[n]), -128, 127)
 * w: FP16 bit patterns [N,K] (one output channel per row).
 */
static int pack_w8_impl(const uint16_t* w, const float* col, int64_t N, int64_t K, int8_t* wq, float* s_ch) {
  if (N < 0 || K <= 0) return PQO_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    const uint16_t* wr = w + n * K;
    float a = 0.0f;
    for (int64_t k = 0; k < K; ++k) {
      float v = fabsf(smoothed(wr[k], col, k));
      if (v > a) a = v;
    }
    if (a == 0.0f) {
      s_ch[n] = 0.0f;
      for (int64_t k = 0; k < K; ++k) wq[n * K + k] = 0;
      continue;
    }
    float s = a / 127.5f;
    s_ch[n] = s;
    for (int64_t k = 0; k < K; ++k) {
      float r = nearbyintf(smoothed(wr[k], col, k) / s);
      wq[n * K + k] = (int8_t)clampf(r, -128.0f, 127.0f);
    }
  }
  return PQO_OK;
}

int pqo_pack_w8(const uint16_t* w, int64_t N, int64_t K, int8_t* wq, float* s_ch) {
  return pack_w8_impl(w, 0, N, K, wq, s_ch);
}

/* Eq. 3, weight side: quantize S W (W stored [N,K], so s multiplies along k).  s: [K] binary32. */
int pqo_pack_w8_smooth(const uint16_t* w, const float* s, int64_t N, int64_t K, int8_t* wq, float* s_ch) {
  if (!s) return PQO_ERR_ARG;
  return pack_w8_impl(w, s, N, K, wq, s_ch);
}

/*
 * Group-wise INT4 weight quantization, Eq. 2 with n = 4, one scale per
 * (output channel, group of `group` consecutive k).
 *   a = max_{k in g} |W[n,k]|;  s_grp[n,g] = fp16(a / 7.5)
 *   code = clamp(rne(W / float(s_grp[n,g])), -8, 7)      (against the stored scale)
 * codes: int8 [N,K] holding values in [-8,7].  s_grp: FP16 bit patterns [N, K/group].
 */
static int pack_w4_impl(const uint16_t* w, const float* col, int64_t N, int64_t K, int64_t group, int8_t* codes,
                        uint16_t* s_grp) {
  if (N < 0 || K <= 0 || group <= 0 || K % group) return PQO_ERR_ARG;
  int64_t G = K / group;
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n) {
    for (int64_t g = 0; g < G; ++g) {
      const uint16_t* wr = w + n * K + g * group;
      float a = 0.0f;
      for (int64_t k = 0; k < group; ++k) {
        float v = fabsf(smoothed(wr[k], col, g * group + k));
        if (v > a) a = v;
      }
      uint16_t s16 = pqo_float_to_half_rne(a / 7.5f);
      float sf = pqo_half_to_float(s16);
      s_grp[n * G + g] = s16;
      for (int64_t k = 0; k < group; ++k) {
        int8_t c = 0;
        if (sf != 0.0f) {
          float r = nearbyintf(smoothed(wr[k], col, g * group + k) / sf);
          c = (int8_t)clampf(r, -8.0f, 7.0f);
        }
        codes[n * K + g * group + k] = c;
      }
    }
  }
  return PQO_OK;
}

int pqo_pack_w4(const uint16_t* w, int64_t N, int64_t K, int64_t group, int8_t* codes,
                uint16_t* s_grp) {
  return pack_w4_impl(w, 0, N, K, group, codes, s_grp);
}

int pqo_pack_w4_smooth(const uint16_t* w, const float* s, int64_t N, int64_t K, int64_t group, int8_t* codes,
                       uint16_t* s_grp) {
  if (!s) return PQO_ERR_ARG;
  return pack_w4_impl(w, s, N, K, group, codes, s_grp);
}

/* Calibration statistic of Eq. 3: max over rows of |A[r,k]| for every column k.  a: FP16 [R,K]. */
int pqo_col_absmax(const uint16_t* a, int64_t R, int64_t K, float* out) {
  if (R < 0 || K <= 0) return PQO_ERR_ARG;
  for (int64_t k = 0; k < K; ++k) out[k] = 0.0f;
  for (int64_t r = 0; r < R; ++r) {
    for (int64_t k = 0; k < K; ++k) {
      float v = fabsf(pqo_half_to_float(a[r * K + k]));
      if (v > out[k]) out[k] = v;
    }
  }
  return PQO_OK;
}

/* Eq. 3 with alpha = 0.5:  s_j = max|X_j|^(1/2) / max|W_j|^(1/2),  s_inv_j = 1 / s_j.
 * x_absmax, w_absmax: [K] column maxima (pqo_col_absmax of the calibration activations and of W). */
int pqo_smooth_scales(const float* x_absmax, const float* w_absmax, int64_t K, float* s, float* s_inv) {
  if (K <= 0) return PQO_ERR_ARG;
  for (int64_t k = 0; k < K; ++k) {
    if (!(x_absmax[k] > 0.0f) || !(w_absmax[k] > 0.0f)) {
      s[k] = 1.0f;
      s_inv[k] = 1.0f;
      continue;
    }
    float num = sqrtf(x_absmax[k]);
    float den = sqrtf(w_absmax[k]);
    s[k] = num / den;
    s_inv[k] = 1.0f / s[k];
  }
  return PQO_OK;
}

/* Eq. 3 with the migration strength alpha a multiple of 1/4 (alpha = a / 4, a = 0 ... 4):
 *   s_j = max|X_j|^alpha / max|W_j|^(1 - alpha),
 * with the quarter powers written as square roots so that every step is a correctly rounded binary32
 * operation: x^(1/4) = sqrtf(sqrtf(x)), x^(1/2) = sqrtf(x), x^(3/4) = sqrtf(x) * sqrtf(sqrtf(x)) (one
 * rounded product), x^0 = 1, x^1 = x; then one division, and s_inv = 1 / s.  a = 2 is pqo_smooth_scales. */
static float quarter_power(float x, int a) {
  switch (a) {
    case 0: return 1.0f;
    case 1: return sqrtf(sqrtf(x));
    case 2: return sqrtf(x);
    case 3: return sqrtf(x) * sqrtf(sqrtf(x));
    default: return x;
  }
}

int pqo_smooth_scales_alpha(const float* x_absmax, const float* w_absmax, int64_t K, int alpha_quarters, float* s,
                            float* s_inv) {
  if (K <= 0 || alpha_quarters < 0 || alpha_quarters > 4) return PQO_ERR_ARG;
  for (int64_t k = 0; k < K; ++k) {
    if (!(x_absmax[k] > 0.0f) || !(w_absmax[k] > 0.0f)) {
      s[k] = 1.0f;
      s_inv[k] = 1.0f;
      continue;
    }
    float num = quarter_power(x_absmax[k], alpha_quarters);
    float den = quarter_power(w_absmax[k], 4 - alpha_quarters);
    s[k] = num / den;
    s_inv[k] = 1.0f / s[k];
  }
  return PQO_OK;
}

/* Interchange form of INT4 codes: byte j of a row holds k = 2j in bits 0-3 and
 * k = 2j+1 in bits 4-7, two's complement. */
int pqo_nibble_pack(const int8_t* codes, int64_t N, int64_t K, uint8_t* bytes) {
  if (K % 2) return PQO_ERR_ARG;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t j = 0; j < K / 2; ++j) {
      uint8_t lo = (uint8_t)codes[n * K + 2 * j] & 0xf;
      uint8_t hi = (uint8_t)codes[n * K + 2 * j + 1] & 0xf;
      bytes[n * (K / 2) + j] = (uint8_t)(lo | (hi << 4));
    }
  return PQO_OK;
}

int pqo_nibble_unpack(const uint8_t* bytes, int64_t N, int64_t K, int8_t* codes) {
  if (K % 2) return PQO_ERR_ARG;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t j = 0; j < K / 2; ++j) {
      uint8_t b = bytes[n * (K / 2) + j];
      int lo = b & 0xf, hi = b >> 4;
      codes[n * K + 2 * j] = (int8_t)(lo >= 8 ? lo - 16 : lo);
      codes[n * K + 2 * j + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
  return PQO_OK;
}

/* ------------------------------------------------------------------ GEMMs */

/*
 * W8A8 linear: ACC[m,n] = sum_k Q[m,k] * Wq[n,k] (exact integer),
 *              Y[m,n]  = fp16( ACC[m,n] * s_tok[m] * s_ch[n] ).
 * acc (int32 [M,N]) and y (FP16 bits [M,N]) may each be NULL to skip that output.
 */
int pqo_gemm_w8a8(const int8_t* q, const float* s_tok, const int8_t* wq, const float* s_ch,
                  int64_t M, int64_t N, int64_t K, int32_t* acc, uint16_t* y) {
  if (M < 0 || N < 0 || K <= 0) return PQO_ERR_ARG;
  int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
  for (int64_t m = 0; m < M; ++m) {
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t k = 0; k < K; ++k) s += (int64_t)q[m * K + k] * (int64_t)wq[n * K + k];
      if (s > INT32_MAX || s < INT32_MIN) overflow |= 1;
      if (acc) acc[m * N + n] = (int32_t)s;
      if (y) {
        double v = (double)s * (double)s_tok[m] * (double)s_ch[n];
        y[m * N + n] = pqo_double_to_half_rne(v);
      }
    }
  }
  return overflow ? PQO_ERR_OVERFLOW : PQO_OK;
}

/*
 * W4A8 linear with per-group dequantization:
 *   ACC_g[m,n] = sum_{k in group g} Q[m,k] * C[n,k]          (exact integer)
 *   R[m,n]     = sum_g ACC_g[m,n] * float(s_grp[n,g])        (g ascending)
 *   Y[m,n]     = fp16( R[m,n] * s_tok[m] )
 * codes: int8 [N,K] with values in [-8,7].  acc_g (int32 [M,N,G]) and y may be NULL.
 */
int pqo_gemm_w4a8(const int8_t* q, const float* s_tok, const int8_t* codes,
                  const uint16_t* s_grp, int64_t group, int64_t M, int64_t N, int64_t K,
                  int32_t* acc_g, uint16_t* y) {
  if (M < 0 || N < 0 || K <= 0 || group <= 0 || K % group) return PQO_ERR_ARG;
  int64_t G = K / group;
  int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
  for (int64_t m = 0; m < M; ++m) {
    for (int64_t n = 0; n < N; ++n) {
      double R = 0.0;
      for (int64_t g = 0; g < G; ++g) {
        int64_t s = 0;
        for (int64_t k = g * group; k < (g + 1) * group; ++k)
          s += (int64_t)q[m * K + k] * (int64_t)codes[n * K + k];
        if (s > INT32_MAX || s < INT32_MIN) overflow |= 1;
        if (acc_g) acc_g[(m * N + n) * G + g] = (int32_t)s;
        R += (double)s * (double)pqo_half_to_float(s_grp[n * G + g]);
      }
      if (y) y[m * N + n] = pqo_double_to_half_rne(R * (double)s_tok[m]);
    }
  }
  return overflow ? PQO_ERR_OVERFLOW : PQO_OK;
}

int pqo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
