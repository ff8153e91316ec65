/*
 * CPU oracle for the expanded W4A4 linear layer (post-training model expansion).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64/int64 statement of what the
 * method computes, written from the paper.  It shares no code, header, table or helper with
 * the CUDA library and is never on the product path: only the tests, the smoke check and the
 * CPU-baseline leg of the benchmark may call it.
 *
 * Notation (paper Sec. 3 -> here): the paper's inputs X are D x N, weights W are N x N' and
 * the expanded order is M.  Here tokens are M, input channels K, expanded channels Kp (K'),
 * output channels N, and weights are stored out x in (row n of W is output channel n), so both
 * operands receive the same map  v -> [v, 0] * H / sqrt(Kp).
 *
 * Parity pins (tests/test_oracle_*.py): H H^T = Kp I with entries +-1 (Sec. 3), the Sylvester
 * case against a library Walsh-Hadamard matrix, truncated-column norms sqrt(K/Kp) (Remark 2),
 * energy and rank preservation (Remarks 1-2), the rotation invariance X W = X_hat W_hat
 * (Sec. 3), quantizer bounds and ties, brute-force / closed-form integer products, bf16
 * rounding against a library conversion; for the asymmetric activation quantizer: code range and
 * end points, |y - s (u - z)| <= s / 2, exactness on an integer grid, and the identity
 * s_x s_w (acc - z wsum) = sum_c [s_x (u - z)] [s_w qw] against a floating-point product.
 * Parity unpinned: xqo_ref_product's use as a quality axis (the paper prints no error figure
 * for round-to-nearest weights on synthetic data); the function itself is a plain product.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ----------------------------------------------------------------------------------------- */
/* Hadamard plan: Kp = p * 2^k, H = H_p (x) S_{2^k}.  The paper only asks for "an expanded
 * M x M Hadamard matrix" (Sec. 3); the construction is a reading: Paley-I / Paley-II for the
 * non-power-of-two factor, Sylvester for the power of two.                                   */

typedef struct {
  int32_t K, Kp, p, log2n, paley_kind, q; /* paley_kind: 0 none (p == 1), 1 Paley-I, 2 Paley-II, 3 Paley-I over GF(7^3) */
} xqo_plan_t;

static int is_prime(int v) {
  if (v < 2) return 0;
  for (int d = 2; (long)d * d <= v; ++d)
    if (v % d == 0) return 0;
  return 1;
}

/* Legendre symbol chi(a) mod prime q: 0 for a == 0, +1 for a non-zero square, -1 otherwise,
 * by Euler's criterion a^((q-1)/2) mod q. */
static int legendre(int a, int q) {
  a %= q;
  if (a < 0) a += q;
  if (a == 0) return 0;
  long r = 1, b = a;
  int e = (q - 1) / 2;
  while (e) {
    if (e & 1) r = (r * b) % q;
    b = (b * b) % q;
    e >>= 1;
  }
  return r == 1 ? 1 : -1;
}

/* The field with 343 = 7^3 elements, for the one prime-power order the paper's sizes need (Table 1: 22016 = 344 * 64,
 * and 344 - 1 = 7^3 = 3 mod 4, so Paley's first construction applies over GF(7^3)).  Elements are the polynomials
 * a0 + a1 x + a2 x^2 over GF(7) modulo x^3 - 5 (irreducible: 5 is not a cube mod 7, the cubes being 0, 1, 6), numbered
 * a0 + 7 a1 + 49 a2. */
static int gf343_sub(int a, int b) {
  int r = 0, w = 1;
  for (int k = 0; k < 3; ++k, w *= 7) {
    int d = (a / w) % 7 - (b / w) % 7;
    if (d < 0) d += 7;
    r += d * w;
  }
  return r;
}
static int gf343_mul(int a, int b) {
  int x[3] = {a % 7, (a / 7) % 7, a / 49}, y[3] = {b % 7, (b / 7) % 7, b / 49}, c[5] = {0, 0, 0, 0, 0};
  for (int i = 0; i < 3; ++i)
    for (int j = 0; j < 3; ++j) c[i + j] += x[i] * y[j];
  /* x^3 = 5, x^4 = 5 x */
  c[0] += 5 * c[3];
  c[1] += 5 * c[4];
  return c[0] % 7 + 7 * (c[1] % 7) + 49 * (c[2] % 7);
}
/* Quadratic character of GF(343): 0 for 0, +1 for a non-zero square, -1 otherwise, by Euler's criterion
 * a^((343-1)/2). */
static int gf343_chi(int a) {
  if (a == 0) return 0;
  int r = 1, b = a, e = 171;
  while (e) {
    if (e & 1) r = gf343_mul(r, b);
    b = gf343_mul(b, b);
    e >>= 1;
  }
  return r == 1 ? 1 : -1;
}

/* Smallest p = odd(Kp) * 2^j, j >= 2, for which a Paley matrix of order p exists over a prime
 * field or over GF(7^3); p = 1 when Kp is a power of two.  Returns 0 on success, 1 on bad arguments, 2 when no
 * such order divides Kp. */
int xqo_plan(int32_t K, int32_t Kp, xqo_plan_t *out) {
  if (!out || K < 1 || Kp < K) return 1;
  int odd = Kp, e = 0;
  while ((odd & 1) == 0) {
    odd >>= 1;
    ++e;
  }
  out->K = K;
  out->Kp = Kp;
  if (odd == 1) {
    out->p = 1;
    out->log2n = e;
    out->paley_kind = 0;
    out->q = 0;
    return 0;
  }
  for (int j = 2; j <= e; ++j) {
    int p = odd << j;
    if (is_prime(p - 1) && (p - 1) % 4 == 3) {
      out->p = p; out->log2n = e - j; out->paley_kind = 1; out->q = p - 1;
      return 0;
    }
    if (is_prime(p / 2 - 1) && (p / 2 - 1) % 4 == 1) {
      out->p = p; out->log2n = e - j; out->paley_kind = 2; out->q = p / 2 - 1;
      return 0;
    }
    if (p - 1 == 343) {
      out->p = p; out->log2n = e - j; out->paley_kind = 3; out->q = 343;
      return 0;
    }
  }
  return 2;
}

/* Entry (r, c) of the order-p factor, +-1. */
static int hp_entry(const xqo_plan_t *pl, int r, int c) {
  const int q = pl->q;
  if (pl->paley_kind == 0) return 1;
  if (pl->paley_kind == 1) {
    /* Paley-I, q = 3 mod 4: border row of +1, border column of -1 below it, core Q + I with
     * Q[i][j] = chi(i - j) the Jacobsthal matrix (skew for these q). */
    if (r == 0) return 1;
    if (c == 0) return -1;
    int i = r - 1, j = c - 1;
    return i == j ? 1 : legendre(i - j, q);
  }
  if (pl->paley_kind == 3) {
    /* the same construction over GF(7^3): rows and columns 1..343 stand for the field elements in their numbering,
     * Q[i][j] = chi(e_i - e_j) */
    if (r == 0) return 1;
    if (c == 0) return -1;
    int i = r - 1, j = c - 1;
    return i == j ? 1 : gf343_chi(gf343_sub(i, j));
  }
  /* Paley-II, q = 1 mod 4: symmetric S of order q + 1 with zero diagonal (S[0][j] = S[j][0] = 1,
   * core Q); every entry of S becomes a 2 x 2 block:  s * [[1,1],[1,-1]]  off the diagonal,
   * [[1,-1],[-1,-1]] on it. */
  int i = r >> 1, u = r & 1, j = c >> 1, v = c & 1;
  if (i == j) return (u == 0 && v == 0) ? 1 : -1;
  int s;
  if (i == 0 || j == 0) s = 1;
  else s = legendre((i - 1) - (j - 1), q);
  return (u == 1 && v == 1) ? -s : s;
}

/* Entry (c, c2) of the full order-Kp matrix.  Channel c = a * 2^k + b: the order-p factor is
 * the outer Kronecker factor, the Sylvester factor S[b][b2] = (-1)^popcount(b & b2) the inner. */
int xqo_hadamard_entry(const xqo_plan_t *pl, int32_t c, int32_t c2) {
  int n = 1 << pl->log2n;
  int a = c / n, b = c % n, a2 = c2 / n, b2 = c2 % n;
  int s = (__builtin_popcount((unsigned)(b & b2)) & 1) ? -1 : 1;
  return s * hp_entry(pl, a, a2);
}

/* Dense rows [0, rows) of H as int8 (+-1), row-major with Kp columns. */
void xqo_hadamard_dense(const xqo_plan_t *pl, int32_t rows, int8_t *out) {
#pragma omp parallel for schedule(static)
  for (int c = 0; c < rows; ++c)
    for (int c2 = 0; c2 < pl->Kp; ++c2)
      out[(size_t)c * pl->Kp + c2] = (int8_t)xqo_hadamard_entry(pl, c, c2);
}

/* ----------------------------------------------------------------------------------------- */
/* bf16 <-> double.  A bf16 is the upper half of an IEEE binary32. */

static double bf16_to_double(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* Round a double to the nearest bf16 (ties to even), directly, without passing through a
 * binary32 rounding first.  bf16: 8 significand bits including the hidden one, binary32's
 * exponent range (normals from 2^-126, subnormal quantum 2^-133). */
static uint16_t double_to_bf16(double v) {
  if (isnan(v)) return 0x7FC0;
  uint16_t sign = signbit(v) ? 0x8000 : 0;
  double a = fabs(v);
  if (a == 0.0) return sign;
  if (isinf(a)) return sign | 0x7F80;
  int e;
  (void)frexp(a, &e);           /* a = m * 2^e, m in [0.5, 1) */
  int qe = e - 8;               /* quantum exponent for 8 significant bits */
  if (qe < -133) qe = -133;     /* subnormal range */
  double r = nearbyint(ldexp(a, -qe)); /* default rounding mode: ties to even */
  double y = ldexp(r, qe);
  if (y >= ldexp(1.0, 128)) return sign | 0x7F80; /* overflow to infinity */
  float f = (float)y;           /* exact: y has at most 8 significant bits */
  uint32_t u;
  memcpy(&u, &f, 4);
  return sign | (uint16_t)(u >> 16);
}

void xqo_bf16_to_f64(const uint16_t *in, int64_t n, double *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_double(in[i]);
}
void xqo_f64_to_bf16(const double *in, int64_t n, uint16_t *out) {
  for (int64_t i = 0; i < n; ++i) out[i] = double_to_bf16(in[i]);
}

/* ----------------------------------------------------------------------------------------- */
/* Rotation (Sec. 3):  y[r][c2] = (1/sqrt(Kp)) * sum_{c < K} x[r][c] * H[c][c2].
 * Only the first K rows of H take part -- that is the truncated N x M matrix of the paper.   */

/* The definition, O(K * Kp) per row. */
void xqo_rotate_dense(const xqo_plan_t *pl, const uint16_t *x_bf16, int64_t rows, int64_t ldx,
                      double *y) {
  const int K = pl->K, Kp = pl->Kp;
  const double gamma = 1.0 / sqrt((double)Kp);
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t r = 0; r < rows; ++r) {
    double *yr = y + r * Kp;
    for (int c2 = 0; c2 < Kp; ++c2) {
      double acc = 0.0;
      for (int c = 0; c < K; ++c)
        acc += bf16_to_double(x_bf16[r * ldx + c]) * (double)xqo_hadamard_entry(pl, c, c2);
      yr[c2] = acc * gamma;
    }
  }
}

/* The same map through the Kronecker structure: view the padded row as a p x 2^k matrix V
 * (V[a][b] = x[a 2^k + b]); then Y = H_p^T V S.  Used for the large shapes; the tests hold it
 * to the dense definition. */
void xqo_rotate_factored(const xqo_plan_t *pl, const uint16_t *x_bf16, int64_t rows, int64_t ldx,
                         double *y) {
  const int K = pl->K, Kp = pl->Kp, p = pl->p, n = 1 << pl->log2n;
  const double gamma = 1.0 / sqrt((double)Kp);
  int8_t *hp = (int8_t *)malloc((size_t)p * p);
  for (int a = 0; a < p; ++a)
    for (int a2 = 0; a2 < p; ++a2) hp[a * p + a2] = (int8_t)hp_entry(pl, a, a2);
#pragma omp parallel
  {
    double *v = (double *)malloc(sizeof(double) * (size_t)Kp);
    double *t = (double *)malloc(sizeof(double) * (size_t)Kp);
#pragma omp for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
      for (int c = 0; c < Kp; ++c) v[c] = c < K ? bf16_to_double(x_bf16[r * ldx + c]) : 0.0;
      /* outer factor: t[a2][b] = sum_a H_p[a][a2] v[a][b] */
      for (int a2 = 0; a2 < p; ++a2)
        for (int b = 0; b < n; ++b) {
          double acc = 0.0;
          for (int a = 0; a < p; ++a) acc += (double)hp[a * p + a2] * v[a * n + b];
          t[a2 * n + b] = acc;
        }
      /* inner factor: unnormalised Walsh-Hadamard butterflies along b */
      for (int a2 = 0; a2 < p; ++a2) {
        double *row = t + (size_t)a2 * n;
        for (int h = 1; h < n; h <<= 1)
          for (int i = 0; i < n; i += 2 * h)
            for (int j = i; j < i + h; ++j) {
              double u = row[j], w = row[j + h];
              row[j] = u + w;
              row[j + h] = u - w;
            }
      }
      for (int c = 0; c < Kp; ++c) y[r * Kp + c] = t[c] * gamma;
    }
    free(v);
    free(t);
  }
  free(hp);
}

/* ----------------------------------------------------------------------------------------- */
/* Quantizer Q (Sec. 4, "Quantization Details": per-channel symmetric weights, per-token
 * activations, 4 bits).  Reading used here for both operands: symmetric, scale = absmax / 7,
 * round half to even, clamp to [-8, 7]; an all-zero row takes scale 1.  The scale crosses the
 * library boundary as binary32, so it is rounded to binary32 first and the rounded value is
 * the one that divides. */
void xqo_quantize(const double *y, int64_t rows, int64_t cols, int8_t *codes, float *scales) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    const double *yr = y + r * cols;
    double amax = 0.0;
    for (int64_t c = 0; c < cols; ++c) {
      double a = fabs(yr[c]);
      if (a > amax) amax = a;
    }
    float s32 = amax > 0.0 ? (float)(amax / 7.0) : 1.0f;
    if (!(s32 > 0.0f)) s32 = 1.0f; /* absmax so small that absmax/7 is not a positive binary32 */
    double s = (double)s32;
    scales[r] = s32;
    for (int64_t c = 0; c < cols; ++c) {
      double q = nearbyint(yr[c] / s);
      if (q > 7.0) q = 7.0;
      if (q < -8.0) q = -8.0;
      codes[r * cols + c] = (int8_t)q;
    }
  }
}

/* Asymmetric variant of the activation quantizer (Sec. 4, "Quantization Details": the paper's
 * activations are per-token asymmetric 4-bit).  The paper gives no formula; the reading used here
 * is the usual min/max affine quantizer with the range forced to contain zero:
 *   lo = min(0, min_c y_c), hi = max(0, max_c y_c), s = (hi - lo) / 15 (s = 1 for an all-zero row),
 *   z = round_half_even(-lo / s) clamped to [0, 15], u_c = clamp(round_half_even(y_c / s) + z, 0, 15),
 * and the value a code stands for is s * (u - z).  As in the symmetric case the scale is rounded
 * to binary32 first (it crosses the library boundary as binary32) and the rounded value divides. */
void xqo_quantize_asym(const double *y, int64_t rows, int64_t cols, uint8_t *codes, float *scales,
                       int32_t *zero_points) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    const double *yr = y + r * cols;
    double lo = 0.0, hi = 0.0;
    for (int64_t c = 0; c < cols; ++c) {
      if (yr[c] < lo) lo = yr[c];
      if (yr[c] > hi) hi = yr[c];
    }
    float s32 = hi > lo ? (float)((hi - lo) / 15.0) : 1.0f;
    if (!(s32 > 0.0f)) s32 = 1.0f;
    double s = (double)s32;
    double z = nearbyint(-lo / s);
    if (z < 0.0) z = 0.0;
    if (z > 15.0) z = 15.0;
    scales[r] = s32;
    zero_points[r] = (int32_t)z;
    for (int64_t c = 0; c < cols; ++c) {
      double q = nearbyint(yr[c] / s) + z;
      if (q > 15.0) q = 15.0;
      if (q < 0.0) q = 0.0;
      codes[r * cols + c] = (uint8_t)q;
    }
  }
}

/* Quantized product with unsigned activation codes and signed weight codes, exact. */
void xqo_gemm_u_i64(const uint8_t *ux, const int8_t *qw, int64_t M, int64_t N, int64_t Kp,
                    int64_t *acc) {
#pragma omp parallel for schedule(static) collapse(2)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t c = 0; c < Kp; ++c) s += (int64_t)ux[m * Kp + c] * (int64_t)qw[n * Kp + c];
      acc[m * N + n] = s;
    }
}

/* Dequantizing epilogue of the asymmetric variant:
 *   sum_c s_x (u - z) * s_w qw = s_x s_w (acc - z * sum_c qw[n][c]),
 * the row sums of the weight codes computed here; one rounding to bf16. */
void xqo_epilogue_asym(const int64_t *acc, const float *s_x, const int32_t *zp, const float *s_w,
                       const int8_t *qw, int64_t M, int64_t N, int64_t Kp, uint16_t *out_bf16) {
  int64_t *wsum = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
  for (int64_t n = 0; n < N; ++n) {
    int64_t t = 0;
    for (int64_t c = 0; c < Kp; ++c) t += qw[n * Kp + c];
    wsum[n] = t;
  }
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n)
      out_bf16[m * N + n] = double_to_bf16((double)(acc[m * N + n] - (int64_t)zp[m] * wsum[n]) *
                                           (double)s_x[m] * (double)s_w[n]);
  free(wsum);
}

/* Two's-complement nibbles, two per byte: byte j of a row holds code 2j in bits 0-3 and code
 * 2j+1 in bits 4-7 (the layout at the rotate_quant -> gemm seam; the paper fixes none). */
void xqo_pack_int4(const int8_t *codes, int64_t rows, int64_t cols, uint8_t *packed) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t j = 0; j < cols / 2; ++j) {
      uint8_t lo = (uint8_t)codes[r * cols + 2 * j] & 0xF;
      uint8_t hi = (uint8_t)codes[r * cols + 2 * j + 1] & 0xF;
      packed[r * (cols / 2) + j] = (uint8_t)(lo | (hi << 4));
    }
}

void xqo_unpack_int4(const uint8_t *packed, int64_t rows, int64_t cols, int8_t *codes) {
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t j = 0; j < cols / 2; ++j) {
      uint8_t b = packed[r * (cols / 2) + j];
      int lo = b & 0xF, hi = b >> 4;
      codes[r * cols + 2 * j] = (int8_t)(lo >= 8 ? lo - 16 : lo);
      codes[r * cols + 2 * j + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
}

/* ----------------------------------------------------------------------------------------- */
/* Quantized product Q(XR) Q(W~) (Sec. 3):  acc[m][n] = sum_c qx[m][c] * qw[n][c], exact.     */
void xqo_gemm_i64(const int8_t *qx, const int8_t *qw, int64_t M, int64_t N, int64_t Kp,
                  int64_t *acc) {
#pragma omp parallel for schedule(static) collapse(2)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      int64_t s = 0;
      for (int64_t c = 0; c < Kp; ++c) s += (int64_t)qx[m * Kp + c] * (int64_t)qw[n * Kp + c];
      acc[m * N + n] = s;
    }
}

/* Dequantizing epilogue: out[m][n] = bf16( acc * s_x[m] * s_w[n] ), one rounding. */
void xqo_epilogue(const int64_t *acc, const float *s_x, const float *s_w, int64_t M, int64_t N,
                  uint16_t *out_bf16) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n)
      out_bf16[m * N + n] =
          double_to_bf16((double)acc[m * N + n] * (double)s_x[m] * (double)s_w[n]);
}

/* Unquantized product of the bf16 inputs in fp64: ref[m][n] = sum_{c<K} x[m][c] W[n][c]. */
void xqo_ref_product(const uint16_t *x_bf16, const uint16_t *w_bf16, int64_t M, int64_t N,
                     int64_t K, double *ref) {
#pragma omp parallel for schedule(static) collapse(2)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double s = 0.0;
      for (int64_t c = 0; c < K; ++c)
        s += bf16_to_double(x_bf16[m * K + c]) * bf16_to_double(w_bf16[n * K + c]);
      ref[m * N + n] = s;
    }
}

int xqo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------------------------------------
 * MXFP4 (Sec. 4 "Quantization Details": the OCP microscaling format, one E8M0 scale for each group
 * of 32 elements, 4-bit E2M1 elements; the conversion rule is the OCP specification's).
 *
 * E2M1 code: bit 3 sign, bits 2-1 exponent, bit 0 mantissa; magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6.
 * Group of 32 consecutive channels with largest magnitude a > 0:
 *   shared exponent e = floor(log2(a)) - 2  (2 is the exponent of the largest E2M1 value, 6 = 1.5 * 2^2),
 *   clamped to [-127, 127]; scale byte = e + 127; element = nearest E2M1 value to v / 2^e, ties to the
 *   value with an even mantissa bit, magnitudes above 6 saturate to 6.
 * A group of zeros takes e = 0 (the specification leaves it open) and all-zero codes.
 * --------------------------------------------------------------------------------------------- */
static const double kE2M1[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

static uint8_t e2m1_encode(double v) {
  const uint8_t sign = (uint8_t)(v < 0.0 ? 8 : 0);
  const double a = fabs(v);
  int best = 7;
  if (a < 6.0) {
    /* between neighbours lo = kE2M1[i], hi = kE2M1[i + 1]: nearest, tie to the even code */
    for (int i = 0; i < 7; ++i) {
      if (a >= kE2M1[i] && a <= kE2M1[i + 1]) {
        const double dl = a - kE2M1[i], dh = kE2M1[i + 1] - a;
        best = dl < dh ? i : (dh < dl ? i + 1 : ((i & 1) ? i + 1 : i));
        break;
      }
    }
  }
  return (uint8_t)(sign | best);
}

double xqo_e2m1_value(uint8_t code) { return (code & 8) ? -kE2M1[code & 7] : kE2M1[code & 7]; }

void xqo_quantize_mx(const double *y, int64_t rows, int64_t cols, uint8_t *codes, uint8_t *scales) {
  const int64_t groups = cols / 32;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t g = 0; g < groups; ++g) {
      const double *v = y + r * cols + g * 32;
      double a = 0.0;
      for (int i = 0; i < 32; ++i)
        if (fabs(v[i]) > a) a = fabs(v[i]);
      int e = 0;
      if (a > 0.0) {
        int ex;
        (void)frexp(a, &ex); /* a = f * 2^ex, f in [0.5, 1): floor(log2 a) = ex - 1 */
        e = ex - 1 - 2;
        if (e < -127) e = -127;
        if (e > 127) e = 127;
      }
      scales[r * groups + g] = (uint8_t)(e + 127);
      const double inv = ldexp(1.0, -e);
      for (int i = 0; i < 32; ++i) codes[r * cols + g * 32 + i] = e2m1_encode(v[i] * inv);
    }
}

/* Product of two MXFP4 matrices in fp64 (every term is exact in binary64; the sum is rounded only by
 * fp64 addition): ref[m][n] = sum_g 2^(ex[m][g] + ew[n][g]) sum_{c in g} vx[m][c] vw[n][c]. */
void xqo_gemm_mx(const uint8_t *cx, const uint8_t *sx, const uint8_t *cw, const uint8_t *sw, int64_t M,
                 int64_t N, int64_t Kp, double *ref) {
  const int64_t groups = Kp / 32;
#pragma omp parallel for schedule(static) collapse(2)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double acc = 0.0;
      for (int64_t g = 0; g < groups; ++g) {
        double part = 0.0; /* sums of multiples of 0.25 below 32 * 36: exact */
        for (int i = 0; i < 32; ++i)
          part += xqo_e2m1_value(cx[m * Kp + g * 32 + i]) * xqo_e2m1_value(cw[n * Kp + g * 32 + i]);
        acc += ldexp(part, (int)sx[m * groups + g] - 127 + (int)sw[n * groups + g] - 127);
      }
      ref[m * N + n] = acc;
    }
}
