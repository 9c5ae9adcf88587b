/*
 * TWEO / FP8 per-tensor linear path -- CPU ORACLE.
 *
 * This file is TEST INFRASTRUCTURE, not product code.  It is a plain, slow,
 * scalar restatement of what the hot path computes, written from the paper's
 * definitions so that a reader can check it against them by eye:
 *
 *   - the TWEO regulariser (paper Eq. 3) and its derivative (paper Eq. 2 times
 *     Eq. 3, differentiated with respect to each activation),
 *   - per-tensor FP8 scaling and casting (paper Sec. 4.3: one scale for the
 *     whole tensor, E4M3 forward / E5M2 gradients; E4M3 range +-448 from the
 *     paper's introduction) with the OCP FP8 code tables,
 *   - the three linear-layer contractions on the quantised operands,
 *   - symmetric AbsMax b-bit quantisation (paper Eq. 4),
 *   - the block output A = x + f(x) the regulariser acts on (paper Sec. 3.3) and the
 *     delayed-scaling state (paper Sec. 4.3: amax history of length 16),
 *   - LayerNorm / RMSNorm (paper Sec. 4.3 runs the LayerNorm components under FP8 too) and
 *     the MLP activations of the paper's models (Sec. 3.2: GELU, GLU variants),
 *   - the FP4 step the paper's conclusion looks ahead to: the 4-bit E2M1 element with the same
 *     per-tensor scaling as the FP8 path.
 *
 * Floating point is FP64 unless the step is *defined* in FP32 (the scale, the
 * scaled value that gets rounded to FP8).  There is no blocking, no SIMD, no
 * BLAS, no reordering: sums run in index order.  OpenMP only splits outer
 * rows between threads, which changes no value.
 *
 * It shares no code, header, table or constant generator with the CUDA path
 * and neither includes the other.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may link or load this.
 *
 * Pins (see the CPU tests): every function below is pinned to something
 * outside itself -- printed values from the paper, closed forms, brute force,
 * finite differences, or an independent library routine.  Nothing here is
 * "parity unpinned".
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_E4M3 0
#define ORACLE_E5M2 1
#define ORACLE_E2M1 2 /* 4-bit codes, one per byte (low nibble), where a GEMM routine takes a format */

/* ------------------------------------------------------------------ bf16 */

/* bf16 is the upper half of an IEEE binary32; widening is exact. */
static float bf16_bits_to_f32(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

float oracle_bf16_to_f32(uint16_t b) { return bf16_bits_to_f32(b); }

/* Round a double to bf16 (8 significant bits, binary32 exponent range),
 * round-to-nearest, ties to even, in ONE rounding from the double.
 * Overflow goes to infinity as IEEE prescribes; NaN maps to 0x7FC0|sign. */
uint16_t oracle_f64_to_bf16(double v) {
  if (isnan(v)) return (uint16_t)(signbit(v) ? 0xFFC0 : 0x7FC0);
  uint16_t sign = signbit(v) ? 0x8000 : 0;
  double a = fabs(v);
  if (a == 0.0) return sign;
  if (isinf(a)) return (uint16_t)(sign | 0x7F80);
  int ex;
  (void)frexp(a, &ex);      /* a = f * 2^ex, f in [0.5,1)            */
  int E = ex - 1;           /* a = m * 2^E,  m in [1,2)              */
  const int MBITS = 7, BIAS = 127, EMIN = -126;
  if (E < EMIN) {           /* subnormal: spacing 2^(EMIN-MBITS)     */
    double q = ldexp(a, -(EMIN - MBITS));
    double r = nearbyint(q); /* default rounding mode = ties-to-even */
    return (uint16_t)(sign | (uint16_t)r); /* r==128 carries into e=1 */
  }
  double q = ldexp(a, -(E - MBITS)); /* in [128,256) */
  double r = nearbyint(q);
  if (r == 256.0) { r = 128.0; E += 1; }
  if (E > 127) return (uint16_t)(sign | 0x7F80);
  return (uint16_t)(sign | ((uint16_t)(E + BIAS) << MBITS) | ((uint16_t)r - 128));
}

void oracle_f64_array_to_bf16(const double* v, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_f64_to_bf16(v[i]);
}

/* ------------------------------------------------------------ FP8 tables */

/* OCP FP8 value of one code.  E4M3: 1 sign, 4 exponent (bias 7), 3 mantissa,
 * no infinities, the single NaN pattern is exponent=15 & mantissa=7; largest
 * finite value is 1.75 * 2^8 = 448 (the range the paper quotes).
 * E5M2: 1 sign, 5 exponent (bias 15), 2 mantissa, IEEE-style inf/NaN;
 * largest finite value is 1.75 * 2^15 = 57344. */
double oracle_fp8_decode(uint8_t code, int fmt) {
  int s = code >> 7;
  double sign = s ? -1.0 : 1.0;
  if (fmt == ORACLE_E4M3) {
    int e = (code >> 3) & 15, m = code & 7;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) return sign * ldexp((double)m, -9);
    return sign * ldexp(1.0 + m / 8.0, e - 7);
  } else {
    int e = (code >> 2) & 31, m = code & 3;
    if (e == 31) return m == 0 ? sign * INFINITY : NAN;
    if (e == 0) return sign * ldexp((double)m, -16);
    return sign * ldexp(1.0 + m / 4.0, e - 15);
  }
}

double oracle_fp8_max(int fmt) { return fmt == ORACLE_E4M3 ? 448.0 : 57344.0; }
static uint8_t fp8_max_code(int fmt) { return fmt == ORACLE_E4M3 ? 0x7E : 0x7B; }

/* Encoder A (arithmetic).  Saturating round-to-nearest-even of a binary32
 * value: NaN -> 0x7F (a NaN carries no sign: IEEE 754 leaves the sign of a NaN
 * product unspecified, so none is propagated); |v| >= max finite (infinity included) -> sign|max
 * code; otherwise the nearest representable value, ties to the even code;
 * zero and values that round to zero keep their sign. */
uint8_t oracle_fp8_encode(float v, int fmt) {
  if (isnan(v)) return 0x7F;
  uint8_t sign = signbit(v) ? 0x80 : 0x00;
  double a = fabs((double)v);
  if (a >= oracle_fp8_max(fmt)) return (uint8_t)(sign | fp8_max_code(fmt));
  if (a == 0.0) return sign;
  const int MBITS = fmt == ORACLE_E4M3 ? 3 : 2;
  const int BIAS = fmt == ORACLE_E4M3 ? 7 : 15;
  const int EMIN = 1 - BIAS;
  int ex;
  (void)frexp(a, &ex);
  int E = ex - 1; /* a = m * 2^E with m in [1,2) */
  if (E < EMIN) {
    /* subnormal grid: multiples of 2^(EMIN-MBITS); a carry to 2^MBITS is the
     * smallest normal number, whose code is exactly that integer. */
    double r = nearbyint(ldexp(a, -(EMIN - MBITS)));
    return (uint8_t)(sign | (uint8_t)r);
  }
  double r = nearbyint(ldexp(a, -(E - MBITS))); /* in [2^MBITS, 2^(MBITS+1)] */
  if (r == (double)(2 << MBITS)) { r = (double)(1 << MBITS); E += 1; }
  return (uint8_t)(sign | ((uint8_t)(E + BIAS) << MBITS) | ((uint8_t)r - (1 << MBITS)));
}

/* Encoder B (brute force).  Same contract, no exponent arithmetic: look at
 * every non-negative finite code, keep the closest decoded value, and on an
 * exact tie keep the code whose last bit is 0.  Used only to cross-check A. */
uint8_t oracle_fp8_encode_search(float v, int fmt) {
  if (isnan(v)) return 0x7F;
  uint8_t sign = signbit(v) ? 0x80 : 0x00;
  double a = fabs((double)v);
  if (a >= oracle_fp8_max(fmt)) return (uint8_t)(sign | fp8_max_code(fmt));
  int best = 0;
  double best_d = INFINITY;
  for (int c = 0; c <= fp8_max_code(fmt); ++c) {
    double d = fabs(oracle_fp8_decode((uint8_t)c, fmt) - a); /* exact in FP64 */
    if (d < best_d || (d == best_d && (c & 1) == 0)) { best_d = d; best = c; }
  }
  return (uint8_t)(sign | best);
}

/* Element-wise application of encoder A (which = 0) or B (which = 1). */
void oracle_fp8_encode_array(const float* v, int64_t n, int fmt, int which, uint8_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i)
    out[i] = which ? oracle_fp8_encode_search(v[i], fmt) : oracle_fp8_encode(v[i], fmt);
}

/* ------------------------------------------------- amax / scale / quantize */

/* amax = max_i |x_i| over the whole tensor (one scale per tensor, Sec. 4.3).
 * NaN elements are skipped (fmax semantics); infinities count. */
float oracle_amax_bf16(const uint16_t* x, int64_t n) {
  float amax = 0.0f;
  for (int64_t i = 0; i < n; ++i) {
    float a = fabsf(bf16_bits_to_f32(x[i]));
    if (a > amax) amax = a; /* false for NaN */
  }
  return amax;
}

/* scale = fl32(FP8MAX / amax) so that the largest element lands on the
 * format's largest finite value; scale_inv = fl32(1 / scale).  Degenerate
 * tensors (amax = 0, or non-finite) get scale 1; a quotient that overflows
 * binary32 is clamped to FLT_MAX. */
void oracle_scale_from_amax(float amax, int fmt, float* scale, float* scale_inv) {
  float s = 1.0f;
  if (amax > 0.0f && isfinite(amax)) {
    volatile float q = (float)oracle_fp8_max(fmt) / amax; /* one fp32 division */
    s = q;
    if (isinf(s)) s = FLT_MAX;
  }
  volatile float inv = 1.0f / s;
  *scale = s;
  *scale_inv = inv;
}

/* q_i = encode( fl32( x_i * scale ) ): one binary32 multiply (round to
 * nearest even, not fused with anything), then one saturating RNE to FP8.
 * sat_count (optional) = number of elements whose scaled magnitude exceeds
 * the largest finite FP8 value, i.e. that the saturation actually clips. */
void oracle_quantize_bf16(const uint16_t* x, int64_t n, int fmt, float scale,
                          uint8_t* q, uint64_t* sat_count) {
  uint64_t sat = 0;
  const float fmax = (float)oracle_fp8_max(fmt);
  for (int64_t i = 0; i < n; ++i) {
    volatile float v = bf16_bits_to_f32(x[i]) * scale;
    q[i] = oracle_fp8_encode(v, fmt);
    if (fabsf(v) > fmax) ++sat; /* false for NaN */
  }
  if (sat_count) *sat_count = sat;
}

/* ------------------------------------------------------------------ GEMMs */
/* All three take the FP8 codes, decode them, and sum in FP64 in index order,
 * then apply the two dequantisation factors.  Storage (row-major):
 *   xq  [M, K]   activations          (ldx  elements between rows)
 *   wq  [N, K]   weights, one row per output feature
 *   dyq [M, N]   output gradients
 * Products of two FP8 values are small dyadic rationals, so for the
 * contraction lengths used here the FP64 sums are exact. */

double oracle_fp4_decode(uint8_t code);
static void fill_table(double* t, int fmt) {
  for (int c = 0; c < 256; ++c)
    t[c] = fmt == ORACLE_E2M1 ? oracle_fp4_decode((uint8_t)(c & 0x0F)) : oracle_fp8_decode((uint8_t)c, fmt);
}

/* forward: Y[i,j] = (sum_k X[i,k] W[j,k]) * sx_inv * sw_inv */
void oracle_gemm_fwd(const uint8_t* xq, int64_t ldx, int fmt_x,
                     const uint8_t* wq, int64_t ldw, int fmt_w,
                     double sx_inv, double sw_inv,
                     int64_t M, int64_t N, int64_t K, double* y, int64_t ldy) {
  double tx[256], tw[256];
  fill_table(tx, fmt_x);
  fill_table(tw, fmt_w);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += tx[xq[i * ldx + k]] * tw[wq[j * ldw + k]];
      y[i * ldy + j] = acc * sx_inv * sw_inv;
    }
}

/* data gradient: dX[i,k] = (sum_n dY[i,n] W[n,k]) * sdy_inv * sw_inv */
void oracle_gemm_dgrad(const uint8_t* dyq, int64_t lddy, int fmt_dy,
                       const uint8_t* wq, int64_t ldw, int fmt_w,
                       double sdy_inv, double sw_inv,
                       int64_t M, int64_t N, int64_t K, double* dx, int64_t lddx) {
  double tdy[256], tw[256];
  fill_table(tdy, fmt_dy);
  fill_table(tw, fmt_w);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i)
    for (int64_t k = 0; k < K; ++k) {
      double acc = 0.0;
      for (int64_t n = 0; n < N; ++n) acc += tdy[dyq[i * lddy + n]] * tw[wq[n * ldw + k]];
      dx[i * lddx + k] = acc * sdy_inv * sw_inv;
    }
}

/* weight gradient: dW[n,k] = (sum_m dY[m,n] X[m,k]) * sx_inv * sdy_inv */
void oracle_gemm_wgrad(const uint8_t* xq, int64_t ldx, int fmt_x,
                       const uint8_t* dyq, int64_t lddy, int fmt_dy,
                       double sx_inv, double sdy_inv,
                       int64_t M, int64_t N, int64_t K, double* dw, int64_t lddw) {
  double tx[256], tdy[256];
  fill_table(tx, fmt_x);
  fill_table(tdy, fmt_dy);
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      double acc = 0.0;
      for (int64_t m = 0; m < M; ++m) acc += tdy[dyq[m * lddy + n]] * tx[xq[m * ldx + k]];
      dw[n * lddw + k] = acc * sx_inv * sdy_inv;
    }
}

/* The same three definitions evaluated only at a list of output positions
 * (rows[t], cols[t]); used where a full FP64 product would take hours. */
void oracle_gemm_fwd_at(const uint8_t* xq, int64_t ldx, int fmt_x,
                        const uint8_t* wq, int64_t ldw, int fmt_w,
                        double sx_inv, double sw_inv, int64_t K,
                        const int64_t* rows, const int64_t* cols, int64_t npts, double* out) {
  double tx[256], tw[256];
  fill_table(tx, fmt_x);
  fill_table(tw, fmt_w);
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < npts; ++t) {
    int64_t i = rows[t], j = cols[t];
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k) acc += tx[xq[i * ldx + k]] * tw[wq[j * ldw + k]];
    out[t] = acc * sx_inv * sw_inv;
  }
}

void oracle_gemm_dgrad_at(const uint8_t* dyq, int64_t lddy, int fmt_dy,
                          const uint8_t* wq, int64_t ldw, int fmt_w,
                          double sdy_inv, double sw_inv, int64_t N,
                          const int64_t* rows, const int64_t* cols, int64_t npts, double* out) {
  double tdy[256], tw[256];
  fill_table(tdy, fmt_dy);
  fill_table(tw, fmt_w);
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < npts; ++t) {
    int64_t i = rows[t], k = cols[t];
    double acc = 0.0;
    for (int64_t n = 0; n < N; ++n) acc += tdy[dyq[i * lddy + n]] * tw[wq[n * ldw + k]];
    out[t] = acc * sdy_inv * sw_inv;
  }
}

void oracle_gemm_wgrad_at(const uint8_t* xq, int64_t ldx, int fmt_x,
                          const uint8_t* dyq, int64_t lddy, int fmt_dy,
                          double sx_inv, double sdy_inv, int64_t M,
                          const int64_t* rows, const int64_t* cols, int64_t npts, double* out) {
  double tx[256], tdy[256];
  fill_table(tx, fmt_x);
  fill_table(tdy, fmt_dy);
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < npts; ++t) {
    int64_t n = rows[t], k = cols[t];
    double acc = 0.0;
    for (int64_t m = 0; m < M; ++m) acc += tdy[dyq[m * lddy + n]] * tx[xq[m * ldx + k]];
    out[t] = acc * sx_inv * sdy_inv;
  }
}

/* ------------------------------------------------------------------- TWEO */

/* Eq. 3 for one block output: the mean over all n elements of
 * (|a_i| / (tau + eps))^p.  eps is added to tau, as printed. */
double oracle_tweo_loss_block(const uint16_t* a, int64_t n, double tau, double eps, double p) {
  const double d = tau + eps;
  double sum = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    double r = fabs((double)bf16_bits_to_f32(a[i])) / d;
    sum += pow(r, p);
  }
  return n > 0 ? sum / (double)n : 0.0;
}

/* Derivative of  c * (1/n) sum_i (|a_i|/(tau+eps))^p  with respect to a_i:
 *   g_i = c * p * sign(a_i) * |a_i|^(p-1) / (n * (tau+eps)^p),   g_i = 0 at a_i = 0.
 * The caller folds lambda(t) (Eq. 2), the 1/L of Eq. 3 and any upstream
 * gradient into the single coefficient c. */
void oracle_tweo_grad_block(const uint16_t* a, int64_t n, double tau, double eps, double p,
                            double c, double* g) {
  const double d = tau + eps;
  const double k = c * p / ((double)n * pow(d, p));
  for (int64_t i = 0; i < n; ++i) {
    double v = (double)bf16_bits_to_f32(a[i]);
    if (v == 0.0 || isnan(v)) { g[i] = v == 0.0 ? 0.0 : NAN; continue; }
    double s = v > 0.0 ? 1.0 : -1.0;
    g[i] = k * s * pow(fabs(v), p - 1.0);
  }
}

/* ------------------------------------------------- Eq. 4, integer AbsMax */

/* s = max|X| + eps;  X_q = round(X / s * Q_b), Q_b = 2^(b-1) - 1, ties to
 * even, clamped to [-Q_b, Q_b] (the clamp only acts when a static s is
 * smaller than the tensor's own maximum).  Returns Q_b. */
int oracle_absmax_qmax(int bits) { return (1 << (bits - 1)) - 1; }

void oracle_absmax_quantize(const double* x, int64_t n, int bits, double s, int32_t* xq) {
  const double Q = (double)oracle_absmax_qmax(bits);
  for (int64_t i = 0; i < n; ++i) {
    double r = nearbyint(x[i] / s * Q);
    if (r > Q) r = Q;
    if (r < -Q) r = -Q;
    xq[i] = (int32_t)r;
  }
}

void oracle_absmax_dequantize(const int32_t* xq, int64_t n, int bits, double s, double* x) {
  const double Q = (double)oracle_absmax_qmax(bits);
  for (int64_t i = 0; i < n; ++i) x[i] = (double)xq[i] / Q * s;
}

double oracle_absmax_scale(const double* x, int64_t n, double eps) {
  double m = 0.0;
  for (int64_t i = 0; i < n; ++i) if (fabs(x[i]) > m) m = fabs(x[i]);
  return m + eps;
}

/* The same quantiser on bf16 tensors in the arithmetic an 8-bit kernel uses, so that the
 * integer codes can be compared bit for bit: everything in binary32, each operation
 * rounded once, in the order Eq. 4 writes them --
 *   s   = fl32(max|X| + eps)                 (per tensor, or per row: one s per channel / token)
 *   c   = fl32(Q_b / s)                      (once per scale)
 *   X_q = clamp(rne_int(fl32(X * c)), -Q_b, Q_b)
 * i.e. Eq. 4's X / s * Q_b evaluated as X * (Q_b / s): one division per scale and one
 * multiplication per element, the form an 8-bit kernel runs at memory speed.
 * NaN elements are skipped by the maximum and quantise to 0. */
float oracle_absmax_scale_bf16(const uint16_t* x, int64_t n, float eps) {
  volatile float s = oracle_amax_bf16(x, n) + eps;
  return s;
}

void oracle_absmax_quantize_bf16(const uint16_t* x, int64_t n, int bits, float s, int8_t* xq) {
  const float Q = (float)oracle_absmax_qmax(bits);
  volatile float c = Q / s;
  for (int64_t i = 0; i < n; ++i) {
    volatile float t = bf16_bits_to_f32(x[i]) * c;
    float r = nearbyintf(t);
    if (r > Q) r = Q;
    if (r < -Q) r = -Q;
    xq[i] = (t != t) ? 0 : (int8_t)r;
  }
}

/* 8-bit linear on the integer codes (Sec. 4.4): Y_mn = (sum_k Xq_mk * Wq_nk) * (sx_m / Q_b) * (sw_n / Q_b),
 * i.e. the product of the dequantised operands of Eq. 4, with one scale per tensor or per
 * row (token for X, output channel for W).  The integer sum is exact; the scales are applied
 * in FP64.  Evaluated at the listed (row, col) points. */
void oracle_int8_gemm_at(const int8_t* xq, int64_t ldx, const int8_t* wq, int64_t ldw, const float* sx,
                         int sx_per_row, const float* sw, int sw_per_row, int bits, int64_t K,
                         const int64_t* rows, const int64_t* cols, int64_t npts, double* y) {
  const double Q = (double)oracle_absmax_qmax(bits);
  for (int64_t t = 0; t < npts; ++t) {
    const int64_t m = rows[t], n = cols[t];
    int64_t acc = 0;
    for (int64_t k = 0; k < K; ++k) acc += (int64_t)xq[m * ldx + k] * (int64_t)wq[n * ldw + k];
    const double a = (double)sx[sx_per_row ? m : 0] / Q, b = (double)sw[sw_per_row ? n : 0] / Q;
    y[t] = (double)acc * a * b;
  }
}

/* ------------------------------------------------------------------ block output */
/* The regulariser acts on the block output A^(l) = x + f(x) (Sec. 3.3: the residual
 * stream plus the block's branch).  With bf16 activations the sum is formed in binary32
 * and rounded once more to bf16 (round to nearest even): a_i = bf16(fl32(x_i + f_i)).
 * Everything downstream (Eq. 3, its gradient, amax, the FP8 cast for the next block) is
 * the functions above applied to these bf16 values. */
void oracle_residual_add_bf16(const uint16_t* x, const uint16_t* f, int64_t n, uint16_t* a) {
  for (int64_t i = 0; i < n; ++i) {
    volatile float s = bf16_bits_to_f32(x[i]) + bf16_bits_to_f32(f[i]); /* one binary32 add */
    a[i] = oracle_f64_to_bf16((double)s);
  }
}

/* ------------------------------------------------------------------ delayed scaling */
/* Sec. 4.3: per-tensor delayed scaling with an amax history of length H (16 in the paper).
 * One update per training step and tensor: the history moves one place (the oldest value
 * drops out), the step's amax enters at index 0, and the scale for the NEXT step is
 * FP8MAX / max(history) -- as oracle_scale_from_amax computes it.  If that maximum is zero
 * or not finite the previous scale is kept. */
void oracle_delayed_scaling_update(float* history, int H, float amax_new, int fmt, float* scale, float* scale_inv) {
  for (int j = H - 1; j > 0; --j) history[j] = history[j - 1];
  history[0] = amax_new;
  float m = 0.0f;
  for (int j = 0; j < H; ++j)
    if (history[j] > m) m = history[j]; /* false for NaN */
  if (m > 0.0f && isfinite(m)) {
    oracle_scale_from_amax(m, fmt, scale, scale_inv);
  } else {
    volatile float inv = 1.0f / *scale;
    *scale_inv = inv;
  }
}

/* ------------------------------------------------------------------ normalisation and MLP activations */
/* Sec. 4.3 puts the LayerNorm components under FP8 as well as the linears: the normalised
 * row is what the next linear consumes, so it is cast with that linear's per-tensor scale.
 * LayerNorm over the last dimension, written out (FP64):
 *     mu = (1/d) sum_j x_j,  var = (1/d) sum_j (x_j - mu)^2   (biased),
 *     y_j = (x_j - mu) / sqrt(var + eps) * gamma_j + beta_j.
 * rms != 0 gives the RMSNorm of the Llama-style blocks instead: mu := 0 and
 *     var := (1/d) sum_j x_j^2, no centring; beta may be NULL (zero).
 * x: bf16 [rows, d]; gamma, beta: binary32 [d]; y: FP64 [rows, d]; mean / rstd (optional): FP64 [rows]. */
void oracle_layernorm(const uint16_t* x, int64_t rows, int64_t d, const float* gamma, const float* beta,
                      double eps, int rms, double* y, double* mean, double* rstd) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    const uint16_t* xr = x + r * d;
    double mu = 0.0;
    if (!rms) {
      for (int64_t j = 0; j < d; ++j) mu += (double)bf16_bits_to_f32(xr[j]);
      mu /= (double)d;
    }
    double var = 0.0;
    for (int64_t j = 0; j < d; ++j) {
      const double c = (double)bf16_bits_to_f32(xr[j]) - mu;
      var += c * c;
    }
    var /= (double)d;
    const double rs = 1.0 / sqrt(var + eps);
    for (int64_t j = 0; j < d; ++j) {
      const double c = (double)bf16_bits_to_f32(xr[j]) - mu;
      y[r * d + j] = c * rs * (double)gamma[j] + (beta ? (double)beta[j] : 0.0);
    }
    if (mean) mean[r] = mu;
    if (rstd) rstd[r] = rs;
  }
}

/* The MLP activations the paper's models use (Sec. 3.2: classic MLPs with GELU, modern
 * MLPs with GLU variants), as their definitions, FP64:
 *   kind 1  GELU(v) = v * Phi(v) = v/2 * (1 + erf(v / sqrt 2))
 *   kind 2  GELU, tanh form: v/2 * (1 + tanh( sqrt(2/pi) * (v + 0.044715 v^3) ))
 *   kind 3  SiLU(v) = v / (1 + exp(-v))   (the gate of SwiGLU: out = SiLU(gate) * up) */
double oracle_activation(double v, int kind) {
  switch (kind) {
    case 1: return 0.5 * v * (1.0 + erf(v / sqrt(2.0)));
    case 2: return 0.5 * v * (1.0 + tanh(sqrt(2.0 / (4.0 * atan(1.0))) * (v + 0.044715 * v * v * v)));
    case 3: return v / (1.0 + exp(-v));
    default: return v;
  }
}

void oracle_activation_array(const double* v, int64_t n, int kind, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_activation(v[i], kind);
}

/* ------------------------------------------------------------------ 8-bit residual stream */
/* Sec. 4.4 quantises the residual stream too: in y = x + f(x) both the stream x and the
 * block's branch f(x) are Eq. 4 codes with static per-tensor scales, and so is y -- no
 * bf16 tensor in between.  Dequantising both inputs with Eq. 4, adding, and quantising the sum
 * with Eq. 4 again, Q_b cancels:
 *   y_q = clamp( round( (x_q s_x / Q_b + f_q s_f / Q_b) / s_y * Q_b ) ) = clamp( round( x_q (s_x / s_y) + f_q (s_f / s_y) ) ),
 * one requantisation multiplier per input.  As in oracle_absmax_quantize_bf16 everything is
 * binary32 so the integer codes can be compared bit for bit:
 *   a = fl32(sx / sy),  b = fl32(sf / sy)                 (once per tensor)
 *   t_i = fl32( fq_i * b + fl32(xq_i * a) )               (one product, one fused multiply-add)
 *   yq_i = clamp(rne_int(t_i), -Q_b, Q_b),  NaN -> 0 */
void oracle_residual_add_q8(const int8_t* xq, const int8_t* fq, int64_t n, int bits, float sx, float sf, float sy,
                            int8_t* yq) {
  const float Q = (float)oracle_absmax_qmax(bits);
  volatile float a = sx / sy, b = sf / sy;
  for (int64_t i = 0; i < n; ++i) {
    volatile float p = (float)xq[i] * a;
    volatile float t = fmaf((float)fq[i], b, p);
    float r = nearbyintf(t);
    if (r > Q) r = Q;
    if (r < -Q) r = -Q;
    yq[i] = (t != t) ? 0 : (int8_t)r;
  }
}

/* The 8-bit linear whose output is requantised with a static per-tensor scale (Sec. 4.4:
 * W8A8 with the activation scales fixed beforehand), at sampled points, in the binary32
 * order an integer-tensor-core epilogue uses so the codes compare bit for bit:
 *   acc  = sum_k Xq_mk Wq_nk                       (exact integer)
 *   y    = fl32( fl32( fl32(acc) * fl32(sx_m * fl32(1 / Q_b^2)) ) * sw_n )
 *   yq   = clamp(rne_int(fl32(y * fl32(Q_b / sy))), -Q_b, Q_b)
 * y equals oracle_int8_gemm_at's FP64 value to binary32 rounding (checked in the tests). */
void oracle_int8_gemm_q8_at(const int8_t* xq, int64_t ldx, const int8_t* wq, int64_t ldw, const float* sx,
                            int sx_per_row, const float* sw, int sw_per_row, int bits, float sy, int64_t K,
                            const int64_t* rows, const int64_t* cols, int64_t npts, int8_t* yq, float* y32) {
  const float Q = (float)oracle_absmax_qmax(bits);
  volatile float post = 1.0f / (Q * Q);
  volatile float cy = Q / sy;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < npts; ++t) {
    const int64_t m = rows[t], n = cols[t];
    int64_t acc = 0;
    for (int64_t k = 0; k < K; ++k) acc += (int64_t)xq[m * ldx + k] * (int64_t)wq[n * ldw + k];
    volatile float ar = sx[sx_per_row ? m : 0] * post;
    volatile float a = (float)(int32_t)acc; /* the tensor core's int32 accumulator, converted round-to-nearest */
    volatile float b = a * ar;
    volatile float y = b * sw[sw_per_row ? n : 0];
    volatile float u = y * cy;
    float r = nearbyintf(u);
    if (r > Q) r = Q;
    if (r < -Q) r = -Q;
    yq[t] = (u != u) ? 0 : (int8_t)r;
    if (y32) y32[t] = y;
  }
}

/* Per-token variant of the quantised residual stream (Sec. 4.4 reports both per-tensor "A8(T)" and
 * per-token "A8(K)" activations with the residual quantised): every row (token) m of x and f(x) carries
 * its own Eq. 4 scale sx[m], sf[m], and the sum gets the AbsMax scale of its own row,
 *   y_mj  = fl32( fq_mj * fl32(sf[m] / Q_b) + fl32(xq_mj * fl32(sx[m] / Q_b)) )     dequantise and add
 *   sy[m] = fl32( max_j |y_mj| + eps )                                              Eq. 4, per row
 *   yq_mj = clamp( rne_int( fl32(y_mj * fl32(Q_b / sy[m])) ), -Q_b, Q_b )
 * everything in binary32 as in oracle_absmax_quantize_bf16, so the codes compare bit for bit. */
void oracle_residual_add_q8_rows(const int8_t* xq, const float* sx, const int8_t* fq, const float* sf, int64_t rows,
                                 int64_t cols, int bits, float eps, int8_t* yq, float* sy) {
  const float Q = (float)oracle_absmax_qmax(bits);
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < rows; ++m) {
    volatile float cx = sx[m] / Q, cf = sf[m] / Q;
    float amax = 0.0f;
    for (int64_t j = 0; j < cols; ++j) {
      volatile float p = (float)xq[m * cols + j] * cx;
      volatile float y = fmaf((float)fq[m * cols + j], cf, p);
      const float a = fabsf(y);
      if (a > amax) amax = a; /* false for NaN */
    }
    volatile float s = amax + eps;
    volatile float c = Q / s;
    sy[m] = s;
    for (int64_t j = 0; j < cols; ++j) {
      volatile float p = (float)xq[m * cols + j] * cx;
      volatile float y = fmaf((float)fq[m * cols + j], cf, p);
      volatile float t = y * c;
      float r = nearbyintf(t);
      if (r > Q) r = Q;
      if (r < -Q) r = -Q;
      yq[m * cols + j] = (t != t) ? 0 : (int8_t)r;
    }
  }
}

/* ------------------------------------------------------------------ FP4 (E2M1) */
/* The paper's conclusion names FP4 training and inference as the step after FP8 and fixes no
 * format.  Reading taken here: the 4-bit floating-point element of the OCP Microscaling formats
 * (E2M1: 1 sign bit, 2 exponent bits with bias 1, 1 mantissa bit; no infinities, no NaN), with ONE
 * scale per tensor exactly as in the FP8 path of Sec. 4.3 (scale = largest finite value / amax).
 *   code = s e e m;   e = 0: (-1)^s * m * 2^-1 ;   e > 0: (-1)^s * (1 + m / 2) * 2^(e - 1)
 * so the magnitudes are 0, 0.5, 1, 1.5, 2, 3, 4, 6. */
double oracle_fp4_decode(uint8_t code) {
  const int s = (code >> 3) & 1, e = (code >> 1) & 3, m = code & 1;
  const double mag = e == 0 ? 0.5 * (double)m : ldexp(1.0 + 0.5 * (double)m, e - 1);
  return s ? -mag : mag;
}

double oracle_fp4_max(void) { return 6.0; }

/* Saturating round-to-nearest-even, by search over the eight magnitudes (the definition written
 * out): the closest value wins, an exact tie goes to the code whose last bit is 0.  |v| >= 6
 * (infinity included) -> sign | 0x7.  The format has no NaN code: a NaN becomes +6 (code 0x7), the
 * "NaN saturates to the largest positive value" convention of conversions into NaN-less formats.
 * Zero and values that round to zero keep their sign. */
uint8_t oracle_fp4_encode(float v) {
  if (isnan(v)) return 0x7;
  const uint8_t sign = signbit(v) ? 0x8 : 0x0;
  const double a = fabs((double)v);
  if (a >= 6.0) return (uint8_t)(sign | 0x7);
  int best = 0;
  double best_d = INFINITY;
  for (int c = 0; c <= 7; ++c) {
    const double d = fabs(oracle_fp4_decode((uint8_t)c) - a); /* exact in FP64 */
    if (d < best_d || (d == best_d && (c & 1) == 0)) { best_d = d; best = c; }
  }
  return (uint8_t)(sign | best);
}

void oracle_fp4_encode_array(const float* v, int64_t n, uint8_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_fp4_encode(v[i]);
}

/* scale = fl32(6 / amax), scale_inv = fl32(1 / scale); the degenerate cases as in
 * oracle_scale_from_amax. */
void oracle_fp4_scale_from_amax(float amax, float* scale, float* scale_inv) {
  float s = 1.0f;
  if (amax > 0.0f && isfinite(amax)) {
    volatile float q = 6.0f / amax;
    s = q;
    if (isinf(s)) s = FLT_MAX;
  }
  volatile float inv = 1.0f / s;
  *scale = s;
  *scale_inv = inv;
}

/* code_i = encode( fl32( x_i * scale ) ): one binary32 multiply, one saturating RNE onto the
 * E2M1 grid.  codes: one code per byte.  packed (optional): two codes per byte, element 2i in the
 * low nibble and element 2i + 1 in the high nibble; an odd n leaves the last high nibble 0. */
void oracle_fp4_quantize_bf16(const uint16_t* x, int64_t n, float scale, uint8_t* codes, uint8_t* packed) {
  for (int64_t i = 0; i < n; ++i) {
    volatile float v = bf16_bits_to_f32(x[i]) * scale;
    codes[i] = oracle_fp4_encode(v);
  }
  if (packed)
    for (int64_t i = 0; i < (n + 1) / 2; ++i)
      packed[i] = (uint8_t)(codes[2 * i] | ((2 * i + 1 < n ? codes[2 * i + 1] : 0) << 4));
}
