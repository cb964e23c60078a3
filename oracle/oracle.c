/*
 * oracle.c - plain, slow, fp64 CPU definitions (see oracle.h).
 * TEST INFRASTRUCTURE ONLY: used by tests, the smoke check and the benchmark's
 * CPU-baseline leg.  Shares nothing with the CUDA library.
 *
 * Build: gcc -O2 -std=c99 -fopenmp -fPIC -shared oracle.c -o liboracle.so -lm
 * (no -ffast-math: the compensated sums and the NaN / inf rules rely on IEEE).
 */
#include "oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int g_last_threads = 1;

/* ---- Neumaier-compensated accumulation ------------------------------------ */
typedef struct { double s, c; } nsum;

static void nsum_add(nsum* a, double v) {
  double t = a->s + v;
  if (fabs(a->s) >= fabs(v)) a->c += (a->s - t) + v;
  else                       a->c += (v - t) + a->s;
  a->s = t;
}
static double nsum_get(const nsum* a) { return a->s + a->c; }

/* ---- exact widening of stored elements to double --------------------------- */
static double widen(const void* base, int dtype, int64_t idx) {
  if (dtype == ORACLE_F32) return (double)((const float*)base)[idx];
  if (dtype == ORACLE_F64) return ((const double*)base)[idx];
  if (dtype == ORACLE_F16) {
    /* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits */
    uint16_t h = ((const uint16_t*)base)[idx];
    int e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);                       /* zero and subnormals */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)m / 1024.0, e - 15);
    return (h & 0x8000) ? -v : v;
  }
  /* bf16: the 16 stored bits are the high half of an IEEE binary32 */
  uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

static int bad_dtype(int dtype) {
  return dtype != ORACLE_F32 && dtype != ORACLE_BF16 && dtype != ORACLE_F64 && dtype != ORACLE_F16;
}

int oracle_widen(const void* base, int dtype, int64_t n, double* out) {
  if (bad_dtype(dtype) || n < 0 || (n > 0 && (!base || !out))) return 1;
  for (int64_t i = 0; i < n; ++i) out[i] = widen(base, dtype, i);
  return 0;
}

/* ---- softmax family --------------------------------------------------------- */

/* classify the row: 0 = ordinary (m finite), 1 = NaN row, 2 = no live entry */
static int softmax_stats(const double* z, int64_t n, double* m_out, double* s_out) {
  double m = -INFINITY;
  int has_nan = 0;
  for (int64_t c = 0; c < n; ++c) {
    if (isnan(z[c])) has_nan = 1;
    else if (z[c] > m) m = z[c];
  }
  if (has_nan || m == INFINITY) return 1;
  if (m == -INFINITY) return 2;
  nsum s = {0.0, 0.0};
  for (int64_t c = 0; c < n; ++c) nsum_add(&s, exp(z[c] - m)); /* exp(-inf) = 0 */
  *m_out = m;
  *s_out = nsum_get(&s);
  return 0;
}

void oracle_softmax_row(const double* z, int64_t n, double* y) {
  double m = 0.0, s = 0.0;
  int kind = softmax_stats(z, n, &m, &s);
  if (kind == 1) { for (int64_t c = 0; c < n; ++c) y[c] = NAN; return; }
  if (kind == 2) { for (int64_t c = 0; c < n; ++c) y[c] = 0.0; return; }
  for (int64_t c = 0; c < n; ++c) y[c] = exp(z[c] - m) / s;
}

void oracle_log_softmax_row(const double* z, int64_t n, double* y) {
  double m = 0.0, s = 0.0;
  int kind = softmax_stats(z, n, &m, &s);
  if (kind == 1) { for (int64_t c = 0; c < n; ++c) y[c] = NAN; return; }
  if (kind == 2) { for (int64_t c = 0; c < n; ++c) y[c] = -INFINITY; return; }
  double ls = log(s);
  for (int64_t c = 0; c < n; ++c) y[c] = (z[c] - m) - ls; /* -inf stays -inf */
}

double oracle_logsumexp_row(const double* z, int64_t n) {
  double m = 0.0, s = 0.0;
  int kind = softmax_stats(z, n, &m, &s);
  if (kind == 1) return NAN;
  if (kind == 2) return -INFINITY;
  return m + log(s);
}

/* ---- normalisations --------------------------------------------------------- */

void oracle_layernorm_row(const double* x, int64_t n, const double* gamma,
                          const double* beta, double eps, double* y) {
  nsum a = {0.0, 0.0};
  for (int64_t c = 0; c < n; ++c) nsum_add(&a, x[c]);
  double mu = nsum_get(&a) / (double)n;
  nsum q = {0.0, 0.0};
  for (int64_t c = 0; c < n; ++c) { double d = x[c] - mu; nsum_add(&q, d * d); }
  double var = nsum_get(&q) / (double)n;
  double sd = sqrt(var + eps);
  for (int64_t c = 0; c < n; ++c) {
    double g = gamma ? gamma[c] : 1.0;
    double b = beta ? beta[c] : 0.0;
    y[c] = (x[c] - mu) / sd * g + b;
  }
}

void oracle_rmsnorm_row(const double* x, int64_t n, const double* w,
                        double eps, double* y) {
  nsum q = {0.0, 0.0};
  for (int64_t c = 0; c < n; ++c) nsum_add(&q, x[c] * x[c]);
  double ms = nsum_get(&q) / (double)n;
  double rms = sqrt(ms + eps);
  for (int64_t c = 0; c < n; ++c) y[c] = x[c] / rms * (w ? w[c] : 1.0);
}

/* ---- array drivers ------------------------------------------------------------ */

static int bad_shape(const void* x, int dtype, int64_t rows, int64_t cols,
                     int64_t stride, const double* out) {
  if (rows < 0 || cols < 0) return 1;
  if (rows == 0 || cols == 0) return 0;
  if (!x || !out) return 1;
  if (stride < cols) return 1;
  if (bad_dtype(dtype)) return 1;
  return 0;
}

static int use_threads(int nthreads) {
#ifdef _OPENMP
  int t = nthreads > 1 ? nthreads : 1;
#else
  int t = 1; (void)nthreads;
#endif
  g_last_threads = t;
  return t;
}

/* z for one row: widen, scale (1.0 for the plain operators: exact), add the additive mask,
 * apply the causal rule */
static void masked_row(const void* x, int dtype, int64_t cols, int64_t x_off,
                       int64_t grow, const oracle_mask* mask, double scale, double* z) {
  for (int64_t c = 0; c < cols; ++c) z[c] = scale * widen(x, dtype, x_off + c);
  if (!mask) return;
  if (mask->additive) {
    int64_t mr = grow % mask->add_rows;
    for (int64_t c = 0; c < cols; ++c)
      z[c] += widen(mask->additive, dtype, mr * mask->add_row_stride + c);
  }
  if (mask->causal) {
    int64_t last_live = grow % mask->causal_period + mask->causal_offset;
    for (int64_t c = 0; c < cols; ++c)
      if (c > last_live) z[c] = -INFINITY;
  }
}

static int softmax_driver(const void* x, int dtype, int64_t rows, int64_t cols,
                          int64_t x_stride, const int64_t* row_ids,
                          const oracle_mask* mask, double* out, int nthreads,
                          int want_log, double scale) {
  if (bad_shape(x, dtype, rows, cols, x_stride, out)) return 1;
  if (!(scale > 0.0) || isinf(scale)) return 1;
  if (mask) {
    if (mask->additive && (mask->add_rows < 1 || mask->add_row_stride < cols)) return 1;
    if (mask->causal && mask->causal_period < 1) return 1;
  }
  int t = use_threads(nthreads);
  if (rows == 0 || cols == 0) return 0;
  int failed = 0;
#pragma omp parallel num_threads(t)
  {
    double* z = (double*)malloc((size_t)cols * sizeof(double));
    if (!z) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
      if (!z) continue;
      int64_t grow = row_ids ? row_ids[i] : i;
      masked_row(x, dtype, cols, i * x_stride, grow, mask, scale, z);
      if (want_log) oracle_log_softmax_row(z, cols, out + i * cols);
      else          oracle_softmax_row(z, cols, out + i * cols);
    }
    free(z);
  }
  return failed;
}

int oracle_softmax(const void* x, int dtype, int64_t rows, int64_t cols,
                   int64_t x_stride, const int64_t* row_ids,
                   const oracle_mask* mask, double* out, int nthreads) {
  return softmax_driver(x, dtype, rows, cols, x_stride, row_ids, mask, out, nthreads, 0, 1.0);
}

int oracle_log_softmax(const void* x, int dtype, int64_t rows, int64_t cols,
                       int64_t x_stride, const int64_t* row_ids,
                       const oracle_mask* mask, double* out, int nthreads) {
  return softmax_driver(x, dtype, rows, cols, x_stride, row_ids, mask, out, nthreads, 1, 1.0);
}

/* softmax / log-softmax of scale * x (+ additive mask, causal rule): the fused pre-scale */
int oracle_softmax_scaled(const void* x, int dtype, int64_t rows, int64_t cols,
                          int64_t x_stride, double scale, const int64_t* row_ids,
                          const oracle_mask* mask, int want_log, double* out, int nthreads) {
  return softmax_driver(x, dtype, rows, cols, x_stride, row_ids, mask, out, nthreads, want_log ? 1 : 0, scale);
}

static double* widen_vector(const void* v, int dtype, int64_t n) {
  double* d = (double*)malloc((size_t)n * sizeof(double));
  if (d) for (int64_t c = 0; c < n; ++c) d[c] = widen(v, dtype, c);
  return d;
}

int oracle_layernorm(const void* x, int dtype, int64_t rows, int64_t cols,
                     int64_t x_stride, const void* gamma, const void* beta,
                     double eps, double* out, int nthreads) {
  if (bad_shape(x, dtype, rows, cols, x_stride, out)) return 1;
  if (!(eps >= 0.0)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0 || cols == 0) return 0;
  double* g = gamma ? widen_vector(gamma, dtype, cols) : NULL;
  double* b = beta ? widen_vector(beta, dtype, cols) : NULL;
  int failed = (gamma && !g) || (beta && !b);
#pragma omp parallel num_threads(t)
  {
    double* xr = (double*)malloc((size_t)cols * sizeof(double));
    if (!xr) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
      if (!xr || failed) continue;
      for (int64_t c = 0; c < cols; ++c) xr[c] = widen(x, dtype, i * x_stride + c);
      oracle_layernorm_row(xr, cols, g, b, eps, out + i * cols);
    }
    free(xr);
  }
  free(g);
  free(b);
  return failed;
}

int oracle_rmsnorm(const void* x, int dtype, int64_t rows, int64_t cols,
                   int64_t x_stride, const void* weight, double eps,
                   double* out, int nthreads) {
  if (bad_shape(x, dtype, rows, cols, x_stride, out)) return 1;
  if (!(eps >= 0.0)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0 || cols == 0) return 0;
  double* w = weight ? widen_vector(weight, dtype, cols) : NULL;
  int failed = (weight && !w);
#pragma omp parallel num_threads(t)
  {
    double* xr = (double*)malloc((size_t)cols * sizeof(double));
    if (!xr) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
      if (!xr || failed) continue;
      for (int64_t c = 0; c < cols; ++c) xr[c] = widen(x, dtype, i * x_stride + c);
      oracle_rmsnorm_row(xr, cols, w, eps, out + i * cols);
    }
    free(xr);
  }
  free(w);
  return failed;
}

/* ---- reduction over a non-last axis (layout of the Unified Sketch figure, Section 3.2.1) ---- */

int oracle_rowop_axis(int op, const void* x, int dtype, int64_t outer, int64_t reduce, int64_t inner,
                      int64_t outer_stride, int64_t reduce_stride, const void* gamma, const void* beta,
                      double eps, double* out, int nthreads) {
  if (op < 0 || op > 3) return 1;
  if (outer < 0 || reduce < 0 || inner < 0) return 1;
  if (bad_dtype(dtype)) return 1;
  if ((op == 2 || op == 3) && !(eps >= 0.0)) return 1;
  int t = use_threads(nthreads);
  if (outer == 0 || reduce == 0 || inner == 0) return 0;
  if (!x || !out) return 1;
  if (reduce_stride < inner || outer_stride < (reduce - 1) * reduce_stride + inner) return 1;
  double* g = (gamma && op >= 2) ? widen_vector(gamma, dtype, reduce) : NULL;
  double* b = (beta && op == 2) ? widen_vector(beta, dtype, reduce) : NULL;
  int failed = (gamma && op >= 2 && !g) || (beta && op == 2 && !b);
  int64_t lines = outer * inner;                      /* one line per (b, d) */
#pragma omp parallel num_threads(t)
  {
    double* z = (double*)malloc((size_t)reduce * sizeof(double));
    double* y = (double*)malloc((size_t)reduce * sizeof(double));
    if (!z || !y) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp for schedule(static)
    for (int64_t l = 0; l < lines; ++l) {
      if (!z || !y || failed) continue;
      int64_t bb = l / inner, d = l % inner;
      for (int64_t f = 0; f < reduce; ++f) z[f] = widen(x, dtype, bb * outer_stride + f * reduce_stride + d);
      if (op == 0) oracle_softmax_row(z, reduce, y);
      else if (op == 1) oracle_log_softmax_row(z, reduce, y);
      else if (op == 2) oracle_layernorm_row(z, reduce, g, b, eps, y);
      else oracle_rmsnorm_row(z, reduce, g, eps, y);
      for (int64_t f = 0; f < reduce; ++f) out[(bb * reduce + f) * inner + d] = y[f];
    }
    free(z);
    free(y);
  }
  free(g);
  free(b);
  return failed;
}

/* ---- fused residual add + normalisation (a "fused variant" of Section 3.6) ----------- */

int oracle_add_norm(int op, const void* x, const void* res, int dtype, int64_t rows, int64_t cols,
                    int64_t x_stride, int64_t res_stride, const void* gamma, const void* beta,
                    double eps, double* out_y, double* out_sum, int nthreads) {
  if (op != 2 && op != 3) return 1;
  if (bad_shape(x, dtype, rows, cols, x_stride, out_y)) return 1;
  if (rows > 0 && cols > 0 && (!res || !out_sum || res_stride < cols)) return 1;
  if (!(eps >= 0.0)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0 || cols == 0) return 0;
  double* g = gamma ? widen_vector(gamma, dtype, cols) : NULL;
  double* b = (beta && op == 2) ? widen_vector(beta, dtype, cols) : NULL;
  int failed = (gamma && !g) || (beta && op == 2 && !b);
#pragma omp parallel for schedule(static) num_threads(t)
  for (int64_t i = 0; i < rows; ++i) {
    if (failed) continue;
    double* s = out_sum + i * cols;
    /* the sum of two widened values is exact in double for fp32 / bf16 storage */
    for (int64_t c = 0; c < cols; ++c) s[c] = widen(x, dtype, i * x_stride + c) + widen(res, dtype, i * res_stride + c);
    if (op == 2) oracle_layernorm_row(s, cols, g, b, eps, out_y + i * cols);
    else oracle_rmsnorm_row(s, cols, g, eps, out_y + i * cols);
  }
  free(g);
  free(b);
  return failed;
}

/* ---- gated activations: SiLU-and-Mul, GELU-and-Mul (named in Section 3.6) ---------- */

double oracle_activation(int act, double a) {
  if (act == 0) return a / (1.0 + exp(-a));                           /* SiLU: a * sigmoid(a) */
  /* GELU: a * Phi(a), Phi(a) = 0.5 (1 + erf(a / sqrt 2)) = 0.5 erfc(-a / sqrt 2); the second
   * form is the same number without the cancellation of 1 + erf in the left tail */
  if (act == 1) return 0.5 * a * erfc(-a * 0.70710678118654752440);
  /* GELU, tanh form: 0.5 a (1 + tanh(u)), u = sqrt(2/pi) (a + 0.044715 a^3); by the identity
   * 0.5 (1 + tanh u) = 1 / (1 + e^(-2u)) it is evaluated without the cancellation of 1 + tanh */
  double u = 0.79788456080286535588 * (a + 0.044715 * a * a * a);
  return a / (1.0 + exp(-2.0 * u));
}

int oracle_act_mul(int act, const void* x, int dtype, int64_t rows, int64_t d, int64_t x_stride,
                   double* out, int nthreads) {
  if (act < 0 || act > 2) return 1;
  if (rows < 0 || d < 0) return 1;
  if (bad_dtype(dtype)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0 || d == 0) return 0;
  if (!x || !out || x_stride < 2 * d) return 1;
#pragma omp parallel for schedule(static) num_threads(t)
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t c = 0; c < d; ++c)
      out[i * d + c] = oracle_activation(act, widen(x, dtype, i * x_stride + c)) * widen(x, dtype, i * x_stride + d + c);
  return 0;
}

/* ---- other reduction-category operators of Section 3.6: arg-max / arg-min, cumulative --- */

/* Does a beat b as the arg-max (want_min 0) or arg-min (want_min 1) candidate?  NaN beats every
 * number (and another NaN does not beat it); equal values (-0 == +0 included) do not beat. */
static int arg_beats(double a, double b, int want_min) {
  if (isnan(b)) return 0;
  if (isnan(a)) return 1;
  return want_min ? (a < b) : (a > b);
}

int oracle_argreduce(int want_min, const void* x, int dtype, int64_t rows, int64_t cols, int64_t x_stride,
                     int64_t* out, int nthreads) {
  if (rows < 0 || cols < 0) return 1;
  if (bad_dtype(dtype)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0) return 0;
  if (cols == 0 || !x || !out || x_stride < cols) return 1;      /* an empty row has no arg-max */
#pragma omp parallel for schedule(static) num_threads(t)
  for (int64_t i = 0; i < rows; ++i) {
    int64_t best = 0;
    double bv = widen(x, dtype, i * x_stride);
    for (int64_t c = 1; c < cols; ++c) {
      double v = widen(x, dtype, i * x_stride + c);
      if (arg_beats(v, bv, want_min)) { bv = v; best = c; }     /* strict: the first of equals stays */
    }
    out[i] = best;
  }
  return 0;
}

int oracle_cumulative(int want_prod, const void* x, int dtype, int64_t rows, int64_t cols, int64_t x_stride,
                      double* out, int nthreads) {
  if (bad_shape(x, dtype, rows, cols, x_stride, out)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0 || cols == 0) return 0;
#pragma omp parallel for schedule(static) num_threads(t)
  for (int64_t i = 0; i < rows; ++i) {
    if (want_prod) {
      double p = 1.0;
      for (int64_t c = 0; c < cols; ++c) { p *= widen(x, dtype, i * x_stride + c); out[i * cols + c] = p; }
    } else {
      nsum s = {0.0, 0.0};                                      /* compensated running sum */
      double plain = 0.0;                                       /* carries inf / NaN as the arithmetic says */
      for (int64_t c = 0; c < cols; ++c) {
        double v = widen(x, dtype, i * x_stride + c);
        nsum_add(&s, v);
        plain += v;
        out[i * cols + c] = isfinite(plain) ? nsum_get(&s) : plain;
      }
    }
  }
  return 0;
}

/* ---- BatchNorm-style column statistics (BatchNorm is listed in Section 3.6) ----------- */

int oracle_colnorm(const void* x, int dtype, int64_t rows, int64_t cols, int64_t x_stride,
                   const void* gamma, const void* beta, double eps, double* out_y, double* out_mean,
                   double* out_var, int nthreads) {
  if (bad_shape(x, dtype, rows, cols, x_stride, out_y)) return 1;
  if (!(eps >= 0.0)) return 1;
  int t = use_threads(nthreads);
  if (rows == 0 || cols == 0) return 0;
  double* g = gamma ? widen_vector(gamma, dtype, cols) : NULL;
  double* b = beta ? widen_vector(beta, dtype, cols) : NULL;
  int failed = (gamma && !g) || (beta && !b);
#pragma omp parallel for schedule(static) num_threads(t)
  for (int64_t c = 0; c < cols; ++c) {
    if (failed) continue;
    nsum s = {0.0, 0.0};
    for (int64_t r = 0; r < rows; ++r) nsum_add(&s, widen(x, dtype, r * x_stride + c));
    double mean = nsum_get(&s) / (double)rows;
    nsum q = {0.0, 0.0};
    for (int64_t r = 0; r < rows; ++r) { double d = widen(x, dtype, r * x_stride + c) - mean; nsum_add(&q, d * d); }
    double var = nsum_get(&q) / (double)rows;                    /* biased, as in the forward pass */
    double rstd = 1.0 / sqrt(var + eps);
    double gc = g ? g[c] : 1.0, bc = b ? b[c] : 0.0;
    for (int64_t r = 0; r < rows; ++r) out_y[r * cols + c] = (widen(x, dtype, r * x_stride + c) - mean) * rstd * gc + bc;
    if (out_mean) out_mean[c] = mean;
    if (out_var) out_var[c] = var;
  }
  free(g);
  free(b);
  return failed;
}

/* ---- the paper's verifier criterion (Section 3.2.3, Eq. 2-3) ------------------ */

double oracle_verifier_fraction(const double* gen, const double* ref, int64_t n,
                                double eps_switch, double tau) {
  if (n <= 0) return 0.0;
  int64_t over = 0;
  for (int64_t i = 0; i < n; ++i) {
    double g = gen[i], r = ref[i];
    if (isnan(g) || isnan(r)) { if (!(isnan(g) && isnan(r))) ++over; continue; }
    if (isinf(g) || isinf(r)) { if (g != r) ++over; continue; }
    double e = fabs(g - r);
    if (fabs(r) > eps_switch) e /= fabs(r);
    if (e > tau) ++over;
  }
  return (double)over / (double)n;
}

int oracle_last_threads(void) { return g_last_threads; }
