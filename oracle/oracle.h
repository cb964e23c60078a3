/*
 * oracle.h - plain fp64 CPU definitions of the last-axis reduce-then-normalise
 * operators (softmax, log-softmax, LayerNorm, RMSNorm, additive / causal mask).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may call it.  It shares no code,
 * header, table or helper with the CUDA library and neither includes the other.
 *
 * Every function works on host memory, one row at a time, in double precision,
 * as the textbook definition written out (sums are Neumaier-compensated so the
 * oracle's own rounding stays near 1e-16 relative).  Where the paper speaks
 * (RMSNorm: sum of squares over the reduced axis, divided by its length, eps
 * added to that mean, square root, then divide - the Unified Sketch figure of
 * Section 3.2.1) the oracle follows it; softmax and LayerNorm are only named by
 * the paper (Section 3.6, Section 4.3) and take their textbook definitions;
 * log-softmax and masking come from the build contract.
 *
 * Parity status: every function below is pinned by tests that run without a GPU
 * (hand-derived worked examples, closed forms, invariants, fp64 library
 * routines, 40-digit brute force).  Nothing here is "parity unpinned".
 */
#ifndef ORACLE_H_
#define ORACLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* storage types of the input arrays */
enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F64 = 2, ORACLE_F16 = 3 };  /* F16: IEEE binary16 */

/* Mask descriptor (NULL pointer = no mask).
 *   z[r,c] = x[r,c] + additive[(r % add_rows) * add_row_stride + c]   (if additive != NULL)
 *   z[r,c] = -inf  where  c > (r % causal_period) + causal_offset      (if causal != 0)
 * r is the GLOBAL row index (row_ids[i] when row_ids is given).
 * The additive array has the same storage type as x. */
typedef struct oracle_mask {
  const void* additive;
  int64_t add_rows;
  int64_t add_row_stride;
  int32_t causal;
  int64_t causal_period;
  int64_t causal_offset;
} oracle_mask;

/* ---- single-row cores on doubles (n >= 1) ------------------------------- */

/* softmax of z[0..n): live set L = {c : z_c > -inf}.
 *   any NaN in z, or max z = +inf  -> every output NaN
 *   L empty                        -> every output +0
 *   else m = max z, s = sum exp(z_c - m), y_c = exp(z_c - m) / s           */
void oracle_softmax_row(const double* z, int64_t n, double* y);

/* log-softmax: y_c = (z_c - m) - ln s; -inf where z_c = -inf;
 *   L empty -> every output -inf; NaN rule as for softmax.                 */
void oracle_log_softmax_row(const double* z, int64_t n, double* y);

/* logsumexp(z) = m + ln s (same special cases: -inf if L empty, NaN rule). */
double oracle_logsumexp_row(const double* z, int64_t n);

/* LayerNorm: mu = sum x / n; var = sum (x-mu)^2 / n (biased);
 *   y_c = (x_c - mu) / sqrt(var + eps) * gamma_c + beta_c
 *   gamma == NULL -> 1, beta == NULL -> 0.                                 */
void oracle_layernorm_row(const double* x, int64_t n, const double* gamma,
                          const double* beta, double eps, double* y);

/* RMSNorm (Unified Sketch figure, Section 3.2.1): ms = sum x^2 / n;
 *   y_c = x_c / sqrt(ms + eps) * w_c;  w == NULL -> 1.                     */
void oracle_rmsnorm_row(const double* x, int64_t n, const double* w,
                        double eps, double* y);

/* ---- array drivers -------------------------------------------------------
 * x: rows x cols elements of storage type dtype, row i starts at x + i*x_stride
 * (elements).  row_ids: NULL -> global row index of row i is i; otherwise
 * row_ids[i] (used only by the mask).  out: rows x cols doubles, contiguous.
 * nthreads <= 1: serial; > 1: rows are divided among that many OpenMP threads
 * (rows are independent; the per-row arithmetic is unchanged).
 * Return 0 on success, 1 on a malformed argument.                          */
int oracle_softmax(const void* x, int dtype, int64_t rows, int64_t cols,
                   int64_t x_stride, const int64_t* row_ids,
                   const oracle_mask* mask, double* out, int nthreads);
int oracle_log_softmax(const void* x, int dtype, int64_t rows, int64_t cols,
                       int64_t x_stride, const int64_t* row_ids,
                       const oracle_mask* mask, double* out, int nthreads);
/* The same pair with a fused pre-scale (a "fused variant", Section 3.6; the attention form
 * softmax(scale * scores + mask)): z = scale * x, then the additive mask (not scaled) and the
 * causal rule as above, then softmax (want_log 0) or log-softmax (want_log 1) of z.
 * scale must be finite and > 0. */
int oracle_softmax_scaled(const void* x, int dtype, int64_t rows, int64_t cols,
                          int64_t x_stride, double scale, const int64_t* row_ids,
                          const oracle_mask* mask, int want_log, double* out, int nthreads);
int oracle_layernorm(const void* x, int dtype, int64_t rows, int64_t cols,
                     int64_t x_stride, const void* gamma, const void* beta,
                     double eps, double* out, int nthreads);
int oracle_rmsnorm(const void* x, int dtype, int64_t rows, int64_t cols,
                   int64_t x_stride, const void* weight, double eps,
                   double* out, int nthreads);

/* ---- reduction over a NON-last axis -----------------------------------------
 * The layout of the paper's RMSNorm sketch (Unified Sketch figure, Section 3.2.1):
 * X[B, F, D1, D2] reduced over F.  Here x is [outer, reduce, inner] with inner
 * (= D1 * D2) contiguous: element (b, f, d) sits at b*outer_stride + f*reduce_stride + d
 * (strides in elements).  For every (b, d) the `reduce` values along f form one row of
 * the operator op (0 softmax, 1 log-softmax, 2 LayerNorm, 3 RMSNorm; no masks);
 * gamma / beta (LayerNorm) or gamma as the weight (RMSNorm) have `reduce` elements of x's
 * storage type and are indexed by f; NULL means 1 / 0.
 * out: outer x reduce x inner doubles, contiguous.  Returns 0, or 1 on a bad argument. */
int oracle_rowop_axis(int op, const void* x, int dtype, int64_t outer, int64_t reduce, int64_t inner,
                      int64_t outer_stride, int64_t reduce_stride, const void* gamma, const void* beta,
                      double eps, double* out, int nthreads);

/* Fused residual add + normalisation, one of the "fused variants" the paper's operator
 * benchmark lists (Section 3.6): s = x + res element by element, out_sum = s, and
 * out_y = LayerNorm(s) (op 2) or RMSNorm(s) (op 3) over the last axis, with the
 * definitions of oracle_layernorm / oracle_rmsnorm (gamma doubles as the RMSNorm weight;
 * beta is ignored by RMSNorm).  x and res share dtype and shape [rows, cols] with their own
 * row strides; the normalisation sees the unrounded sum.  out_y, out_sum: rows x cols
 * doubles, contiguous.  Returns 0, or 1 on a bad argument. */
int oracle_add_norm(int op, const void* x, const void* res, int dtype, int64_t rows, int64_t cols,
                    int64_t x_stride, int64_t res_stride, const void* gamma, const void* beta,
                    double eps, double* out_y, double* out_sum, int nthreads);

/* Gated activations, "SiLU-and-Mul" and "GELU-and-Mul" of the paper's operator benchmark
 * (Section 3.6 names them; the formulas are the textbook ones).  x is [rows, 2 d] with row
 * stride x_stride >= 2 d: the first d columns are the gate a, the last d the factor b;
 * out[i, c] = act(a[i, c]) * b[i, c], rows x d doubles, contiguous.
 *   act 0: SiLU   a / (1 + e^-a)
 *   act 1: GELU   a * Phi(a) = 0.5 a (1 + erf(a / sqrt 2))
 *   act 2: GELU, tanh form   0.5 a (1 + tanh(sqrt(2 / pi) (a + 0.044715 a^3)))
 * Returns 0, or 1 on a bad argument. */
double oracle_activation(int act, double a);
int oracle_act_mul(int act, const void* x, int dtype, int64_t rows, int64_t d, int64_t x_stride,
                   double* out, int nthreads);

/* Arg-max / arg-min over the last axis ("argmax/argmin" of the reduction category, Section
 * 3.6).  out[i] = the smallest column index at which row i attains its maximum (want_min 0) or
 * minimum (want_min 1).  Comparisons are made on the stored values, exactly: -0 and +0 are
 * equal; a NaN counts as the extreme for both (the first NaN of a row wins), as in numpy and
 * torch.  cols == 0 with rows > 0 is an error (no index exists).  Returns 0, or 1. */
int oracle_argreduce(int want_min, const void* x, int dtype, int64_t rows, int64_t cols, int64_t x_stride,
                     int64_t* out, int nthreads);

/* Cumulative sum (want_prod 0) or product (want_prod 1) along the last axis ("cumulative
 * operations", Section 3.6): out[i, c] = x[i, 0] (+ or *) ... (+ or *) x[i, c], inclusive,
 * in double (the sum compensated).  out: rows x cols doubles, contiguous.  Returns 0, or 1. */
int oracle_cumulative(int want_prod, const void* x, int dtype, int64_t rows, int64_t cols, int64_t x_stride,
                      double* out, int nthreads);

/* BatchNorm-style column statistics (BatchNorm is among the operators Section 3.6 lists; the
 * formula is the textbook training-mode forward): for every column c of x[rows, cols]
 *   mean_c = sum_r x[r,c] / rows,  var_c = sum_r (x[r,c] - mean_c)^2 / rows  (biased),
 *   y[r,c] = (x[r,c] - mean_c) / sqrt(var_c + eps) * gamma_c + beta_c   (NULL: 1 / 0).
 * out_y: rows x cols doubles; out_mean / out_var: cols doubles each or NULL.  Returns 0 or 1. */
int oracle_colnorm(const void* x, int dtype, int64_t rows, int64_t cols, int64_t x_stride,
                   const void* gamma, const void* beta, double eps, double* out_y, double* out_mean,
                   double* out_var, int nthreads);

/* The exact value of n stored elements as doubles (how every driver reads its input). */
int oracle_widen(const void* base, int dtype, int64_t n, double* out);

/* The paper's correctness criterion (Section 3.2.3, Eq. 2-3): element error is
 * |gen-ref|/|ref| when |ref| > eps_switch, else |gen-ref|; returns the fraction
 * of elements whose error exceeds tau (the kernel passes iff that fraction is
 * <= tau).  Elements where both are NaN, or both the same infinity, count as
 * error 0; a NaN/inf mismatch counts as exceeding tau.                     */
double oracle_verifier_fraction(const double* gen, const double* ref, int64_t n,
                                double eps_switch, double tau);

/* number of OpenMP threads the last array driver call actually used */
int oracle_last_threads(void);

#ifdef __cplusplus
}
#endif
#endif /* ORACLE_H_ */
