/*
 * akg.h - C ABI of the B200 (sm_100a) row-operator library.
 *
 * Last-axis reduce-then-normalise operators over a row-major matrix
 * X[rows, cols]: softmax, log-softmax, LayerNorm, RMSNorm, with optional
 * additive and/or causal masking for the softmax pair.  One fused kernel per
 * call: every live input element is read from HBM once and every output
 * element written once.  fp32, bf16 or fp16 storage; all arithmetic in fp32; a bf16
 * result is rounded once (nearest-even) at the store.
 *
 * General rules for every entry point
 *   - Pointers named x, y, gamma, beta, weight and akg_mask.additive are DEVICE
 *     pointers on the current device unless the function name ends in _host.
 *     The caller owns every buffer; the library allocates no device memory.
 *   - Strides are in ELEMENTS and must be >= cols.  Vectors (gamma, beta,
 *     weight) hold cols contiguous elements of the same dtype as x.
 *   - The call validates its arguments, enqueues work on `stream` (a
 *     cudaStream_t passed as void*; NULL = the legacy default stream) and
 *     returns without synchronising.  It never throws, aborts or changes the
 *     current device.  Calls from several host threads are safe.
 *   - rows == 0 or cols == 0 is AKG_OK with nothing launched.  Any alignment of
 *     pointers and strides is accepted: 16-byte aligned rows select vectorised
 *     kernels, anything else a scalar kernel with the same results.
 *   - In place (y == x with equal strides) is allowed, and so are two column
 *     windows of one buffer that share no element (x = buf[:, :cols], y = buf[:, cols:]
 *     with the same row stride); any other overlap of x and y is
 *     AKG_ERR_INVALID_ARG.
 *   - On AKG_ERR_INVALID_ARG / AKG_ERR_UNSUPPORTED nothing has been launched.
 *     AKG_ERR_CUDA reports a failed launch (the CUDA error is consumed; its
 *     text is available from akg_last_error_string on the same thread).
 */
#ifndef AKG_H_
#define AKG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum akg_status {
  AKG_OK = 0,
  AKG_ERR_INVALID_ARG = 1,
  AKG_ERR_UNSUPPORTED = 2,
  AKG_ERR_CUDA = 3,
  AKG_ERR_DEVICE_TIMEOUT = 4
} akg_status;

/* Storage types.  AKG_F16 (IEEE half, the paper's float16 regime of Section 4.1) behaves like
 * AKG_BF16 everywhere: widened once, fp32 arithmetic, one round-to-nearest-even at the store
 * (a result beyond 65504 becomes an infinity, as the conversion says). */
typedef enum akg_dtype { AKG_F32 = 0, AKG_BF16 = 1, AKG_F16 = 2 } akg_dtype;

/* Kernel families (for akg_set_variant; AKG_VARIANT_AUTO lets the library choose).
 *   STREAM  scalar loads, any alignment, statistics pass + second read of the row
 *   REG     row held in registers, 128-bit loads, warp- or CTA-per-row
 *   TMA     persistent CTAs, rows staged in a shared-memory ring by bulk-copy engine
 *   CLUSTER one thread-block cluster per row, row resident in the cluster's shared
 *           memory, partial statistics exchanged through distributed shared memory */
typedef enum akg_variant {
  AKG_VARIANT_AUTO = 0,
  AKG_VARIANT_STREAM = 1,
  AKG_VARIANT_REG = 2,
  AKG_VARIANT_TMA = 3,
  AKG_VARIANT_CLUSTER = 4
} akg_variant;

/* Mask for the softmax pair (pass NULL for "no mask").  Not part of the paper;
 * defined by this library:
 *   z[r,c] = x[r,c] + additive[(r % add_rows) * add_row_stride + c]    if additive != NULL
 *   z[r,c] = -inf   where  c > (r % causal_period) + causal_offset     if causal != 0
 * The causal rule is applied from indices: masked input elements are never read
 * and may hold anything.  additive has the dtype of x; -inf entries are allowed. */
typedef struct akg_mask {
  const void* additive;     /* device pointer or NULL                              */
  int64_t add_rows;         /* >= 1 when additive != NULL                          */
  int64_t add_row_stride;   /* elements, >= cols                                   */
  int32_t causal;           /* 0 or 1                                              */
  int64_t causal_period;    /* P >= 1 when causal                                  */
  int64_t causal_offset;    /* normally 0; may be negative                         */
} akg_mask;

/* Softmax over the last axis ("Softmax" in the reduction category, Section 3.6;
 * textbook definition).  Per row, with z the masked input and L = {c: z_c > -inf}:
 *   y_c = exp(z_c - max z) / sum_c exp(z_c - max z);   y_c = +0 for c not in L.
 * A row with no live entry yields +0 everywhere, bit-exactly.  A live NaN, or a
 * +inf maximum, makes the whole row NaN. */
akg_status akg_softmax(const void* x, void* y, int64_t rows, int64_t cols,
                       int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                       const akg_mask* mask, void* stream);

/* Log-softmax over the last axis: y_c = (z_c - max z) - ln sum_c exp(z_c - max z),
 * i.e. x - logsumexp(x); y_c = -inf for masked entries; a row with no live entry
 * yields -inf everywhere.  NaN rule as for akg_softmax.  Same arguments. */
akg_status akg_log_softmax(const void* x, void* y, int64_t rows, int64_t cols,
                           int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                           const akg_mask* mask, void* stream);

/* LayerNorm over the last axis (the operator whose statistics and normalisation
 * the paper's Section 4.3 describes as fused into one kernel):
 *   mu = mean(x), var = mean((x - mu)^2) (biased),
 *   y_c = (x_c - mu) / sqrt(var + eps) * gamma_c + beta_c.
 * gamma == NULL means 1, beta == NULL means 0.  eps >= 0 (NaN is rejected). */
akg_status akg_layernorm(const void* x, void* y, int64_t rows, int64_t cols,
                         int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                         const void* gamma, const void* beta, float eps, void* stream);

/* RMSNorm over the last axis (the Unified Sketch figure of Section 3.2.1: sum of
 * squares, divided by the axis length, eps added, square root, divide):
 *   y_c = x_c / sqrt(mean(x^2) + eps) * weight_c;  weight == NULL means 1. */
akg_status akg_rmsnorm(const void* x, void* y, int64_t rows, int64_t cols,
                       int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                       const void* weight, float eps, void* stream);

typedef enum akg_op {
  AKG_OP_SOFTMAX = 0,
  AKG_OP_LOG_SOFTMAX = 1,
  AKG_OP_LAYERNORM = 2,
  AKG_OP_RMSNORM = 3
} akg_op;

/* Any of the four operators above on HOST buffers (no counterpart in the paper; the
 * operator definitions are the ones cited at akg_softmax .. akg_rmsnorm).
 *   x_host, y_host, gamma_host, beta_host : HOST pointers (page-locked memory lets the
 *     copies overlap; pageable memory works but serialises).  gamma_host is the
 *     RMSNorm weight; beta_host is used by LayerNorm only; mask (softmax pair only)
 *     may carry the causal rule, an additive mask is AKG_ERR_UNSUPPORTED here.
 *   workspace : DEVICE pointer, 16-byte aligned, workspace_bytes long, owned by the
 *     caller; the library allocates no device memory.  Any size from
 *     3 * round_up(cols * element size, 256) (+ the vectors) works; the size returned
 *     by akg_host_workspace_bytes lets copies and kernels overlap fully.
 * The rows are cut into chunks; chunk i is copied host -> workspace slot (i mod 3),
 * processed in place by the same kernels as the device entry points, and copied back,
 * on one of three internal streams, so uploads, kernels and downloads of different
 * chunks overlap.  The work is ordered after everything already enqueued on `stream`,
 * and `stream` waits for it; the call itself returns without synchronising (the host
 * buffers and the workspace must stay valid until `stream` has caught up).  In place
 * (y_host == x_host, equal strides) is allowed.  Calls on the same device are
 * serialised by an internal lock while they enqueue.  Errors as for the device entry
 * points; a workspace that is NULL, misaligned or too small is AKG_ERR_INVALID_ARG. */
akg_status akg_rowop_host(akg_op op, const void* x_host, void* y_host, int64_t rows, int64_t cols,
                          int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                          const void* gamma_host, const void* beta_host, float eps,
                          const akg_mask* mask, void* workspace, size_t workspace_bytes, void* stream);

/* Workspace size (bytes) with which akg_rowop_host pipelines about a dozen chunks of
 * at least 4 MiB; 0 for a malformed shape. */
size_t akg_host_workspace_bytes(int64_t rows, int64_t cols, akg_dtype dtype, int has_gamma, int has_beta);

/* The same four operators over a NON-last axis: x and y are [outer, reduce, inner]
 * DEVICE arrays with inner contiguous; element (b, f, d) is at
 * b * outer_stride + f * reduce_stride + d (strides in elements,
 * reduce_stride >= inner, outer_stride >= (reduce - 1) * reduce_stride + inner).
 * This is the layout of the paper's RMSNorm sketch (Unified Sketch figure, Section
 * 3.2.1: X[B, F, D1, D2] reduced over F, i.e. outer = B, reduce = F, inner = D1 * D2).
 * For every (b, d) the `reduce` values along f are one row of the operator:
 *   RMSNorm    y = x / sqrt(mean_f(x^2) + eps) * gamma[f]        (the sketch, gamma = NULL)
 *   LayerNorm  y = (x - mean_f) / sqrt(var_f + eps) * gamma[f] + beta[f]
 *   softmax / log-softmax over f (no masks on this entry point)
 * gamma / beta: DEVICE vectors of `reduce` elements of x's dtype, indexed by f, or NULL
 * (1 / 0); ignored by the softmax pair.  One kernel: a reduced axis of up to 128 entries is
 * held in registers, a longer one takes two passes, the second served by L2; either way HBM
 * sees each element once in and once out.  16-byte aligned bases and strides with inner a
 * multiple of the vector width take 128-bit accesses, anything else a scalar path with the
 * same results.  In place (y == x, equal strides) is allowed.
 * Enqueues on `stream` and returns; errors as for the last-axis entry points. */
akg_status akg_rowop_axis(akg_op op, const void* x, void* y, int64_t outer, int64_t reduce, int64_t inner,
                          int64_t x_outer_stride, int64_t x_reduce_stride, int64_t y_outer_stride,
                          int64_t y_reduce_stride, akg_dtype dtype, const void* gamma, const void* beta,
                          float eps, void* stream);

/* Softmax / log-softmax with a fused pre-scale (a "fused variant", Section 3.6; the paper
 * gives no formula: this is the attention form softmax(scale * scores + mask)):
 *   z[r,c] = scale * x[r,c] + additive[...]  (the additive mask is NOT scaled), causal rule as
 *   for akg_softmax; y = softmax(z) if log_output == 0, log-softmax(z) otherwise.
 * scale must be finite and > 0 (AKG_ERR_INVALID_ARG otherwise).  Everything else - masks,
 * special rows, strides, alignment, in place, errors - as for akg_softmax / akg_log_softmax;
 * scale == 1 gives bit-identical results to them.  The scale costs no extra instruction:
 * the kernels fold it into the constant of the exponential. */
akg_status akg_softmax_scaled(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                              int64_t y_row_stride, akg_dtype dtype, float scale, const akg_mask* mask,
                              int log_output, void* stream);

/* Fused residual add + normalisation over the last axis (one of the "fused variants" of the
 * paper's operator benchmark, Section 3.6; the paper gives no formula, this is the usual
 * pre-norm residual step):
 *   s = x + residual;   sum_out = s;   y = LayerNorm(s) or RMSNorm(s)
 * op is AKG_OP_LAYERNORM or AKG_OP_RMSNORM, with the definitions, gamma / beta (beta ignored
 * by RMSNorm) and eps of akg_layernorm / akg_rmsnorm.  x, residual, y, sum_out: DEVICE
 * matrices [rows, cols] of `dtype`, each with its own row stride in elements (>= cols).
 * The sum is formed in fp32 from the widened operands; the normalisation sees that fp32
 * sum, sum_out receives it rounded once to `dtype`.  sum_out may be NULL (the sum is then
 * not stored).  Aliasing: y and sum_out may each be exactly x or exactly residual (same base
 * and stride - e.g. sum_out == residual updates the residual stream in place, y == x
 * overwrites the branch input) or disjoint from them; y and sum_out must not overlap each
 * other; x and residual may overlap freely.  Rows of a whole number of 16-byte vectors per
 * thread (cols a multiple of 128 fp32 / 256 bf16 elements, up to 32768 / 65536, everything
 * 16-byte aligned) move every byte once; other shapes take a scalar two-pass kernel with
 * the same results.  Enqueues on `stream` and returns; errors as for akg_layernorm, plus
 * AKG_ERR_INVALID_ARG for a NULL residual or a forbidden overlap. */
akg_status akg_add_norm(akg_op op, const void* x, const void* residual, void* y, void* sum_out,
                        int64_t rows, int64_t cols, int64_t x_row_stride, int64_t res_row_stride,
                        int64_t y_row_stride, int64_t sum_row_stride, akg_dtype dtype,
                        const void* gamma, const void* beta, float eps, void* stream);

/* Gated activations "SiLU-and-Mul" / "GELU-and-Mul" (named among the operators of the paper's
 * benchmark, Section 3.6; textbook formulas).  x: DEVICE matrix [rows, 2 d] with row stride
 * x_row_stride >= 2 d elements; the first d columns of a row are the gate a, the last d the
 * factor b.  y: DEVICE matrix [rows, d], row stride y_row_stride >= d:
 *   y[r, c] = act(a[r, c]) * b[r, c]
 *   AKG_ACT_SILU       act(a) = a / (1 + e^-a)
 *   AKG_ACT_GELU       act(a) = 0.5 a (1 + erf(a / sqrt 2))
 *   AKG_ACT_GELU_TANH  act(a) = 0.5 a (1 + tanh(sqrt(2 / pi) (a + 0.044715 a^3)))
 * fp32 arithmetic on the widened inputs, one rounding at the store.  y may be x itself with
 * the same row stride (the result replaces the gate half); any other overlap is
 * AKG_ERR_INVALID_ARG.  16-byte aligned bases and strides with d a multiple of the vector
 * width take 128-bit accesses, anything else a scalar path with the same results.  Enqueues
 * on `stream` and returns; errors as for the other entry points. */
typedef enum akg_act { AKG_ACT_SILU = 0, AKG_ACT_GELU = 1, AKG_ACT_GELU_TANH = 2 } akg_act;
akg_status akg_act_mul(akg_act act, const void* x, void* y, int64_t rows, int64_t d,
                       int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype, void* stream);

/* Arg-max (want_min == 0) or arg-min (want_min == 1) over the last axis ("argmax/argmin" of the
 * reduction category, Section 3.6).  x: DEVICE matrix [rows, cols] of `dtype`; index_out: DEVICE
 * vector of `rows` int64.  index_out[r] = the smallest column at which row r attains its maximum
 * (minimum).  Values are compared exactly as stored: -0 equals +0, and a NaN counts as the extreme
 * for both operators (the first NaN of a row wins), as in numpy and torch.  cols == 0 with
 * rows > 0 is AKG_ERR_INVALID_ARG.  Reads every element once; any alignment. */
akg_status akg_argreduce(int want_min, const void* x, int64_t* index_out, int64_t rows, int64_t cols,
                         int64_t x_row_stride, akg_dtype dtype, void* stream);

/* Cumulative sum (want_prod == 0) or product (want_prod == 1) along the last axis ("cumulative
 * operations" of the reduction category, Section 3.6), inclusive:
 *   y[r, c] = x[r, 0] (+ or *) ... (+ or *) x[r, c].
 * One pass (each element read once, written once), fp32 arithmetic, one rounding at the store.
 * The partial results are combined as a tree (vector, warp, CTA, chunk), not left to right: the
 * rounding differs from a sequential loop by the usual O(log cols) ulps of the running magnitude,
 * and a product whose sequential partials stay finite may overflow in a tree partial.  In place
 * (y == x, equal strides) is allowed; any alignment. */
akg_status akg_cumulative(int want_prod, const void* x, void* y, int64_t rows, int64_t cols,
                          int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype, void* stream);

/* BatchNorm-style column normalisation (BatchNorm is among the operators the paper's benchmark
 * lists, Section 3.6; the training-mode forward with batch statistics): for every column c of the
 * DEVICE matrix x[rows, cols]
 *   mean_c = sum_r x[r,c] / rows,   var_c = sum_r (x[r,c] - mean_c)^2 / rows   (biased),
 *   y[r,c] = (x[r,c] - mean_c) / sqrt(var_c + eps) * gamma_c + beta_c.
 * gamma / beta: DEVICE vectors of cols elements of `dtype`, or NULL (1 / 0).  mean_out / var_out:
 * DEVICE vectors of cols floats that receive the statistics, or NULL.  workspace: DEVICE memory,
 * 8-byte aligned, owned by the caller, not read before it is written; the size returned by
 * akg_colnorm_workspace_bytes (blocks * cols * 8 bytes with at most 256 blocks: about 1 MiB for a
 * thousand columns) lets the rows be cut into enough blocks to fill the GPU, a smaller one (at
 * least cols * 8 bytes) into fewer.  Two kernels are enqueued on `stream` (statistics per row block, then merge
 * and normalise); x is read twice, the second time from L2 while the matrix fits there.  In place
 * (y == x, equal strides) is allowed; any alignment; errors as for akg_layernorm, plus
 * AKG_ERR_INVALID_ARG for a NULL, misaligned or too small workspace. */
akg_status akg_colnorm(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                       int64_t y_row_stride, akg_dtype dtype, const void* gamma, const void* beta, float eps,
                       float* mean_out, float* var_out, void* workspace, size_t workspace_bytes, void* stream);
size_t akg_colnorm_workspace_bytes(int64_t rows, int64_t cols);

/* Size of the staging area built into the library (see akg_rowop_host_static). */
#define AKG_STATIC_STAGING_BYTES (16u << 20)

/* akg_rowop_host for callers that cannot provide a device workspace (the paper has no
 * counterpart: this is a convenience of this library).  Meant for code that is given
 * host buffers and a stream but no way to allocate device memory: a plug-in inside an
 * application whose memory pool it may not touch, a service that must not allocate
 * after start-up, a host-only component of a larger pipeline.  Same operators, same
 * arguments and the same results as akg_rowop_host, minus the workspace: the chunks are
 * staged in a fixed area of AKG_STATIC_STAGING_BYTES (16 MiB) that is part of the
 * library image.  Every GPU on which the library is loaded holds that area until the
 * process exits, whether or not this function is ever called.
 *   - Nothing is allocated or freed here or in anything this function calls, and no
 *     streams or events are created: uploads, kernels and downloads run one after the
 *     other on `stream` (no overlap between them; use akg_rowop_host for throughput).
 *   - Size limit: one row plus gamma / beta must fit the area, i.e.
 *     round_up(cols * element size, 256) * (1 + number of vectors) <=
 *     AKG_STATIC_STAGING_BYTES; a longer row is AKG_ERR_UNSUPPORTED with a message
 *     naming the limit, and nothing is enqueued.  Any number of rows is fine.
 *   - The first call on each device looks up the device address of the area (with that
 *     device current) and keeps it; make that first call outside any stream capture.
 *   - The area is shared by all calls on the device and keeps the previous call's data.
 *     Nothing in it needs clearing (every chunk is overwritten by its upload before a
 *     kernel reads it), but two calls whose work overlaps on the GPU, from different
 *     streams or threads, race on it: keep such calls on one stream, or order them.
 * Errors otherwise as for akg_rowop_host. */
akg_status akg_rowop_host_static(akg_op op, const void* x_host, void* y_host, int64_t rows, int64_t cols,
                                 int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                                 const void* gamma_host, const void* beta_host, float eps,
                                 const akg_mask* mask, void* stream);

/* Human-readable name of a status code (static storage, never NULL). */
const char* akg_status_string(akg_status status);

/* Text of the most recent failure on the calling thread ("" if none). */
const char* akg_last_error_string(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int akg_version(void);

/* Force a kernel family for subsequent calls from any thread (testing and
 * benchmarking aid).  A forced family that cannot run the given call (alignment,
 * row length) makes that call return AKG_ERR_UNSUPPORTED.  Returns
 * AKG_ERR_INVALID_ARG for an unknown value.  AKG_VARIANT_AUTO restores choice. */
akg_status akg_set_variant(akg_variant variant);

/* Override one launch-geometry choice for subsequent calls (benchmarking aid; 0
 * restores the library's own choice).  Keys: "reg_threads", "reg_vpt" (CTA size and
 * 16-byte vectors per thread of the register-resident family; both must be set),
 * for akg_cumulative "reg_vpt" 1 / 3 is how many chunks ahead of the scan a CTA per row loads),
 * "reg_group" (32 = a warp per row, 1 = a CTA per row), "grid_cap" (maximum CTAs;
 * rows beyond it are taken in a grid-stride loop); for the shared-memory ring
 * families "cluster_size" (CTAs per row: 1, 2, 4, 8, 16), "smem_nbuf" (ring depth
 * limit), "smem_threads" (256, 512, 1024), "smem_ctas" (CTAs per SM the ring is
 * sized for), "tma_mode" (1 = ring-fed register kernels, 2 = shared-memory passes),
 * "cluster_mode" (1 = row resident in the cluster's shared memory, 2 = two streaming
 * passes with the second served by L2, 3 = unmasked softmax rows resident in the cluster's
 * registers), "reg_general" (1 = never the predicate-free
 * normalisation kernel), "interleave" (1 = visit causal rows short/long alternately),
 * "host_chunks", "host_min_kib" (host-buffer entry point: chunks per call, smallest chunk),
 * "host_full_upload" (1 = upload the masked columns of causal rows too),
 * "split_exchange" (two-pass cluster kernel: 1 = partial statistics exchanged under a
 * cluster barrier per row instead of st.async + mbarrier), "split_l2" (its L2 priority
 * scheme: 1 = no "keep" marks, 2 = marks without demotion), "reg_flex" (register family:
 * 1 = the runtime-thread-count normalisation kernel also where a fixed shape fits, 2 = never
 * a runtime-thread-count kernel, 4 = no eight-vector threads for 16-bit RMSNorm, 5 = never
 * the packed 16-bit / fp32 runtime-thread-count kernels), "packed_vpt" (vectors per thread of
 * those kernels, 2 .. 8), "pdl" (1 = programmatic dependent launch also for cluster launches,
 * 2 = never), "axis_r", "axis_nc", "axis_mode", "axis_lc" (non-last-axis kernels: rows per
 * thread, column blocks per CTA, lane layout, lanes along the columns).  Two keys exist for the test
 * of the failure path only: "test_wait_us" (limit of the kernels' bounded waits in
 * microseconds; 0 = two seconds) and "test_no_copies" (1 = the ring kernels issue no
 * bulk copy, so that every wait on one runs out and the call reports
 * AKG_ERR_DEVICE_TIMEOUT through akg_device_status).
 * A geometry the library was not
 * built for makes the next call return AKG_ERR_CUDA.  Unknown key:
 * AKG_ERR_INVALID_ARG. */
akg_status akg_set_tuning(const char* key, int value);

/* Name of the kernel family and geometry the last successful call on this thread
 * launched, e.g. "reg<f32,t256,v4>" (static/thread-local storage). */
const char* akg_last_kernel_name(void);

/* Bytes that the last akg_rowop_host call on this thread copied from host to device and from
 * device to host (either pointer may be NULL).  The upload is smaller than the matrix under a
 * causal mask: the masked columns of a row are never read by the kernels, so they are not sent
 * either (chunks lie inside a causal period and carry the columns up to their last row's live
 * length).  Always returns AKG_OK. */
akg_status akg_last_host_copy_bytes(size_t* h2d_bytes, size_t* d2h_bytes);

/* Reads the device-side status word of the current device (synchronises with
 * the device).  0 = clean; non-zero = a bounded wait (on a bulk copy, or on the
 * partial statistics of a cluster peer) ran out in some kernel since the last
 * call; the word is reset to 0 by this call.  Every such wait is limited to two
 * seconds of the device's global timer.  A CTA whose wait ran out stores nothing
 * from then on, issues no further copy and still takes part in its barriers, so the
 * kernel ends by itself and the context stays usable; the output of that call is
 * undefined (partly written).  Returns AKG_OK, AKG_ERR_DEVICE_TIMEOUT, or
 * AKG_ERR_CUDA. */
akg_status akg_device_status(int* word_out);

#ifdef __cplusplus
}
#endif
#endif /* AKG_H_ */
