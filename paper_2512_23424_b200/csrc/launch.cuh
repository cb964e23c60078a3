// Host-side launch plan and the per-operator launcher template.  Each operator's
// translation unit instantiates launch_op<OP> once, so the four operators compile in
// parallel; api.cu sees only the declarations.
#pragma once

#include <cuda_runtime.h>

#include "common.cuh"

namespace akg {

enum Variant : int { V_AUTO = 0, V_STREAM = 1, V_REG = 2, V_TMA = 3, V_CLUSTER = 4 };

struct LaunchPlan {
  int variant;        // V_STREAM .. V_CLUSTER
  int threads;        // CTA size
  int group;          // threads per row (32 or threads) for V_REG
  int vpt;            // 16-byte vectors per thread for V_REG
  unsigned grid;      // CTAs (V_CLUSTER: a multiple of cluster)
  int cluster;        // CTAs per cluster (V_CLUSTER), else 1
  int stages;         // ring depth (V_TMA)
  size_t smem;        // dynamic shared memory per CTA
  int mode;           // V_TMA: 1 = register kernels fed by a ring, 0 = shared-memory-resident kernel
  int pdl;            // 1 = launch with programmatic stream serialisation (see pdl_prologue)
  int split_l2;       // two-pass split kernel: L2 priority scheme (0 = default, see split_kernel)
};

template <int OP>
cudaError_t launch_op(const LaunchPlan& plan, int dtype, const RowParams& p, cudaStream_t stream);

// Two-pass non-last-axis kernel (op_axis.cu), 256 threads.  vec: 16-byte vectors along the
// inner axis are usable.  A warp lies 1 << lc_shift lanes along the columns and the rest along
// rows; strips_per_outer counts strips of (1 << lc_shift) lanes; grid as for launch_axis_reg.
cudaError_t launch_axis(int op, int dtype, bool vec, const AxisParams& p, dim3 grid, unsigned strips_per_outer,
                        int lc_shift, int pdl, cudaStream_t stream);

// Register-resident non-last-axis kernel (op_axis_reg.cu): a CTA of nf x nc warps, nf
// along the reduced axis with r rows per thread (reduce <= nf * r, r in {2, 4, 8}), nc
// column blocks of 32 lanes.  mode: what a lane holds of a row - 0 one element, 1 one 16-byte
// vector, 2 (bf16) one 8-byte vector widened to floats; axis_reg_width gives its elements.
// strips_per_outer counts strips of nc * 32 lanes; grid = (strips of one outer index, outer
// indices), either may be smaller.
int axis_reg_width(int dtype, int mode);
cudaError_t launch_axis_reg(int op, int dtype, int mode, int r, const AxisParams& p, dim3 grid,
                            unsigned strips_per_outer, int nf, int nc, int pdl, cudaStream_t stream);

// Fused residual add + LayerNorm / RMSNorm (op_fused.cu): a CTA of `threads` (a multiple of 32)
// per row of exactly threads * vpt 16-byte vectors; p.res / p.sum carry the extra streams.
cudaError_t launch_add_norm(int op, int dtype, int vpt, int threads, const RowParams& p, unsigned grid, int pdl,
                            cudaStream_t stream);

// Gated activations (op_act.cu).  act: 0 SiLU, 1 GELU, 2 GELU tanh form.  vec: 16-byte vectors.
// grid = (chunks of act_mul_unroll() * threads lanes of one row, rows), either may be smaller.
int act_mul_unroll();
cudaError_t launch_act_mul(int act, int dtype, bool vec, const ActParams& p, dim3 grid, int threads, int pdl,
                           cudaStream_t stream);

// Arg-max / arg-min and cumulative sum / product over the last axis (op_scan.cu).
// warp_rows: a warp per row (eight rows per CTA of 256), else a CTA per row.  Cumulative: a CTA of
// `threads` (a multiple of 32, at most 256) per row, chunks of scan_unroll() * threads vectors.
int scan_unroll();
// segments > 1: every row is cut into that many pieces of seg_vecs vectors (elements when !vec), one
// CTA each, merged by an atomic maximum on the output word (three launches).
cudaError_t launch_argreduce(bool want_min, int dtype, bool vec, bool warp_rows, const void* x, long long* out,
                             long long rows, long long cols, long long xs, unsigned grid, unsigned segments,
                             long long seg_vecs, int pdl, cudaStream_t stream);
cudaError_t launch_cumulative(bool want_prod, int dtype, bool vec, const void* x, void* y, long long rows,
                              long long cols, long long xs, long long ys, unsigned grid, int threads, bool warp_rows,
                              int pdl, cudaStream_t stream, int depth = 1);   // depth: chunks loaded ahead (1 or 3)

// Short vectorised rows (at most 4 * lanes vectors, lanes in {4, 8, 16}): 32 / lanes rows per warp, CTAs of 256.
cudaError_t launch_cumulative_short(bool want_prod, int dtype, int lanes, const void* x, void* y, long long rows,
                                    long long cols, long long xs, long long ys, unsigned grid, int pdl, cudaStream_t stream);

// Few, long rows: a cluster of `cluster` CTAs (256 threads) per row, slices of slice_vecs vectors, the carry
// of a slice from its cluster peers (scan_split_kernel); vectorised rows only.  clusters = 0: one resident wave.
cudaError_t launch_cumulative_split(bool want_prod, int dtype, const void* x, void* y, long long rows, long long cols,
                                    long long xs, long long ys, int cluster, int slice_vecs, long long clusters,
                                    int* status, unsigned wait_us, cudaStream_t stream);

// Short unmasked rows, 32 / lanes rows per warp (op_short.cu): lanes in {4, 8, 16, 32}, rows of
// up to short_max_vectors(lanes) vectors.
int short_rows_per_cta(int lanes);
int short_max_vectors(int lanes);
cudaError_t launch_short(int op, int dtype, int lanes, const RowParams& p, unsigned grid, int pdl, cudaStream_t stream);

// BatchNorm-style column normalisation (op_colnorm.cu): two kernels, grid (column strips of
// (1 << lc_shift) lanes, row blocks of p.rows_per_block rows).  colnorm_row_slots: rows a CTA walks at once.
int colnorm_row_slots(int lc_shift);
cudaError_t launch_colnorm(int dtype, bool vec, const ColParams& p, dim3 grid, int pdl, cudaStream_t stream);

extern template cudaError_t launch_op<OP_SOFTMAX>(const LaunchPlan&, int, const RowParams&, cudaStream_t);
extern template cudaError_t launch_op<OP_LOG_SOFTMAX>(const LaunchPlan&, int, const RowParams&, cudaStream_t);
extern template cudaError_t launch_op<OP_LAYERNORM>(const LaunchPlan&, int, const RowParams&, cudaStream_t);
extern template cudaError_t launch_op<OP_RMSNORM>(const LaunchPlan&, int, const RowParams&, cudaStream_t);

}  // namespace akg
