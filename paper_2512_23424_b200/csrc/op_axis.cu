// Two-pass kernels of the non-last-axis operators (any length of the reduced axis) and their
// launcher.
#include "kernels_axis.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <int OP, typename T, int MODE>
cudaError_t launch_axis_typed(const AxisParams& p, dim3 grid, unsigned spo, int lc_shift, int pdl, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kAxisThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  const int slots = kAxisThreads >> lc_shift;
  return cudaLaunchKernelEx(&cfg, axis_kernel<OP, T, MODE>, p, spo, lc_shift,
                            static_cast<int>(p.reduce / slots), static_cast<int>(p.reduce % slots));
}

template <int OP>
cudaError_t launch_axis_op(int dtype, bool vec, const AxisParams& p, dim3 grid, unsigned spo, int lc_shift, int pdl,
                           cudaStream_t s) {
  if (dtype == DT_F32)
    return vec ? launch_axis_typed<OP, float, 1>(p, grid, spo, lc_shift, pdl, s)
               : launch_axis_typed<OP, float, 0>(p, grid, spo, lc_shift, pdl, s);
  if (dtype == DT_F16)
    return vec ? launch_axis_typed<OP, __half, 1>(p, grid, spo, lc_shift, pdl, s)
               : launch_axis_typed<OP, __half, 0>(p, grid, spo, lc_shift, pdl, s);
  return vec ? launch_axis_typed<OP, __nv_bfloat16, 1>(p, grid, spo, lc_shift, pdl, s)
             : launch_axis_typed<OP, __nv_bfloat16, 0>(p, grid, spo, lc_shift, pdl, s);
}

}  // namespace

cudaError_t launch_axis(int op, int dtype, bool vec, const AxisParams& p, dim3 grid, unsigned strips_per_outer,
                        int lc_shift, int pdl, cudaStream_t stream) {
  if (lc_shift < 0 || lc_shift > 5) return cudaErrorInvalidValue;
  switch (op) {
    case OP_SOFTMAX: return launch_axis_op<OP_SOFTMAX>(dtype, vec, p, grid, strips_per_outer, lc_shift, pdl, stream);
    case OP_LOG_SOFTMAX: return launch_axis_op<OP_LOG_SOFTMAX>(dtype, vec, p, grid, strips_per_outer, lc_shift, pdl, stream);
    case OP_LAYERNORM: return launch_axis_op<OP_LAYERNORM>(dtype, vec, p, grid, strips_per_outer, lc_shift, pdl, stream);
    case OP_RMSNORM: return launch_axis_op<OP_RMSNORM>(dtype, vec, p, grid, strips_per_outer, lc_shift, pdl, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace akg
