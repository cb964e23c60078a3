// Kernels and launcher of the non-last-axis operators (their own translation unit).
#include "kernels_axis.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <int OP, typename T, bool VEC>
cudaError_t launch_axis_typed(const AxisParams& p, unsigned grid, long long strips_per_outer, int pdl,
                              cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, axis_kernel<OP, T, VEC, 256>, p, strips_per_outer);
}

template <int OP>
cudaError_t launch_axis_op(int dtype, bool vec, const AxisParams& p, unsigned grid, long long spo, int pdl,
                           cudaStream_t s) {
  if (dtype == DT_F32)
    return vec ? launch_axis_typed<OP, float, true>(p, grid, spo, pdl, s)
               : launch_axis_typed<OP, float, false>(p, grid, spo, pdl, s);
  return vec ? launch_axis_typed<OP, __nv_bfloat16, true>(p, grid, spo, pdl, s)
             : launch_axis_typed<OP, __nv_bfloat16, false>(p, grid, spo, pdl, s);
}

}  // namespace

cudaError_t launch_axis(int op, int dtype, bool vec, const AxisParams& p, unsigned grid,
                        long long strips_per_outer, int pdl, cudaStream_t stream) {
  switch (op) {
    case OP_SOFTMAX: return launch_axis_op<OP_SOFTMAX>(dtype, vec, p, grid, strips_per_outer, pdl, stream);
    case OP_LOG_SOFTMAX: return launch_axis_op<OP_LOG_SOFTMAX>(dtype, vec, p, grid, strips_per_outer, pdl, stream);
    case OP_LAYERNORM: return launch_axis_op<OP_LAYERNORM>(dtype, vec, p, grid, strips_per_outer, pdl, stream);
    case OP_RMSNORM: return launch_axis_op<OP_RMSNORM>(dtype, vec, p, grid, strips_per_outer, pdl, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace akg
