// Register-resident kernels of the non-last-axis operators and their launcher.
#include "kernels_axis_reg.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <int OP, typename T, int MODE, int R>
cudaError_t launch_axis_reg_r(const AxisParams& p, dim3 grid, unsigned spo, int nf, int nc, int pdl,
                              cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = grid;
  cfg.blockDim = dim3(32u * nf * nc);
  cfg.dynamicSmemBytes = 4u * axis_reg_smem_floats(OP == OP_RMSNORM ? 1 : 2, nf, nc, AxisRaw<T, MODE>::W);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, axis_reg_kernel<OP, T, MODE, R>, p, spo, nf, nc,
                            static_cast<int>(p.reduce / nf), static_cast<int>(p.reduce % nf));
}

template <int OP, typename T, int MODE>
cudaError_t launch_axis_reg_m(int r, const AxisParams& p, dim3 grid, unsigned spo, int nf, int nc, int pdl,
                              cudaStream_t s) {
  switch (r) {
    case 2: return launch_axis_reg_r<OP, T, MODE, 2>(p, grid, spo, nf, nc, pdl, s);
    case 4: return launch_axis_reg_r<OP, T, MODE, 4>(p, grid, spo, nf, nc, pdl, s);
    case 8: return launch_axis_reg_r<OP, T, MODE, 8>(p, grid, spo, nf, nc, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

template <int OP>
cudaError_t launch_axis_reg_op(int dtype, int mode, int r, const AxisParams& p, dim3 grid, unsigned spo,
                               int nf, int nc, int pdl, cudaStream_t s) {
  if (dtype == DT_F32) {
    if (mode == 1) return launch_axis_reg_m<OP, float, 1>(r, p, grid, spo, nf, nc, pdl, s);
    if (mode == 0) return launch_axis_reg_m<OP, float, 0>(r, p, grid, spo, nf, nc, pdl, s);
    return cudaErrorInvalidValue;
  }
  if (dtype == DT_F16) {
    if (mode == 1) return launch_axis_reg_m<OP, __half, 1>(r, p, grid, spo, nf, nc, pdl, s);
    if (mode == 0) return launch_axis_reg_m<OP, __half, 0>(r, p, grid, spo, nf, nc, pdl, s);
    return cudaErrorInvalidValue;
  }
  if (mode == 2) return launch_axis_reg_m<OP, __nv_bfloat16, 2>(r, p, grid, spo, nf, nc, pdl, s);
  if (mode == 1) return launch_axis_reg_m<OP, __nv_bfloat16, 1>(r, p, grid, spo, nf, nc, pdl, s);
  return launch_axis_reg_m<OP, __nv_bfloat16, 0>(r, p, grid, spo, nf, nc, pdl, s);
}

}  // namespace

int axis_reg_width(int dtype, int mode) {
  if (mode == 0) return 1;
  if (mode == 2) return 4;
  return dtype == DT_F32 ? 4 : 8;
}

cudaError_t launch_axis_reg(int op, int dtype, int mode, int r, const AxisParams& p, dim3 grid,
                            unsigned strips_per_outer, int nf, int nc, int pdl, cudaStream_t stream) {
  if (nf < 1 || nc < 1 || nf * nc > kAxisMaxWarps || p.reduce > static_cast<long long>(nf) * r)
    return cudaErrorInvalidValue;
  switch (op) {
    case OP_SOFTMAX: return launch_axis_reg_op<OP_SOFTMAX>(dtype, mode, r, p, grid, strips_per_outer, nf, nc, pdl, stream);
    case OP_LOG_SOFTMAX: return launch_axis_reg_op<OP_LOG_SOFTMAX>(dtype, mode, r, p, grid, strips_per_outer, nf, nc, pdl, stream);
    case OP_LAYERNORM: return launch_axis_reg_op<OP_LAYERNORM>(dtype, mode, r, p, grid, strips_per_outer, nf, nc, pdl, stream);
    case OP_RMSNORM: return launch_axis_reg_op<OP_RMSNORM>(dtype, mode, r, p, grid, strips_per_outer, nf, nc, pdl, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace akg
