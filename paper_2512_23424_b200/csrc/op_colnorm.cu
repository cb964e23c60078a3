// BatchNorm-style column normalisation: kernels and launcher.
#include "kernels_colnorm.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <typename K>
cudaError_t launch_col(K kernel, const ColParams& p, dim3 grid, int pdl, cudaStream_t s) {
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
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <typename T, int MODE>
cudaError_t launch_colnorm_t(const ColParams& p, dim3 grid, int pdl, cudaStream_t s) {
  cudaError_t e = launch_col(col_stat_kernel<T, MODE>, p, grid, pdl, s);
  if (e != cudaSuccess) return e;
  {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(static_cast<unsigned>((p.cols + 7) / 8));
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    e = cudaLaunchKernelEx(&cfg, col_finish_kernel, p, static_cast<int>(grid.y));
    if (e != cudaSuccess) return e;
  }
  return launch_col(col_apply_kernel<T, MODE>, p, grid, pdl, s);
}

}  // namespace

int colnorm_row_slots(int lc_shift) { return kAxisThreads >> lc_shift; }

cudaError_t launch_colnorm(int dtype, bool vec, const ColParams& p, dim3 grid, int pdl, cudaStream_t stream) {
  if (dtype == DT_F32) return vec ? launch_colnorm_t<float, 1>(p, grid, pdl, stream) : launch_colnorm_t<float, 0>(p, grid, pdl, stream);
  if (dtype == DT_F16) return vec ? launch_colnorm_t<__half, 1>(p, grid, pdl, stream) : launch_colnorm_t<__half, 0>(p, grid, pdl, stream);
  return vec ? launch_colnorm_t<__nv_bfloat16, 1>(p, grid, pdl, stream) : launch_colnorm_t<__nv_bfloat16, 0>(p, grid, pdl, stream);
}

}  // namespace akg
