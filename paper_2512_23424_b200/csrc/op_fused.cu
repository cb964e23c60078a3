// Fused residual add + normalisation: kernels and launcher.
#include "kernels_fused.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <int OP, typename T, int VPT>
cudaError_t launch_add_norm_v(const RowParams& p, unsigned grid, int threads, int pdl, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, add_norm_flex<OP, T, VPT>, p, 1.0f / static_cast<float>(threads / 32));
}

template <int OP, typename T>
cudaError_t launch_add_norm_t(int vpt, const RowParams& p, unsigned grid, int threads, int pdl, cudaStream_t s) {
  switch (vpt) {
    case 1: return launch_add_norm_v<OP, T, 1>(p, grid, threads, pdl, s);
    case 2: return launch_add_norm_v<OP, T, 2>(p, grid, threads, pdl, s);
    case 3: return launch_add_norm_v<OP, T, 3>(p, grid, threads, pdl, s);
    case 4: return launch_add_norm_v<OP, T, 4>(p, grid, threads, pdl, s);
    case 5: return launch_add_norm_v<OP, T, 5>(p, grid, threads, pdl, s);
    case 6: return launch_add_norm_v<OP, T, 6>(p, grid, threads, pdl, s);
    case 7: return launch_add_norm_v<OP, T, 7>(p, grid, threads, pdl, s);
    case 8: return launch_add_norm_v<OP, T, 8>(p, grid, threads, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_add_norm(int op, int dtype, int vpt, int threads, const RowParams& p, unsigned grid, int pdl,
                            cudaStream_t stream) {
  if (threads < 32 || threads > 1024 || threads % 32) return cudaErrorInvalidValue;
  if (op == OP_LAYERNORM)
    return dtype == DT_F32 ? launch_add_norm_t<OP_LAYERNORM, float>(vpt, p, grid, threads, pdl, stream)
           : dtype == DT_F16 ? launch_add_norm_t<OP_LAYERNORM, __half>(vpt, p, grid, threads, pdl, stream)
                             : launch_add_norm_t<OP_LAYERNORM, __nv_bfloat16>(vpt, p, grid, threads, pdl, stream);
  if (op == OP_RMSNORM)
    return dtype == DT_F32 ? launch_add_norm_t<OP_RMSNORM, float>(vpt, p, grid, threads, pdl, stream)
           : dtype == DT_F16 ? launch_add_norm_t<OP_RMSNORM, __half>(vpt, p, grid, threads, pdl, stream)
                             : launch_add_norm_t<OP_RMSNORM, __nv_bfloat16>(vpt, p, grid, threads, pdl, stream);
  return cudaErrorInvalidValue;
}

}  // namespace akg
