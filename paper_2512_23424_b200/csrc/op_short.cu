// Short rows, several per warp: kernels and launcher.
#include "kernels_short.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <typename K>
cudaError_t launch_short_k(K kernel, const RowParams& p, unsigned grid, int pdl, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kShortThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int OP, typename T, bool CAUSAL>
cudaError_t launch_short_l(int lanes, const RowParams& p, unsigned grid, int pdl, cudaStream_t s) {
  switch (lanes) {
    case 4: return launch_short_k(short_rows_kernel<OP, T, 4, CAUSAL>, p, grid, pdl, s);
    case 8: return launch_short_k(short_rows_kernel<OP, T, 8, CAUSAL>, p, grid, pdl, s);
    case 16: return launch_short_k(short_rows_kernel<OP, T, 16, CAUSAL>, p, grid, pdl, s);
    case 32: return launch_short_k(short_rows_kernel<OP, T, 32, CAUSAL>, p, grid, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

template <int OP, typename T>
cudaError_t launch_short_c(int lanes, const RowParams& p, unsigned grid, int pdl, cudaStream_t s) {
  if constexpr (OpTraits<OP>::kSoftmaxLike) {
    if (p.causal) return launch_short_l<OP, T, true>(lanes, p, grid, pdl, s);
  }
  return launch_short_l<OP, T, false>(lanes, p, grid, pdl, s);
}

template <int OP>
cudaError_t launch_short_t(int dtype, int lanes, const RowParams& p, unsigned grid, int pdl, cudaStream_t s) {
  if (dtype == DT_F32) return launch_short_c<OP, float>(lanes, p, grid, pdl, s);
  if (dtype == DT_F16) return launch_short_c<OP, __half>(lanes, p, grid, pdl, s);
  return launch_short_c<OP, __nv_bfloat16>(lanes, p, grid, pdl, s);
}

}  // namespace

int short_rows_per_cta(int lanes) { return (kShortThreads / 32) * (32 / lanes); }
int short_max_vectors(int lanes) { return lanes * kShortVecs; }

cudaError_t launch_short(int op, int dtype, int lanes, const RowParams& p, unsigned grid, int pdl, cudaStream_t stream) {
  switch (op) {
    case OP_SOFTMAX: return launch_short_t<OP_SOFTMAX>(dtype, lanes, p, grid, pdl, stream);
    case OP_LOG_SOFTMAX: return launch_short_t<OP_LOG_SOFTMAX>(dtype, lanes, p, grid, pdl, stream);
    case OP_LAYERNORM: return launch_short_t<OP_LAYERNORM>(dtype, lanes, p, grid, pdl, stream);
    default: return launch_short_t<OP_RMSNORM>(dtype, lanes, p, grid, pdl, stream);
  }
}

}  // namespace akg
