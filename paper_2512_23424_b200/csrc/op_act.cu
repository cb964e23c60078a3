// Gated activations (SiLU-and-Mul, GELU-and-Mul): kernels and launcher.
#include "kernels_act.cuh"
#include "launch.cuh"

namespace akg {
namespace {

constexpr int kActU = 4;        // vectors of a and of b per thread and iteration

template <int ACT, typename T, bool VEC>
cudaError_t launch_act_typed(const ActParams& p, dim3 grid, int threads, int pdl, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, act_mul_kernel<ACT, T, VEC, kActU>, p);
}

template <int ACT>
cudaError_t launch_act_a(int dtype, bool vec, const ActParams& p, dim3 grid, int threads, int pdl, cudaStream_t s) {
  if (dtype == DT_F32)
    return vec ? launch_act_typed<ACT, float, true>(p, grid, threads, pdl, s)
               : launch_act_typed<ACT, float, false>(p, grid, threads, pdl, s);
  if (dtype == DT_F16)
    return vec ? launch_act_typed<ACT, __half, true>(p, grid, threads, pdl, s)
               : launch_act_typed<ACT, __half, false>(p, grid, threads, pdl, s);
  return vec ? launch_act_typed<ACT, __nv_bfloat16, true>(p, grid, threads, pdl, s)
             : launch_act_typed<ACT, __nv_bfloat16, false>(p, grid, threads, pdl, s);
}

}  // namespace

int act_mul_unroll() { return kActU; }

cudaError_t launch_act_mul(int act, int dtype, bool vec, const ActParams& p, dim3 grid, int threads, int pdl,
                           cudaStream_t stream) {
  if (threads < 32 || threads > 256 || threads % 32) return cudaErrorInvalidValue;
  switch (act) {
    case ACT_SILU: return launch_act_a<ACT_SILU>(dtype, vec, p, grid, threads, pdl, stream);
    case ACT_GELU: return launch_act_a<ACT_GELU>(dtype, vec, p, grid, threads, pdl, stream);
    case ACT_GELU_TANH: return launch_act_a<ACT_GELU_TANH>(dtype, vec, p, grid, threads, pdl, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace akg
