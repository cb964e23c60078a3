// Kernels and launcher of one operator (compiled as its own translation unit).
#include "launch_impl.cuh"

namespace akg {
template cudaError_t launch_op<OP_LOG_SOFTMAX>(const LaunchPlan&, int, const RowParams&, cudaStream_t);
}  // namespace akg
