// Arg-max / arg-min and cumulative sum / product over the last axis: kernels and launchers.
#include <map>
#include <mutex>

#include "kernels_arg.cuh"
#include "kernels_scan.cuh"
#include "launch.cuh"

namespace akg {
namespace {

template <typename K, typename... Args>
cudaError_t launch_grid(K kernel, dim3 grid, int threads, int pdl, cudaStream_t s, Args... args) {
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
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename K, typename P>
cudaError_t launch_1d(K kernel, const P& p, unsigned grid, int threads, int pdl, cudaStream_t s) {
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
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <bool MIN, typename T>
cudaError_t launch_arg_t(bool vec, bool warp_rows, const ArgParams& p, unsigned grid, int pdl, cudaStream_t s) {
  if (vec) return warp_rows ? launch_1d(arg_kernel<MIN, T, 32, 256, true>, p, grid, 256, pdl, s)
                            : launch_1d(arg_kernel<MIN, T, 256, 256, true>, p, grid, 256, pdl, s);
  return warp_rows ? launch_1d(arg_kernel<MIN, T, 32, 256, false>, p, grid, 256, pdl, s)
                   : launch_1d(arg_kernel<MIN, T, 256, 256, false>, p, grid, 256, pdl, s);
}

// rows cut into `segments` pieces of seg_vecs vectors: clear, per-segment maxima, finish
template <bool MIN, typename T>
cudaError_t launch_arg_split_t(bool vec, const ArgParams& p, unsigned segments, long long seg_vecs, int pdl,
                               cudaStream_t s) {
  const unsigned small = static_cast<unsigned>(p.rows < 65536 ? (p.rows + 255) / 256 : 256);
  cudaError_t e = launch_grid(arg_clear_kernel, dim3(small), 256, pdl, s, p);
  if (e != cudaSuccess) return e;
  const dim3 grid(segments, static_cast<unsigned>(p.rows < 65535 ? p.rows : 65535));
  e = vec ? launch_grid(arg_split_kernel<MIN, T, true>, grid, 256, pdl, s, p, seg_vecs)
          : launch_grid(arg_split_kernel<MIN, T, false>, grid, 256, pdl, s, p, seg_vecs);
  if (e != cudaSuccess) return e;
  return launch_grid(arg_finish_kernel, dim3(small), 256, pdl, s, p);
}

template <bool PROD, typename T>
cudaError_t launch_scan_t(bool vec, bool warp_rows, const ScanParams& p, unsigned grid, int threads, int pdl,
                          cudaStream_t s, int depth) {
  if (vec && warp_rows) return launch_1d(scan_kernel<PROD, T, true, true>, p, grid, 32 * kScanMaxWarps, pdl, s);
  if (vec && depth > 1) return launch_1d(scan_flat_kernel<PROD, T, 3>, p, grid, threads, pdl, s);
  return vec ? launch_1d(scan_flat_kernel<PROD, T, 1>, p, grid, threads, pdl, s)
             : launch_1d(scan_kernel<PROD, T, false>, p, grid, threads, pdl, s);
}

template <bool PROD, typename T>
cudaError_t launch_scan_short_t(int lanes, const ScanParams& p, unsigned grid, int pdl, cudaStream_t s) {
  if (lanes == 4) return launch_1d(scan_short_kernel<PROD, T, 4>, p, grid, 256, pdl, s);
  if (lanes == 8) return launch_1d(scan_short_kernel<PROD, T, 8>, p, grid, 256, pdl, s);
  if (lanes == 16) return launch_1d(scan_short_kernel<PROD, T, 16>, p, grid, 256, pdl, s);
  return cudaErrorInvalidValue;
}

// scan_split_kernel: a cluster of `cluster` CTAs per row; clusters = 0 asks for one resident wave
template <bool PROD, typename T>
cudaError_t launch_scan_split_t(const ScanParams& p, int cluster, int slice_vecs, long long clusters, int* status,
                                unsigned wait_us, cudaStream_t s) {
  auto kernel = scan_split_kernel<PROD, T>;
  static std::mutex mu;
  static std::map<std::pair<int, int>, int> resident;   // (device, cluster) -> co-resident clusters
  static std::map<int, bool> prepared;
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int max_clusters = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!prepared[dev]) {
      err = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (err != cudaSuccess) return err;
      prepared[dev] = true;
    }
    auto key = std::make_pair(dev, cluster);
    auto it = resident.find(key);
    if (it == resident.end()) {
      cfg.gridDim = dim3(static_cast<unsigned>(cluster) * 1024u);
      int n = 0;
      err = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
      if (err != cudaSuccess) return err;
      it = resident.emplace(key, n).first;
    }
    max_clusters = it->second;
  }
  if (max_clusters < 1) return cudaErrorLaunchOutOfResources;
  long long n = max_clusters;
  if (clusters > 0 && clusters < n) n = clusters;
  if (n > p.rows) n = p.rows;
  if (n < 1) n = 1;
  cfg.gridDim = dim3(static_cast<unsigned>(n * cluster));
  return cudaLaunchKernelEx(&cfg, kernel, p, slice_vecs, status, wait_us);
}

}  // namespace

int scan_unroll() { return kScanU; }

cudaError_t launch_cumulative_short(bool want_prod, int dtype, int lanes, const void* x, void* y, long long rows,
                                    long long cols, long long xs, long long ys, unsigned grid, int pdl, cudaStream_t stream) {
  ScanParams p;
  p.x = x; p.y = y; p.rows = rows; p.cols = cols; p.xs = xs; p.ys = ys;
  if (dtype == DT_F32)
    return want_prod ? launch_scan_short_t<true, float>(lanes, p, grid, pdl, stream)
                     : launch_scan_short_t<false, float>(lanes, p, grid, pdl, stream);
  if (dtype == DT_F16)
    return want_prod ? launch_scan_short_t<true, __half>(lanes, p, grid, pdl, stream)
                     : launch_scan_short_t<false, __half>(lanes, p, grid, pdl, stream);
  return want_prod ? launch_scan_short_t<true, __nv_bfloat16>(lanes, p, grid, pdl, stream)
                   : launch_scan_short_t<false, __nv_bfloat16>(lanes, p, grid, pdl, stream);
}

cudaError_t launch_cumulative_split(bool want_prod, int dtype, const void* x, void* y, long long rows, long long cols,
                                    long long xs, long long ys, int cluster, int slice_vecs, long long clusters,
                                    int* status, unsigned wait_us, cudaStream_t stream) {
  ScanParams p;
  p.x = x; p.y = y; p.rows = rows; p.cols = cols; p.xs = xs; p.ys = ys;
  if (dtype == DT_F32)
    return want_prod ? launch_scan_split_t<true, float>(p, cluster, slice_vecs, clusters, status, wait_us, stream)
                     : launch_scan_split_t<false, float>(p, cluster, slice_vecs, clusters, status, wait_us, stream);
  if (dtype == DT_F16)
    return want_prod ? launch_scan_split_t<true, __half>(p, cluster, slice_vecs, clusters, status, wait_us, stream)
                     : launch_scan_split_t<false, __half>(p, cluster, slice_vecs, clusters, status, wait_us, stream);
  return want_prod ? launch_scan_split_t<true, __nv_bfloat16>(p, cluster, slice_vecs, clusters, status, wait_us, stream)
                   : launch_scan_split_t<false, __nv_bfloat16>(p, cluster, slice_vecs, clusters, status, wait_us, stream);
}

cudaError_t launch_argreduce(bool want_min, int dtype, bool vec, bool warp_rows, const void* x, long long* out,
                             long long rows, long long cols, long long xs, unsigned grid, unsigned segments,
                             long long seg_vecs, int pdl, cudaStream_t stream) {
  ArgParams p;
  p.x = x; p.out = out; p.rows = rows; p.cols = cols; p.xs = xs;
  if (segments > 1) {
    if (dtype == DT_F32)
      return want_min ? launch_arg_split_t<true, float>(vec, p, segments, seg_vecs, pdl, stream)
                      : launch_arg_split_t<false, float>(vec, p, segments, seg_vecs, pdl, stream);
    if (dtype == DT_F16)
      return want_min ? launch_arg_split_t<true, __half>(vec, p, segments, seg_vecs, pdl, stream)
                      : launch_arg_split_t<false, __half>(vec, p, segments, seg_vecs, pdl, stream);
    return want_min ? launch_arg_split_t<true, __nv_bfloat16>(vec, p, segments, seg_vecs, pdl, stream)
                    : launch_arg_split_t<false, __nv_bfloat16>(vec, p, segments, seg_vecs, pdl, stream);
  }
  if (dtype == DT_F32)
    return want_min ? launch_arg_t<true, float>(vec, warp_rows, p, grid, pdl, stream)
                    : launch_arg_t<false, float>(vec, warp_rows, p, grid, pdl, stream);
  if (dtype == DT_F16)
    return want_min ? launch_arg_t<true, __half>(vec, warp_rows, p, grid, pdl, stream)
                    : launch_arg_t<false, __half>(vec, warp_rows, p, grid, pdl, stream);
  return want_min ? launch_arg_t<true, __nv_bfloat16>(vec, warp_rows, p, grid, pdl, stream)
                  : launch_arg_t<false, __nv_bfloat16>(vec, warp_rows, p, grid, pdl, stream);
}

cudaError_t launch_cumulative(bool want_prod, int dtype, bool vec, const void* x, void* y, long long rows,
                              long long cols, long long xs, long long ys, unsigned grid, int threads, bool warp_rows,
                              int pdl, cudaStream_t stream, int depth) {
  if (threads < 32 || threads > 32 * kScanMaxWarps || threads % 32) return cudaErrorInvalidValue;
  ScanParams p;
  p.x = x; p.y = y; p.rows = rows; p.cols = cols; p.xs = xs; p.ys = ys;
  if (dtype == DT_F32)
    return want_prod ? launch_scan_t<true, float>(vec, warp_rows, p, grid, threads, pdl, stream, depth)
                     : launch_scan_t<false, float>(vec, warp_rows, p, grid, threads, pdl, stream, depth);
  if (dtype == DT_F16)
    return want_prod ? launch_scan_t<true, __half>(vec, warp_rows, p, grid, threads, pdl, stream, depth)
                     : launch_scan_t<false, __half>(vec, warp_rows, p, grid, threads, pdl, stream, depth);
  return want_prod ? launch_scan_t<true, __nv_bfloat16>(vec, warp_rows, p, grid, threads, pdl, stream, depth)
                   : launch_scan_t<false, __nv_bfloat16>(vec, warp_rows, p, grid, threads, pdl, stream, depth);
}

}  // namespace akg
