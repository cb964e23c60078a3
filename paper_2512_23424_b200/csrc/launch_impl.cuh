// Definition of launch_op<OP>; included only by the per-operator translation units.
#pragma once

#include <map>
#include <mutex>
#include <tuple>

#include "kernels_basic.cuh"
#include "kernels_reg.cuh"
#include "kernels_softmax.cuh"
#include "kernels_ring.cuh"
#include "kernels_smem.cuh"
#include "kernels_split.cuh"
#include "launch.cuh"

namespace akg {

// The (threads-per-row, vectors-per-thread, CTA size) shapes reg_kernel is built for.
// api.cu's planner only ever asks for one of these.
#define AKG_REG_SHAPES(X) \
  X(32, 1, 128) X(32, 2, 128) X(32, 4, 128) X(32, 8, 128) \
  X(128, 1, 128) X(128, 2, 128) X(128, 4, 128) \
  X(256, 1, 256) X(256, 2, 256) X(256, 4, 256) X(256, 8, 256) \
  X(512, 1, 512) X(512, 2, 512) X(512, 4, 512) X(512, 8, 512) \
  X(1024, 1, 1024) X(1024, 2, 1024) X(1024, 4, 1024) X(1024, 8, 1024)

// Shapes that are compiled for element type T.  The 16-bit types never get a CTA of 1024 threads or eight
// vectors per thread in a CTA of 256 and more from the planner (rows beyond 2048 vectors leave the register
// family, and the fat-thread normalisation is reg_norm_flex); those bodies spilled 0.2 - 1 KB per thread.
template <typename T, int G_, int V_, int T_>
constexpr bool kRegShapeBuilt = sizeof(T) == 4 || !((T_) >= 1024 || ((V_) == 8 && (T_) >= 256));

// Fill the launch attributes: programmatic stream serialisation when the plan asks for
// it, a cluster dimension when cluster > 1.  Returns the number of attributes set.
inline unsigned launch_attrs(cudaLaunchAttribute* attr, const LaunchPlan& plan, int cluster) {
  unsigned n = 0;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (plan.pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  return n;
}

// A plain (non-cluster) launch with the plan's attributes.
template <typename... KArgs, typename... Args>
cudaError_t launch_plain(void (*kernel)(KArgs...), const LaunchPlan& plan, unsigned grid, int threads, size_t smem,
                         cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(static_cast<unsigned>(threads));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = launch_attrs(attr, plan, 1);
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// A launch of one of the packed / runtime-thread-count register kernels with a cluster of plan.cluster CTAs
// per row (plan.grid counts CTAs, a multiple of the cluster size).
template <typename... KArgs, typename... Args>
cudaError_t launch_reg_cluster(void (*kernel)(KArgs...), const LaunchPlan& plan, cudaStream_t s, Args... args) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, bool> prepared;     // (kernel, device) -> non-portable sizes allowed
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (plan.cluster > 8) {
    std::lock_guard<std::mutex> lock(mu);
    auto key = std::make_pair(reinterpret_cast<const void*>(kernel), dev);
    if (!prepared[key]) {
      err = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (err != cudaSuccess) return err;
      prepared[key] = true;
    }
  }
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(plan.cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(plan.grid);
  cfg.blockDim = dim3(static_cast<unsigned>(plan.threads));
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// Launch smem_kernel (TMA ring, optionally clustered).  plan.grid == 0 asks for as many
// clusters as can be co-resident (capped by the number of rows).
template <int OP, typename T, int THREADS>
cudaError_t launch_smem(const LaunchPlan& plan, const RowParams& p, cudaStream_t s) {
  auto kernel = smem_kernel<OP, T, THREADS>;
  static std::mutex mu;
  static std::map<std::tuple<int, int, size_t>, int> resident;   // (device, cluster, smem) -> clusters
  static std::map<int, bool> prepared;                             // device -> attributes set
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;       // always first: the occupancy query reads it
  attr[0].val.clusterDim.x = static_cast<unsigned>(plan.cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = plan.smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;

  int max_clusters = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!prepared[dev]) {
      err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
      if (err != cudaSuccess) return err;
      err = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (err != cudaSuccess) return err;
      prepared[dev] = true;
    }
    auto key = std::make_tuple(dev, plan.cluster, plan.smem);
    auto it = resident.find(key);
    if (it == resident.end()) {
      cfg.gridDim = dim3(static_cast<unsigned>(plan.cluster) * 1024u);
      int n = 0;
      err = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
      if (err != cudaSuccess) return err;
      it = resident.emplace(key, n).first;
    }
    max_clusters = it->second;
  }
  if (max_clusters < 1) return cudaErrorLaunchOutOfResources;
  long long clusters = plan.grid ? plan.grid / plan.cluster : max_clusters;
  if (clusters > p.rows) clusters = p.rows;
  if (clusters < 1) clusters = 1;
  cfg.gridDim = dim3(static_cast<unsigned>(clusters * plan.cluster));
  SmemGeom g;
  g.nbuf = plan.stages;
  g.slice_vecs = plan.vpt;          // V_TMA / V_CLUSTER reuse the field: vectors per CTA slice
  g.buf_bytes = static_cast<unsigned>((static_cast<size_t>(plan.vpt) * 16 + 127) & ~static_cast<size_t>(127));
  if (plan.pdl) {
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kernel, p, g, plan.variant == V_CLUSTER ? (plan.mode == 1 ? 0 : (plan.mode == 2 ? 2 : 1)) : (plan.mode == 2 ? 2 : 1));
}

// Launch a ring-fed register kernel (persistent; plan.grid == 0 asks for one full wave).
template <typename Kernel>
cudaError_t launch_ring(Kernel kernel, int threads, const LaunchPlan& plan, const RowParams& p, cudaStream_t s) {
  static std::mutex mu;
  static std::map<std::tuple<const void*, int, size_t>, int> wave;   // (kernel, device, smem) -> CTAs per wave
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  int ctas = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    auto key = std::make_tuple(reinterpret_cast<const void*>(kernel), dev, plan.smem);
    auto it = wave.find(key);
    if (it == wave.end()) {
      // the kernels also hold a few hundred bytes of static shared memory
      err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kMaxDynSmem) - 2048);
      if (err != cudaSuccess) return err;
      int per_sm = 0, sms = 0;
      err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, plan.smem);
      if (err != cudaSuccess) return err;
      err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (err != cudaSuccess) return err;
      it = wave.emplace(key, per_sm * sms).first;
    }
    ctas = it->second;
  }
  if (ctas < 1) return cudaErrorLaunchOutOfResources;
  long long grid = plan.grid ? plan.grid : ctas;
  if (grid > p.rows) grid = p.rows;
  return launch_plain(kernel, plan, static_cast<unsigned>(grid), threads, plan.smem, s, p, plan.stages);
}

// Launch split_kernel (cluster per row, two streaming passes, second one from L2).
template <int OP, typename T, int THREADS>
cudaError_t launch_split(const LaunchPlan& plan, const RowParams& p, cudaStream_t s) {
  auto kernel = split_kernel<OP, T, THREADS>;
  static std::mutex mu;
  static std::map<std::pair<int, int>, int> resident;   // (device, cluster) -> co-resident clusters
  static std::map<int, bool> prepared;
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;       // always first: the occupancy query reads it
  attr[0].val.clusterDim.x = static_cast<unsigned>(plan.cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(THREADS);
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
    auto key = std::make_pair(dev, plan.cluster);
    auto it = resident.find(key);
    if (it == resident.end()) {
      cfg.gridDim = dim3(static_cast<unsigned>(plan.cluster) * 1024u);
      int n = 0;
      err = cudaOccupancyMaxActiveClusters(&n, kernel, &cfg);
      if (err != cudaSuccess) return err;
      it = resident.emplace(key, n).first;
    }
    max_clusters = it->second;
  }
  if (max_clusters < 1) return cudaErrorLaunchOutOfResources;
  long long clusters = max_clusters;                     // one resident wave, optionally capped
  if (plan.grid && plan.grid / plan.cluster < clusters) clusters = plan.grid / plan.cluster;
  if (clusters > p.rows) clusters = p.rows;
  if (clusters < 1) clusters = 1;
  cfg.gridDim = dim3(static_cast<unsigned>(clusters * plan.cluster));
  if (plan.pdl) {
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kernel, p, plan.vpt, plan.mode == 1 ? 0 : 1, plan.split_l2);
}

template <int OP, typename T>
cudaError_t launch_typed(const LaunchPlan& plan, const RowParams& p, cudaStream_t s) {
  if (plan.variant == V_STREAM) {
    return launch_plain(stream_kernel<OP, T, 256>, plan, plan.grid, 256, 0, s, p);
  }
  if (plan.variant == V_REG && plan.mode == 3) {            // runtime thread count, exact fit, 16-bit row kept packed
    if constexpr (OpTraits<OP>::kSoftmaxLike && sizeof(T) == 2) {
      switch (plan.vpt) {
#define AKG_PACKED_SM_CASE(V_)                                                                              \
  case V_:                                                                                                  \
    if (plan.cluster > 1) return launch_reg_cluster(reg_softmax_packed<OP, T, V_>, plan, s, p);             \
    return launch_plain(reg_softmax_packed<OP, T, V_>, plan, plan.grid, plan.threads, 0, s, p);
        AKG_PACKED_SM_CASE(2) AKG_PACKED_SM_CASE(3) AKG_PACKED_SM_CASE(4) AKG_PACKED_SM_CASE(5)
        AKG_PACKED_SM_CASE(6) AKG_PACKED_SM_CASE(7) AKG_PACKED_SM_CASE(8)
#undef AKG_PACKED_SM_CASE
        default: break;
      }
    }
    if constexpr (OpTraits<OP>::kSoftmaxLike && sizeof(T) == 4) {    // fp32: the same scheme on widened values
      switch (plan.vpt) {
#define AKG_FLEX_SM_CASE(V_)                                                                                \
  case V_:                                                                                                  \
    if (plan.cluster > 1) return launch_reg_cluster(reg_softmax_flex<OP, V_>, plan, s, p);                  \
    return launch_plain(reg_softmax_flex<OP, V_>, plan, plan.grid, plan.threads, 0, s, p);
        AKG_FLEX_SM_CASE(2) AKG_FLEX_SM_CASE(3) AKG_FLEX_SM_CASE(4) AKG_FLEX_SM_CASE(5)
        AKG_FLEX_SM_CASE(6) AKG_FLEX_SM_CASE(7) AKG_FLEX_SM_CASE(8)
#undef AKG_FLEX_SM_CASE
        default: break;
      }
    }
    if constexpr (!OpTraits<OP>::kSoftmaxLike && sizeof(T) == 2) {
      const float inv_warps = 1.0f / static_cast<float>(plan.threads / 32);
      switch (plan.vpt) {
#define AKG_PACKED_CASE(V_) \
  case V_: return launch_plain(reg_norm_packed<OP, T, V_>, plan, plan.grid, plan.threads, 0, s, p, inv_warps);
        AKG_PACKED_CASE(2) AKG_PACKED_CASE(3) AKG_PACKED_CASE(4) AKG_PACKED_CASE(5)
        AKG_PACKED_CASE(6) AKG_PACKED_CASE(7) AKG_PACKED_CASE(8)
#undef AKG_PACKED_CASE
        default: break;
      }
    }
    return cudaErrorInvalidConfiguration;
  }
  if (plan.variant == V_REG && plan.mode == 2) {            // runtime thread count, exact fit
    if constexpr (!OpTraits<OP>::kSoftmaxLike) {
      const float inv_warps = 1.0f / static_cast<float>(plan.threads / 32);
      switch (plan.vpt) {
#define AKG_FLEX_CASE(V_) \
  case V_: return launch_plain(reg_norm_flex<OP, T, V_>, plan, plan.grid, plan.threads, 0, s, p, inv_warps);
        AKG_FLEX_CASE(1) AKG_FLEX_CASE(2) AKG_FLEX_CASE(3) AKG_FLEX_CASE(4)
        AKG_FLEX_CASE(5) AKG_FLEX_CASE(6) AKG_FLEX_CASE(7) AKG_FLEX_CASE(8)
#undef AKG_FLEX_CASE
        default: break;
      }
    }
    return cudaErrorInvalidConfiguration;
  }
  if (plan.variant == V_REG) {
    // plan.stages == 1 marks a row of exactly group * vpt vectors (the predicate-free
    // normalisation kernel); the softmax pair always takes its own lean kernel.
#define AKG_REG_CASE(G_, V_, T_)                                              \
  if (plan.group == (G_) && plan.vpt == (V_) && plan.threads == (T_)) {       \
    if constexpr (!kRegShapeBuilt<T, G_, V_, T_>) {                           \
      return cudaErrorInvalidConfiguration;                                   \
    } else if constexpr (OpTraits<OP>::kSoftmaxLike) {                        \
      return launch_plain(reg_softmax<OP, T, G_, V_, T_>, plan, plan.grid, T_, 0, s, p);      \
    } else {                                                                  \
      if (plan.stages == 1)                                                   \
        return launch_plain(reg_norm_full<OP, T, G_, V_, T_>, plan, plan.grid, T_, 0, s, p);  \
      return launch_plain(reg_kernel<OP, T, G_, V_, T_>, plan, plan.grid, T_, 0, s, p);       \
    }                                                                         \
  }
    AKG_REG_SHAPES(AKG_REG_CASE)
#undef AKG_REG_CASE
    // a warp per row with an odd number of vectors per lane (768, 1280, 1536 ... columns): exact
    // fits of the normalisation kernel only
    if constexpr (!OpTraits<OP>::kSoftmaxLike) {
      if (plan.stages == 1 && plan.group == 32 && plan.threads == 128) {
        switch (plan.vpt) {
          case 3: return launch_plain(reg_norm_full<OP, T, 32, 3, 128>, plan, plan.grid, 128, 0, s, p);
          case 5: return launch_plain(reg_norm_full<OP, T, 32, 5, 128>, plan, plan.grid, 128, 0, s, p);
          case 6: return launch_plain(reg_norm_full<OP, T, 32, 6, 128>, plan, plan.grid, 128, 0, s, p);
          case 7: return launch_plain(reg_norm_full<OP, T, 32, 7, 128>, plan, plan.grid, 128, 0, s, p);
          default: break;
        }
      }
    }
    return cudaErrorInvalidConfiguration;
  }
  if (plan.variant == V_TMA && plan.mode == 1) {             // ring-fed register kernels
#define AKG_RING_CASE(G_, V_, T_)                                                                  \
  if ((G_) == (T_) && plan.vpt == (V_) && plan.threads == (T_)) {                                  \
    if constexpr ((G_) == (T_) && (V_) <= 4 && (T_) <= 512) {                                      \
      if constexpr (OpTraits<OP>::kSoftmaxLike)                                                    \
        return launch_ring(ring_softmax<OP, T, V_, T_>, T_, plan, p, s);                           \
      else                                                                                         \
        return launch_ring(ring_norm_full<OP, T, V_, T_>, T_, plan, p, s);                         \
    }                                                                                              \
  }
    AKG_REG_SHAPES(AKG_RING_CASE)
#undef AKG_RING_CASE
    return cudaErrorInvalidConfiguration;
  }
  if (plan.variant == V_CLUSTER && plan.stages == 0) {       // no ring: the two-pass split kernel
    if (plan.threads == 256) return launch_split<OP, T, 256>(plan, p, s);
    if (plan.threads == 512) return launch_split<OP, T, 512>(plan, p, s);
    if (plan.threads == 1024) return launch_split<OP, T, 1024>(plan, p, s);
    return cudaErrorInvalidConfiguration;
  }
  if (plan.variant == V_TMA || plan.variant == V_CLUSTER) {
    if (plan.threads == 256) return launch_smem<OP, T, 256>(plan, p, s);
    if (plan.threads == 512) return launch_smem<OP, T, 512>(plan, p, s);
    if (plan.threads == 1024) return launch_smem<OP, T, 1024>(plan, p, s);
    return cudaErrorInvalidConfiguration;
  }
  return cudaErrorInvalidConfiguration;
}

template <int OP>
cudaError_t launch_op(const LaunchPlan& plan, int dtype, const RowParams& p, cudaStream_t stream) {
  if (dtype == DT_F32) return launch_typed<OP, float>(plan, p, stream);
  if (dtype == DT_F16) return launch_typed<OP, __half>(plan, p, stream);
  return launch_typed<OP, __nv_bfloat16>(plan, p, stream);
}

}  // namespace akg
