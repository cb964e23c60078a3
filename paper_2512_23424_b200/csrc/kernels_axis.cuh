// axis_kernel: the four operators over a NON-last axis of x[outer, reduce, inner] (inner
// contiguous) - the layout of the paper's RMSNorm sketch (Unified Sketch figure, Section
// 3.2.1: X[B, F, D1, D2] reduced over F, inner = D1 * D2).
//
// Threads own columns, not rows: a CTA takes a strip of 32 lanes x W contiguous columns
// (W = one 16-byte vector, or one element on the unaligned path) of one outer index, and
// its THREADS / 32 warps split the reduced axis between them (warp w takes f = w, w + NW,
// ...), so every load is a fully coalesced 512-byte row segment.  Pass 1 keeps running
// statistics per column in registers (block-wise online max / rescaled sum, block-wise
// mean / M2 with Chan's merge, sum of squares), the warps' partials are merged through
// shared memory, and pass 2 re-reads the strip - still in L2, it was read microseconds
// earlier and the planner bounds the strips in flight - to normalise and store.  HBM sees
// one read and one write per element.
#pragma once

#include "kernels_split.cuh"

namespace akg {

template <typename T, bool VEC> struct AxisLane {
  using E = Elem<T>;
  static constexpr int W = VEC ? E::EPV : 1;
  static __device__ __forceinline__ void load(const T* p, uint64_t pol, float (&f)[W]) {
    if constexpr (VEC) {
      float t[E::EPV];
      E::unpack(ld_hint(p, pol), t);
#pragma unroll
      for (int j = 0; j < W; ++j) f[j] = t[j];
    } else {
      f[0] = E::load1(p, 0);
    }
  }
  static __device__ __forceinline__ void store(T* p, const float (&f)[W]) {
    if constexpr (VEC) {
      float t[E::EPV];
#pragma unroll
      for (int j = 0; j < W; ++j) t[j] = f[j];
      st_stream(p, E::pack(t));
    } else {
      E::store1(p, 0, f[0]);
    }
  }
};

// Fold UB values of one column (consecutive f of this warp) into its running statistics.
template <int OP, int UB>
__device__ __forceinline__ void fold_column(Stat& st, const float (&z)[UB], int n) {
  if (OpTraits<OP>::kSoftmaxLike) {
    float mv = kNegInf;
#pragma unroll
    for (int u = 0; u < UB; ++u) if (u < n) mv = fmaxf(mv, z[u]);
    const float mn = fmaxf(st.a, mv);
    const float ms = (mn == kNegInf) ? 0.f : mn;
    float acc = st.b * exp_diff(st.a, ms);
#pragma unroll
    for (int u = 0; u < UB; ++u) if (u < n) acc += exp_diff(z[u], ms);
    st.a = mn; st.b = acc;
  } else if (OP == OP_LAYERNORM) {
    float sum = 0.f;
#pragma unroll
    for (int u = 0; u < UB; ++u) if (u < n) sum += z[u];
    const float cnt = static_cast<float>(n);
    const float mean = sum / cnt;
    float m2 = 0.f;
#pragma unroll
    for (int u = 0; u < UB; ++u) if (u < n) { const float d = z[u] - mean; m2 = fmaf(d, d, m2); }
    st = stat_merge<OP>(st, Stat{cnt, mean, m2});
  } else {
#pragma unroll
    for (int u = 0; u < UB; ++u) if (u < n) st.a = fmaf(z[u], z[u], st.a);
  }
}

template <int OP, typename T, bool VEC, int THREADS>
__global__ void __launch_bounds__(THREADS) axis_kernel(const AxisParams p, const long long strips_per_outer) {
  pdl_prologue();
  using L = AxisLane<T, VEC>;
  using E = Elem<T>;
  constexpr int W = L::W;
  constexpr int NF = THREADS / 32;          // warps = lanes along the reduced axis
  constexpr int UB = 4;                     // f values per block (loads in flight per thread)
  __shared__ Stat part[NF][32 * W];

  const int dl = threadIdx.x & 31;
  const int fl = threadIdx.x >> 5;
  const long long F = p.reduce;
  const uint64_t keep = l2_policy_keep();
  const uint64_t drop = l2_policy_drop();
  const long long strips = p.outer * strips_per_outer;

  for (long long s = blockIdx.x; s < strips; s += gridDim.x) {
    const long long b = s / strips_per_outer;
    const long long col0 = (s - b * strips_per_outer) * (32 * W) + static_cast<long long>(dl) * W;
    const bool active = col0 < p.inner;
    const T* xb = reinterpret_cast<const T*>(p.x) + b * p.xso + col0;
    T* yb = reinterpret_cast<T*>(p.y) + b * p.yso + col0;

    // ---- pass 1: per-column statistics over this warp's share of the reduced axis
    Stat st[W];
#pragma unroll
    for (int j = 0; j < W; ++j) st[j] = stat_identity<OP>();
    if (active) {
      for (long long f0 = fl; f0 < F; f0 += static_cast<long long>(NF) * UB) {
        float z[UB][W];
        int n = 0;
#pragma unroll
        for (int u = 0; u < UB; ++u) {
          const long long f = f0 + static_cast<long long>(u) * NF;
          if (f < F) { L::load(xb + f * p.xsf, keep, z[u]); n = u + 1; }
        }
#pragma unroll
        for (int j = 0; j < W; ++j) {
          float col[UB];
#pragma unroll
          for (int u = 0; u < UB; ++u) col[u] = z[u][j];
          fold_column<OP, UB>(st[j], col, n);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < W; ++j) part[fl][dl * W + j] = st[j];
    __syncthreads();

    // ---- merge the warps' partials (every warp does it for its own use) and finalise
    RowScalars rs[W];
#pragma unroll
    for (int j = 0; j < W; ++j) {
      Stat r = part[0][dl * W + j];
#pragma unroll
      for (int w = 1; w < NF; ++w) r = stat_merge<OP>(r, part[w][dl * W + j]);
      rs[j] = finalize<OP>(r, F, p.eps);
    }

    // ---- pass 2: second read (L2), normalise, store
    if (active) {
      for (long long f0 = fl; f0 < F; f0 += static_cast<long long>(NF) * UB) {
        float z[UB][W];
#pragma unroll
        for (int u = 0; u < UB; ++u) {
          const long long f = f0 + static_cast<long long>(u) * NF;
          if (f < F) L::load(xb + f * p.xsf, drop, z[u]);
        }
#pragma unroll
        for (int u = 0; u < UB; ++u) {
          const long long f = f0 + static_cast<long long>(u) * NF;
          if (f < F) {
            float g = 1.f, be = 0.f;
            if (!OpTraits<OP>::kSoftmaxLike) {
              if (p.gamma != nullptr) g = E::load1(p.gamma, f);
              if (OP == OP_LAYERNORM && p.beta != nullptr) be = E::load1(p.beta, f);
            }
            float o[W];
#pragma unroll
            for (int j = 0; j < W; ++j) {
              if (OP == OP_SOFTMAX) o[j] = exp_diff(z[u][j], rs[j].p) * rs[j].q;
              else o[j] = apply_one<OP>(z[u][j], rs[j], 0.f, g, be);
            }
            L::store(yb + f * p.ysf, o);
          }
        }
      }
    }
    __syncthreads();                       // `part` is rewritten by the next strip
  }
}

}  // namespace akg
