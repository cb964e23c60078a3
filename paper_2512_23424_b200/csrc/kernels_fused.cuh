// Fused variants of the normalisations (the operator benchmark of the paper lists "fused
// variants" among its categories, Section 3.6): residual add + LayerNorm / RMSNorm.
//
// add_norm_flex: s = x + res, sum_out = s, y = norm(s) in one pass over HBM - two input
// streams, two output streams, nothing read twice.  Same scheme as reg_norm_flex: a CTA per
// row, rows of exactly blockDim.x * VPT 16-byte vectors, the row in registers.  All 2 * VPT
// loads of a thread are issued before the first use; the sum is formed in fp32 from the
// widened operands, stored (rounded once) and normalised unrounded.
#pragma once

#include "kernels_reg.cuh"

namespace akg {

template <int OP, typename T, int VPT>
__global__ void __launch_bounds__(1024, 1) add_norm_flex(const RowParams p, const float inv_warps) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int N = VPT * EPV;
  static_assert(OP == OP_LAYERNORM || OP == OP_RMSNORM, "normalisations only");
  __shared__ float red[2][2][32];
  const int G = blockDim.x;
  const int NW = G >> 5;
  const int tg = threadIdx.x;
  const float inv_cols = 1.0f / static_cast<float>(p.cols);
  const long long step = static_cast<long long>(G) * EPV;
  int parity = 0;
  for (long long row = blockIdx.x; row < p.rows; row += gridDim.x, parity ^= 1) {
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + tg * EPV;
    const T* rr = reinterpret_cast<const T*>(p.res) + row * p.rs + tg * EPV;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + tg * EPV;
    uint4 rx[VPT], rq[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) rx[k] = ld_stream(xr + k * step);
#pragma unroll
    for (int k = 0; k < VPT; ++k) rq[k] = ld_stream(rr + k * step);
    float v[N];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      float a[EPV], b[EPV];
      E::unpack(rx[k], a);
      E::unpack(rq[k], b);
#pragma unroll
      for (int j = 0; j < EPV; ++j) v[k * EPV + j] = a[j] + b[j];
    }
    if (p.sum != nullptr) {
      T* sr = reinterpret_cast<T*>(p.sum) + row * p.ss + tg * EPV;
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        float o[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) o[j] = v[k * EPV + j];
        st_stream(sr + k * step, E::pack(o));
      }
    }
    float mean, rstd;
    flex_row_stats<OP, N>(v, red[parity], NW, inv_warps, inv_cols, p.eps, mean, rstd);
    const T* gp = reinterpret_cast<const T*>(p.gamma) + tg * EPV;
    const T* bp = reinterpret_cast<const T*>(p.beta) + tg * EPV;
    // every affine vector present: no defaults to materialise per element (as in norm_row_full);
    // 16-bit storage: the centring as one fused multiply-add with the row constant -mean * rstd
    const bool affine_all = p.gamma != nullptr && (OP != OP_LAYERNORM || p.beta != nullptr);
    constexpr bool kFusedCentre = (sizeof(T) == 2);
    const float neg_mean_rstd = -mean * rstd;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      float g[EPV], b[EPV], o[EPV];
      if (affine_all) {
        E::unpack(ld_cached(gp + k * step), g);
        if (OP == OP_LAYERNORM) E::unpack(ld_cached(bp + k * step), b);
      } else {
#pragma unroll
        for (int j = 0; j < EPV; ++j) { g[j] = 1.f; b[j] = 0.f; }
        if (p.gamma != nullptr) E::unpack(ld_cached(gp + k * step), g);
        if (OP == OP_LAYERNORM && p.beta != nullptr) E::unpack(ld_cached(bp + k * step), b);
      }
#pragma unroll
      for (int j = 0; j < EPV; ++j) {
        if (OP == OP_LAYERNORM) o[j] = kFusedCentre ? fmaf(fmaf(v[k * EPV + j], rstd, neg_mean_rstd), g[j], b[j])
                                                    : fmaf((v[k * EPV + j] - mean) * rstd, g[j], b[j]);
        else o[j] = v[k * EPV + j] * rstd * g[j];
      }
      st_stream(yr + k * step, E::pack(o));
    }
  }
}

}  // namespace akg
