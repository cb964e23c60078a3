// short_rows_kernel: rows of up to 128 vectors, plain or under the causal rule, several rows per warp.
//
// A warp per row leaves most of a warp waiting when the row is one or two vectors per lane (a
// bf16 row of 256 columns is 32 vectors): the row's latency chain (load, two reductions, store)
// is paid for 512 bytes.  Here L = 4 .. 32 lanes own a row and hold up to four of its vectors
// each (vector l, l + L, ...), so a warp works on 32 / L rows at once: four loads in flight
// per lane whatever the row length, and reductions of log2 L shuffle steps.  Control flow is
// uniform over the warp (lanes without a row or a vector compute on neutral values and skip
// the store), so the shuffles always name the full warp.  Under a causal mask a row's vectors
// beyond its live prefix are not read, the masked part of the boundary vector counts as -inf and
// masked outputs get the fill value (+0, -inf, or NaN for a NaN row), as in the register kernels.
//
// The arithmetic is that of the register kernels: softmax against the row maximum with one
// exponential per element, log-softmax as scale (x - max) - ln S, LayerNorm with the exact two
// sweeps (mean, then centred squares), RMSNorm from the sum of squares; fp32 throughout, one
// rounding at the store.
#pragma once

#include "kernels_reg.cuh"

namespace akg {

template <int L> __device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int m = L / 2; m >= 1; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  return v;
}
template <int L> __device__ __forceinline__ float group_max(float v) {
#pragma unroll
  for (int m = L / 2; m >= 1; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
  return v;
}

constexpr int kShortThreads = 128;
constexpr int kShortVecs = 4;                 // vectors per lane

// CAUSAL: compiled with the causal rule (softmax pair only); the plain form carries none of its bookkeeping.
template <int OP, typename T, int L, bool CAUSAL>
__global__ void __launch_bounds__(kShortThreads, 8) short_rows_kernel(const RowParams p) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int K = kShortVecs;
  constexpr int RPW = 32 / L;                  // rows per warp
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  constexpr bool kFused = (sizeof(T) == 2);    // 16-bit storage: exponent / centring as one multiply-add
  const int lane = threadIdx.x & 31;
  const int sub = lane % L;
  const int grp = lane / L;
  const int nvec = static_cast<int>(p.cols / EPV);
  const float inv_cols = 1.0f / static_cast<float>(p.cols);
  const long long warps = static_cast<long long>(gridDim.x) * (kShortThreads / 32);
  const long long warp0 = static_cast<long long>(blockIdx.x) * (kShortThreads / 32) + (threadIdx.x >> 5);
  bool ok[K];
#pragma unroll
  for (int k = 0; k < K; ++k) ok[k] = sub + k * L < nvec;

  for (long long r0 = warp0 * RPW; r0 < p.rows; r0 += warps * RPW) {
    const long long row = r0 + grp;
    const bool have = row < p.rows;
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + sub * EPV;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + sub * EPV;
    static_assert(!CAUSAL || SM, "the causal rule belongs to the softmax pair");
    const int live = (CAUSAL && have) ? static_cast<int>(live_cols(p, row)) : static_cast<int>(p.cols);
    const bool masked = CAUSAL && live < static_cast<int>(p.cols);
    bool in[K];                                    // vector k holds live data
#pragma unroll
    for (int k = 0; k < K; ++k) in[k] = have && ok[k] && (!CAUSAL || (sub + k * L) * EPV < live);
    uint4 raw[K];
#pragma unroll
    for (int k = 0; k < K; ++k)
      if (in[k]) raw[k] = ld_stream(xr + k * L * EPV);
    float v[K][EPV];
#pragma unroll
    for (int k = 0; k < K; ++k) {
      if (in[k]) {
        E::unpack(raw[k], v[k]);
        if (masked) {
#pragma unroll
          for (int j = 0; j < EPV; ++j) if ((sub + k * L) * EPV + j >= live) v[k][j] = kNegInf;
        }
      } else {
#pragma unroll
        for (int j = 0; j < EPV; ++j) v[k][j] = SM ? kNegInf : 0.f;
      }
    }

    if (SM) {
      float m = kNegInf;
#pragma unroll
      for (int k = 0; k < K; ++k)
#pragma unroll
        for (int j = 0; j < EPV; ++j) m = fmaxf(m, v[k][j]);
      const float M = group_max<L>(m);
      const float ms = (M == kNegInf) ? 0.f : M;             // keeps -inf - -inf out of the exponent
      const float neg_m_l2 = -ms * p.l2e;
      float s = 0.f;
#pragma unroll
      for (int k = 0; k < K; ++k)
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
          const float e = kFused ? ex2_approx(fmaf(v[k][j], p.l2e, neg_m_l2)) : exp_diff(v[k][j], ms, p.l2e);
          s += e;
          if (OP == OP_SOFTMAX) v[k][j] = e;                 // softmax keeps the exponentials
        }
      const float S = group_sum<L>(s);
      const bool dead = (M == kNegInf) && !(S != S);         // only -inf entries (a NaN row is not dead)
      const float scale = dead ? 0.f : __frcp_rn(S);
      const float lse = logf(S);
      const float m_out = dead ? 0.f : M, lse_out = dead ? 0.f : lse;   // a dead row comes out as -inf by itself
      const float neg_shift = -fmaf(m_out, p.scale, lse_out);           // 16-bit log-softmax: one multiply-add per element
      const float fill = (S != S) ? __int_as_float(0x7fc00000) : (OP == OP_SOFTMAX ? 0.f : kNegInf);
#pragma unroll
      for (int k = 0; k < K; ++k) {
        float o[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
          if (OP == OP_SOFTMAX) o[j] = v[k][j] * scale;
          else o[j] = kFused ? fmaf(v[k][j], p.scale, neg_shift) : fmaf(v[k][j] - m_out, p.scale, -lse_out);
        }
        if (masked) {
#pragma unroll
          for (int j = 0; j < EPV; ++j) if ((sub + k * L) * EPV + j >= live) o[j] = fill;
        }
        if (have && ok[k]) st_stream(yr + k * L * EPV, E::pack(o));
      }
    } else {
      float mean = 0.f, rstd;
      if (OP == OP_RMSNORM) {
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
          for (int j = 0; j < EPV; j += 2) { s0 = fmaf(v[k][j], v[k][j], s0); s1 = fmaf(v[k][j + 1], v[k][j + 1], s1); }
        rstd = rsqrt_refined(fmaf(group_sum<L>(s0 + s1), inv_cols, p.eps));
      } else {
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
          for (int j = 0; j < EPV; j += 2) { s0 += v[k][j]; s1 += v[k][j + 1]; }
        const float sum = group_sum<L>(s0 + s1);
        mean = sum * inv_cols;
        // (one residual step: the rounded 1 / cols would bias every row's mean the same way, by up to 2^-24 |mean|)
        mean = fmaf(fmaf(-mean, static_cast<float>(p.cols), sum), inv_cols, mean);
        float q0 = 0.f, q1 = 0.f;
#pragma unroll
        for (int k = 0; k < K; ++k) {
          if (ok[k]) {                                       // vectors beyond the row are not part of it
#pragma unroll
            for (int j = 0; j < EPV; j += 2) {
              const float d0 = v[k][j] - mean, d1 = v[k][j + 1] - mean;
              q0 = fmaf(d0, d0, q0); q1 = fmaf(d1, d1, q1);
            }
          }
        }
        rstd = rsqrt_refined(fmaf(group_sum<L>(q0 + q1), inv_cols, p.eps));
      }
      const float neg_mean_rstd = -mean * rstd;
      const T* gp = reinterpret_cast<const T*>(p.gamma) + sub * EPV;
      const T* bp = reinterpret_cast<const T*>(p.beta) + sub * EPV;
#pragma unroll
      for (int k = 0; k < K; ++k) {
        if (have && ok[k]) {
          float g[EPV], b[EPV], o[EPV];
#pragma unroll
          for (int j = 0; j < EPV; ++j) { g[j] = 1.f; b[j] = 0.f; }
          if (p.gamma != nullptr) E::unpack(ld_cached(gp + k * L * EPV), g);
          if (OP == OP_LAYERNORM && p.beta != nullptr) E::unpack(ld_cached(bp + k * L * EPV), b);
#pragma unroll
          for (int j = 0; j < EPV; ++j) {
            if (OP == OP_LAYERNORM) o[j] = kFused ? fmaf(fmaf(v[k][j], rstd, neg_mean_rstd), g[j], b[j])
                                                  : fmaf((v[k][j] - mean) * rstd, g[j], b[j]);
            else o[j] = v[k][j] * rstd * g[j];
          }
          st_stream(yr + k * L * EPV, E::pack(o));
        }
      }
    }
  }
}

}  // namespace akg
