// Lean register-resident normalisation (the fast path of the REG family).
//
//   norm_row_full   one row of LayerNorm / RMSNorm when the row is exactly G * VPT
//                   vectors: no predicates, equal-count pairwise mean / M2 merges (no
//                   divisions), one CTA barrier per row.  The row comes either from
//                   global memory or from a shared-memory buffer a bulk copy filled.
//   reg_norm_full   the kernel around it: a warp or a CTA per row, grid-stride
//
// The instruction count per element is what bounds these kernels once the loads are
// wide enough, so everything per-row (reductions, reciprocal square root) is kept to a
// few dozen instructions per thread.
#pragma once

#include "kernels_basic.cuh"
#include "tma.cuh"

namespace akg {

// s / N for the N values of a thread.  Unless N is a power of two the rounded reciprocal is off by up to half an
// ulp, and the product s * (1 / N) is off the same way in every thread of every row: a bias of the row mean of
// up to 2^-24 |mean| that no merge averages out.  It shows where |mean| is many standard deviations (mean / std
// = 30: results next to zero were off by 6e-6, beyond two ulps of a 16-bit result); one residual step takes it out.
template <int N> __device__ __forceinline__ float thread_mean(float s) {
  constexpr float inv = 1.0f / N;
  const float q = s * inv;
  if constexpr ((N & (N - 1)) == 0) return q;
  return fmaf(fmaf(-q, static_cast<float>(N), s), inv, q);
}

// Mean of the NW warp means held by lanes 0 .. NW - 1 (mw; `mine` marks them): lane 0's value plus the mean of
// the differences from it, so that the rounded 1 / NW (inv_warps; NW is any number up to 32) and the rounding of
// the sum act on the differences only, not on the mean's own magnitude.
__device__ __forceinline__ float mean_of_warp_means(float mw, bool mine, float inv_warps) {
  const float ref = __shfl_sync(0xffffffffu, mw, 0);
  return fmaf(warp_sum(mine ? mw - ref : 0.f), inv_warps, ref);
}

// Occupancy target of the register-resident kernels: at least 1024 threads per SM, i.e.
// at most 64 registers per thread (occupancy, not instruction count, bounds them next).
template <int THREADS> constexpr int kRegMinBlocks = (1024 / THREADS) > 0 ? (1024 / THREADS) : 1;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
  return v;
}

// red: [2][NW] floats of shared memory reserved for this row (callers alternate two sets).
template <int OP, typename T, int G, int VPT, int THREADS, bool RING = false>
__device__ __forceinline__ void norm_row_full(const RowParams& p, long long row, int tg,
                                              float (*red)[(G / 32) > 1 ? (G / 32) : 1],
                                              uint32_t ring_buf = 0, bool dead = false) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int N = VPT * EPV;
  constexpr int NW = G / 32;
  static_assert(OP == OP_LAYERNORM || OP == OP_RMSNORM, "normalisations only");
  static_assert((NW & (NW - 1)) == 0, "warps per row must be a power of two");
  const float inv_cols = 1.0f / static_cast<float>(N * G);
  const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + tg * EPV;
  T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + tg * EPV;

  uint4 raw[VPT];
#pragma unroll
  for (int k = 0; k < VPT; ++k)
    raw[k] = RING ? lds128(ring_buf + static_cast<uint32_t>(tg + k * G) * 16u) : ld_stream(xr + k * G * EPV);
  float v[N];
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    float f[EPV];
    E::unpack(raw[k], f);
#pragma unroll
    for (int j = 0; j < EPV; ++j) v[k * EPV + j] = f[j];
  }

  float mean = 0.f, rstd;
  if (OP == OP_RMSNORM) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) { s0 = fmaf(v[i], v[i], s0); s1 = fmaf(v[i + 1], v[i + 1], s1); }
    float ss = warp_sum(s0 + s1);
    if (NW > 1) {
      if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = ss;
      __syncthreads();
      ss = red[0][threadIdx.x & (NW - 1)];
#pragma unroll
      for (int m = NW / 2; m >= 1; m >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, m);
    }
    rstd = rsqrt_refined(fmaf(ss, inv_cols, p.eps));
  } else {
    // thread tile: exact two-pass mean and M2 over N values
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) { s0 += v[i]; s1 += v[i + 1]; }
    float mu = thread_mean<N>(s0 + s1);
    float q0 = 0.f, q1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) {
      const float d0 = v[i] - mu, d1 = v[i + 1] - mu;
      q0 = fmaf(d0, d0, q0); q1 = fmaf(d1, d1, q1);
    }
    float m2 = q0 + q1;
    // equal-count pairwise merges: both sides hold c values, so
    //   mean = (ma + mb) / 2,  M2 = M2a + M2b + (mb - ma)^2 * c / 2
    float half_c = 0.5f * N;
#pragma unroll
    for (int m = 1; m <= 16; m <<= 1) {
      const float mb = __shfl_xor_sync(0xffffffffu, mu, m);
      const float qb = __shfl_xor_sync(0xffffffffu, m2, m);
      const float d = mb - mu;
      mu = fmaf(0.5f, d, mu);
      m2 = fmaf(d * d, half_c, m2 + qb);
      half_c *= 2.f;
    }
    if (NW > 1) {
      if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = mu; red[1][threadIdx.x >> 5] = m2; }
      __syncthreads();
      mu = red[0][threadIdx.x & (NW - 1)];
      m2 = red[1][threadIdx.x & (NW - 1)];
#pragma unroll
      for (int m = 1; m < NW; m <<= 1) {
        const float mb = __shfl_xor_sync(0xffffffffu, mu, m);
        const float qb = __shfl_xor_sync(0xffffffffu, m2, m);
        const float d = mb - mu;
        mu = fmaf(0.5f, d, mu);
        m2 = fmaf(d * d, half_c, m2 + qb);
        half_c *= 2.f;
      }
    }
    mean = mu;
    rstd = rsqrt_refined(fmaf(m2, inv_cols, p.eps));
  }

  // (ring kernels: a thread whose wait for the row ran out took part in the reduction above, for its
  // CTA's barrier, and stores nothing)
  if (RING && dead) return;
  // 16-bit storage: (x - mean) * rstd as one fused multiply-add with the row constant -mean * rstd
  // (its rounding, 2^-24 |mean| rstd, is far inside the 2^-9 of the stored result); fp32 keeps
  // the exact difference
  constexpr bool kFusedCentre = (sizeof(T) == 2);
  const float neg_mean_rstd = -mean * rstd;
  const T* gp = reinterpret_cast<const T*>(p.gamma) + tg * EPV;
  const T* bp = reinterpret_cast<const T*>(p.beta) + tg * EPV;
  // every affine vector present (the usual call): unpack straight into the arithmetic; otherwise
  // defaults are materialised per element first (two instructions per element that the usual call
  // would pay for nothing: measured 1.75 of 16 instructions per bf16 LayerNorm element)
  const bool affine_all = p.gamma != nullptr && (OP != OP_LAYERNORM || p.beta != nullptr);
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    float g[EPV], b[EPV], o[EPV];
    if (affine_all) {
      E::unpack(ld_cached(gp + k * G * EPV), g);
      if (OP == OP_LAYERNORM) E::unpack(ld_cached(bp + k * G * EPV), b);
    } else {
#pragma unroll
      for (int j = 0; j < EPV; ++j) { g[j] = 1.f; b[j] = 0.f; }
      if (p.gamma != nullptr) E::unpack(ld_cached(gp + k * G * EPV), g);
      if (OP == OP_LAYERNORM && p.beta != nullptr) E::unpack(ld_cached(bp + k * G * EPV), b);
    }
#pragma unroll
    for (int j = 0; j < EPV; ++j) {
      if (OP == OP_LAYERNORM) o[j] = kFusedCentre ? fmaf(fmaf(v[k * EPV + j], rstd, neg_mean_rstd), g[j], b[j])
                                                  : fmaf((v[k * EPV + j] - mean) * rstd, g[j], b[j]);
      else o[j] = v[k * EPV + j] * rstd * g[j];
    }
    st_stream(yr + k * G * EPV, E::pack(o));
  }
}

// Row statistics of the flex scheme: every thread of the CTA holds N values of the row; NW
// warps.  red: [2][32] floats of shared memory reserved for this row.  One barrier.
template <int OP, int N>
__device__ __forceinline__ void flex_row_stats(const float (&v)[N], float (*red)[32], int NW, float inv_warps,
                                               float inv_cols, float eps, float& mean, float& rstd) {
  mean = 0.f;
  if (OP == OP_RMSNORM) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) { s0 = fmaf(v[i], v[i], s0); s1 = fmaf(v[i + 1], v[i + 1], s1); }
    float ss = warp_sum(s0 + s1);
    if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = ss;
    __syncthreads();
    ss = 0.f;
    for (int w = 0; w < NW; ++w) ss += red[0][w];
    rstd = rsqrt_refined(fmaf(ss, inv_cols, eps));
  } else {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) { s0 += v[i]; s1 += v[i + 1]; }
    float mu = thread_mean<N>(s0 + s1);
    float q0 = 0.f, q1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) {
      const float d0 = v[i] - mu, d1 = v[i + 1] - mu;
      q0 = fmaf(d0, d0, q0); q1 = fmaf(d1, d1, q1);
    }
    float m2 = q0 + q1;
    float half_c = 0.5f * N;
#pragma unroll
    for (int m = 1; m <= 16; m <<= 1) {                 // equal-count merges inside the warp
      const float mb = __shfl_xor_sync(0xffffffffu, mu, m);
      const float qb = __shfl_xor_sync(0xffffffffu, m2, m);
      const float d = mb - mu;
      mu = fmaf(0.5f, d, mu);
      m2 = fmaf(d * d, half_c, m2 + qb);
      half_c *= 2.f;
    }
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = mu; red[1][threadIdx.x >> 5] = m2; }
    __syncthreads();
    // lane l takes warp l's pair (nothing beyond the CTA's warps): three shuffle sums instead of three
    // shared loads and a dependent chain per warp of the CTA
    const bool mine = static_cast<int>(threadIdx.x & 31) < NW;
    const float mw = mine ? red[0][threadIdx.x & 31] : 0.f;
    const float qsum = warp_sum(mine ? red[1][threadIdx.x & 31] : 0.f);
    mean = mean_of_warp_means(mw, mine, inv_warps);
    const float d = mine ? mw - mean : 0.f;
    const float dev = warp_sum(d * d);
    rstd = rsqrt_refined(fmaf(fmaf(dev, 32.0f * N, qsum), inv_cols, eps));
  }
}

// The cross-thread part of flex_row_stats on its own: every thread brings the statistics of its own n
// values - LayerNorm: (mu, m2) = their mean and sum of squared deviations; RMSNorm: mu = their sum of squares.
template <int OP>
__device__ __forceinline__ void flex_merge(float mu, float m2, int n, float (*red)[32], int NW, float inv_warps,
                                           float inv_cols, float eps, float& mean, float& rstd) {
  mean = 0.f;
  if (OP == OP_RMSNORM) {
    float ss = warp_sum(mu);
    if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = ss;
    __syncthreads();
    ss = 0.f;
    for (int w = 0; w < NW; ++w) ss += red[0][w];
    rstd = rsqrt_refined(fmaf(ss, inv_cols, eps));
  } else {
    float half_c = 0.5f * static_cast<float>(n);
#pragma unroll
    for (int m = 1; m <= 16; m <<= 1) {                 // equal-count merges inside the warp
      const float mb = __shfl_xor_sync(0xffffffffu, mu, m);
      const float qb = __shfl_xor_sync(0xffffffffu, m2, m);
      const float d = mb - mu;
      mu = fmaf(0.5f, d, mu);
      m2 = fmaf(d * d, half_c, m2 + qb);
      half_c *= 2.f;
    }
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = mu; red[1][threadIdx.x >> 5] = m2; }
    __syncthreads();
    const bool mine = static_cast<int>(threadIdx.x & 31) < NW;
    const float mw = mine ? red[0][threadIdx.x & 31] : 0.f;
    const float qsum = warp_sum(mine ? red[1][threadIdx.x & 31] : 0.f);
    mean = mean_of_warp_means(mw, mine, inv_warps);
    const float d = mine ? mw - mean : 0.f;
    const float dev = warp_sum(d * d);
    rstd = rsqrt_refined(fmaf(fmaf(dev, 32.0f * static_cast<float>(n), qsum), inv_cols, eps));
  }
}

// reg_norm_packed: reg_norm_flex for the 16-bit types with the row kept PACKED in registers (four
// registers per vector instead of eight) and the stored values fed to the arithmetic as they are
// (Elem::add_wide / sub_wide / fma_wide: widened inside the instruction, on the FMA pipe).  Eight vectors
// per thread then fit 64 registers, so a row needs half the threads of the widened form: the per-row
// work that every thread pays (shuffle merges, barrier, the warps' pairs) is spread over twice the
// elements, eight loads per thread are in flight, and four CTAs of 256 share an SM.
//   RMSNorm   sum x^2 with one fma_wide per element; y = (x * w) * rstd, the product of two 16-bit values
//             being exact in fp32
//   LayerNorm exact two sweeps over the thread's values (sum with add_wide, deviations with sub_wide),
//             equal-count merges as in reg_norm_flex; y = beta + ((x - mean) * rstd) * gamma
template <int OP, typename T, int VPT>
__global__ void __launch_bounds__(1024, 1) reg_norm_packed(const RowParams p, const float inv_warps) {
  pdl_prologue();
  using E = Elem<T>;
  static_assert(sizeof(T) == 2, "16-bit storage only");
  static_assert(OP == OP_LAYERNORM || OP == OP_RMSNORM, "normalisations only");
  constexpr int EPV = E::EPV;
  constexpr int N = VPT * EPV;
  __shared__ float red[2][2][32];
  const int G = blockDim.x;
  const int NW = G >> 5;
  const int tg = threadIdx.x;
  const float inv_cols = 1.0f / static_cast<float>(p.cols);
  const bool affine_all = p.gamma != nullptr && (OP != OP_LAYERNORM || p.beta != nullptr);
  int parity = 0;
  for (long long row = blockIdx.x; row < p.rows; row += gridDim.x, parity ^= 1) {
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + tg * EPV;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + tg * EPV;
    uint4 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) raw[k] = ld_stream(xr + static_cast<long long>(k) * G * EPV);
    float mu, m2 = 0.f;
    if (OP == OP_RMSNORM) {
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(w[i], h0, h1);
          s0 = E::fma_wide(h0, h0, s0);
          s1 = E::fma_wide(h1, h1, s1);
        }
      }
      mu = s0 + s1;
    } else {
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(w[i], h0, h1);
          s0 = E::add_wide(h0, s0);
          s1 = E::add_wide(h1, s1);
        }
      }
      mu = thread_mean<N>(s0 + s1);
      float q0 = 0.f, q1 = 0.f;
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(w[i], h0, h1);
          const float d0 = E::sub_wide(h0, mu), d1 = E::sub_wide(h1, mu);
          q0 = fmaf(d0, d0, q0);
          q1 = fmaf(d1, d1, q1);
        }
      }
      m2 = q0 + q1;
    }
    float mean, rstd;
    flex_merge<OP>(mu, m2, N, red[parity], NW, inv_warps, inv_cols, p.eps, mean, rstd);

    const T* gp = reinterpret_cast<const T*>(p.gamma) + tg * EPV;
    const T* bp = reinterpret_cast<const T*>(p.beta) + tg * EPV;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const uint32_t xw[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
      uint32_t out[4];
      if (affine_all) {
        const uint4 gv = ld_cached(gp + static_cast<long long>(k) * G * EPV);
        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
        if (OP == OP_RMSNORM) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            unsigned short x0, x1, g0, g1;
            halves(xw[i], x0, x1);
            halves(gw[i], g0, g1);
            out[i] = E::pack2(E::fma_wide(x0, g0, 0.f) * rstd, E::fma_wide(x1, g1, 0.f) * rstd);
          }
        } else {
          const uint4 bv = ld_cached(bp + static_cast<long long>(k) * G * EPV);
          const uint32_t bw[4] = {bv.x, bv.y, bv.z, bv.w};
          float ga[EPV];
          E::unpack(gv, ga);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            unsigned short x0, x1, b0, b1;
            halves(xw[i], x0, x1);
            halves(bw[i], b0, b1);
            out[i] = E::pack2(E::add_wide(b0, E::sub_wide(x0, mean) * rstd * ga[2 * i]),
                              E::add_wide(b1, E::sub_wide(x1, mean) * rstd * ga[2 * i + 1]));
          }
        }
      } else {
        // an absent gamma or beta (1 / 0): the plain formula on unpacked values
        float v[EPV], g[EPV], b[EPV], o[EPV];
        E::unpack(raw[k], v);
#pragma unroll
        for (int j = 0; j < EPV; ++j) { g[j] = 1.f; b[j] = 0.f; }
        if (p.gamma != nullptr) E::unpack(ld_cached(gp + static_cast<long long>(k) * G * EPV), g);
        if (OP == OP_LAYERNORM && p.beta != nullptr) E::unpack(ld_cached(bp + static_cast<long long>(k) * G * EPV), b);
#pragma unroll
        for (int j = 0; j < EPV; ++j)
          o[j] = (OP == OP_LAYERNORM) ? fmaf((v[j] - mean) * rstd, g[j], b[j]) : v[j] * rstd * g[j];
        const uint4 ov = E::pack(o);
        out[0] = ov.x; out[1] = ov.y; out[2] = ov.z; out[3] = ov.w;
      }
      st_stream(yr + static_cast<long long>(k) * G * EPV, make_uint4(out[0], out[1], out[2], out[3]));
    }
  }
}

// reg_norm_flex: the same predicate-free scheme for rows of exactly blockDim.x * VPT
// vectors where blockDim.x is any multiple of 32 (hidden sizes such as 5120, 6144, 7168).
// A CTA per row.  Every warp holds the same number of values, so the warps' (mean, M2)
// pairs combine without divisions:  mean = avg(mean_w),  M2 = sum(M2_w) + c * sum((mean_w - mean)^2)
// with c = values per warp; every thread reads the NW pairs from shared memory.
// (64 values per thread, i.e. eight 16-bit vectors, are only launched with up to 256 threads and get
// 128 registers; everything else keeps the 64-register bound of a full-size CTA)
template <int OP, typename T, int VPT>
__global__ void __launch_bounds__((VPT * Elem<T>::EPV >= 64) ? 256 : 1024, (VPT * Elem<T>::EPV >= 64) ? 2 : 1)
reg_norm_flex(const RowParams p, const float inv_warps) {
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
  int parity = 0;
  for (long long row = blockIdx.x; row < p.rows; row += gridDim.x, parity ^= 1) {
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + tg * EPV;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + tg * EPV;
    uint4 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) raw[k] = ld_stream(xr + static_cast<long long>(k) * G * EPV);
    float v[N];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      float f[EPV];
      E::unpack(raw[k], f);
#pragma unroll
      for (int j = 0; j < EPV; ++j) v[k * EPV + j] = f[j];
    }
    float mean, rstd;
    flex_row_stats<OP, N>(v, red[parity], NW, inv_warps, inv_cols, p.eps, mean, rstd);
    constexpr bool kFusedCentre = (sizeof(T) == 2);        // as in norm_row_full
    const float neg_mean_rstd = -mean * rstd;
    const T* gp = reinterpret_cast<const T*>(p.gamma) + tg * EPV;
    const T* bp = reinterpret_cast<const T*>(p.beta) + tg * EPV;
    const bool affine_all = p.gamma != nullptr && (OP != OP_LAYERNORM || p.beta != nullptr);   // as in norm_row_full
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      float g[EPV], b[EPV], o[EPV];
      if (affine_all) {
        E::unpack(ld_cached(gp + static_cast<long long>(k) * G * EPV), g);
        if (OP == OP_LAYERNORM) E::unpack(ld_cached(bp + static_cast<long long>(k) * G * EPV), b);
      } else {
#pragma unroll
        for (int j = 0; j < EPV; ++j) { g[j] = 1.f; b[j] = 0.f; }
        if (p.gamma != nullptr) E::unpack(ld_cached(gp + static_cast<long long>(k) * G * EPV), g);
        if (OP == OP_LAYERNORM && p.beta != nullptr) E::unpack(ld_cached(bp + static_cast<long long>(k) * G * EPV), b);
      }
#pragma unroll
      for (int j = 0; j < EPV; ++j) {
        if (OP == OP_LAYERNORM) o[j] = kFusedCentre ? fmaf(fmaf(v[k * EPV + j], rstd, neg_mean_rstd), g[j], b[j])
                                                    : fmaf((v[k * EPV + j] - mean) * rstd, g[j], b[j]);
        else o[j] = v[k * EPV + j] * rstd * g[j];
      }
      st_stream(yr + static_cast<long long>(k) * G * EPV, E::pack(o));
    }
  }
}

template <int OP, typename T, int G, int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS, kRegMinBlocks<THREADS>) reg_norm_full(const RowParams p) {
  pdl_prologue();
  constexpr int RPC = THREADS / G;
  constexpr int NW = G / 32;
  __shared__ float red[2][2][NW > 1 ? NW : 1];
  const int tg = threadIdx.x % G;
  const int grp = threadIdx.x / G;
  int parity = 0;
  for (long long rb = static_cast<long long>(blockIdx.x) * RPC; rb < p.rows;
       rb += static_cast<long long>(gridDim.x) * RPC, parity ^= 1) {
    const long long row = rb + grp;
    if (G != THREADS && row >= p.rows) continue;
    norm_row_full<OP, T, G, VPT, THREADS>(p, row, tg, red[parity]);
  }
}

}  // namespace akg
