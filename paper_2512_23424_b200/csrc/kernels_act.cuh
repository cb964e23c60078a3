// Gated activations: SiLU-and-Mul and GELU-and-Mul (named among the operators of the paper's
// benchmark, Section 3.6).  x is [rows, 2 d]: the first d columns of a row are the gate a, the
// last d the factor b; y[r, c] = act(a[r, c]) * b[r, c].  Purely element-wise: two reads and
// one write per output element, bound by HBM.  A CTA walks a chunk of one row; every thread
// issues its 2 * U vector loads before the first use; whole tiles are unpredicated.
//   SiLU        a / (1 + e^-a)
//   GELU        0.5 a (1 + erf(a / sqrt 2)) = a Phi(a), Phi from an own approximation (below)
//   GELU (tanh) 0.5 a (1 + tanh(u)), u = sqrt(2 / pi) (a + 0.044715 a^3); since
//               0.5 (1 + tanh u) = 1 / (1 + e^(-2u)) it costs the same as SiLU
#pragma once

#include "common.cuh"

namespace akg {

enum Act : int { ACT_SILU = 0, ACT_GELU = 1, ACT_GELU_TANH = 2 };

// 1 / (1 + e^-t): two special-function evaluations (about 1 ulp each), both flushing
// subnormal results to zero: a sigmoid below 2^-126 (t < -87.3) is returned as 0
__device__ __forceinline__ float sigmoid_f32(float t) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + ex2_approx(-t * kLog2e)));
  return r;
}

// The normal distribution function Phi(a) = 0.5 erfc(-a / sqrt 2).  With x = |a| / sqrt 2 and
// t = 1 / (1 + x / 2), exp(x^2) erfc(x) / t is smooth on (0, 1] and is fitted by a polynomial
// h(t) (coefficients and their measured error: gen_phi_coeffs.py), so
//   Phi(-|a|) = 0.5 exp(-a^2 / 2) t h(t)
// holds its RELATIVE accuracy in the far left tail, where 1 + erf(.) cancels: degree 9 is
// 4e-7 near the centre (fp32 output), degree 5 is 7e-5 (enough for a 16-bit output; degree 4,
// 3.9e-4, failed the parity test on bf16).  One reciprocal, one exponential, DEG multiply-adds;
// the factor 0.5 is folded into the coefficients at compile time.
template <int DEG> __device__ __forceinline__ float normal_cdf(float a) {
  constexpr float c9[10] = {2.820947468e-01f, 2.821037173e-01f, 2.465246618e-01f, 1.803003252e-01f,
                            5.878400058e-02f, 7.814583927e-02f, -1.966046691e-01f, 2.911409736e-02f,
                            6.519216299e-02f, -2.565501817e-02f};
  constexpr float c5[6] = {2.820831239e-01f, 2.829633951e-01f, 2.377409786e-01f,
                           2.017114013e-01f, 8.792584389e-02f, -9.248869121e-02f};
  static_assert(DEG == 9 || DEG == 5, "fitted degrees");
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(fabsf(a), 0.35355339059327376220f, 1.0f)));
  float h = 0.5f * ((DEG == 9) ? c9[9] : c5[5]);
#pragma unroll
  for (int i = DEG - 1; i >= 0; --i) h = fmaf(h, t, 0.5f * ((DEG == 9) ? c9[i] : c5[i]));
  const float q = t * h * ex2_approx(a * a * (-0.5f * kLog2e));             // Phi(-|a|)
  return a > 0.f ? 1.0f - q : q;
}

// degree of the fit by storage type: fp32 9, 16-bit 5
template <typename T> constexpr int kPhiDegree = (sizeof(T) == 4) ? 9 : 5;

template <int ACT, typename T> __device__ __forceinline__ float act_gate(float a) {
  if (ACT == ACT_SILU) return a * sigmoid_f32(a);
  if (ACT == ACT_GELU) return a * normal_cdf<kPhiDegree<T>>(a);
  const float u2 = 1.5957691216057307117f * fmaf(0.044715f * a * a, a, a);      // 2 u
  return a * sigmoid_f32(u2);
}

// VEC: 16-byte vectors (d, the strides and the bases are multiples of a vector), else elements.
template <int ACT, typename T, bool VEC, int U>
__global__ void __launch_bounds__(256, 4) act_mul_kernel(const ActParams p) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int W = VEC ? E::EPV : 1;
  const long long dv = p.d / W;                                   // lanes of work per row
  const long long step = static_cast<long long>(blockDim.x);
  // vector indices inside a row fit 32 bits (the entry point checks d): the inner loop then
  // costs one wide multiply-add per address instead of 64-bit index arithmetic per access,
  // which was a third of the instructions of the 16-bit GELU (11 of 31 per element)
  const int dvi = static_cast<int>(dv);
  const int stepi = static_cast<int>(blockDim.x);
  for (long long row = blockIdx.y; row < p.rows; row += gridDim.y) {
    const T* xa = reinterpret_cast<const T*>(p.x) + row * p.xs;
    const T* xb = xa + p.d;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys;
    if (VEC) {
      const uint4* pa = reinterpret_cast<const uint4*>(xa);
      const uint4* pb = reinterpret_cast<const uint4*>(xb);
      uint4* py = reinterpret_cast<uint4*>(yr);
      for (int v0 = static_cast<int>(blockIdx.x) * stepi * U + static_cast<int>(threadIdx.x); v0 < dvi;
           v0 += static_cast<int>(gridDim.x) * stepi * U) {
        uint4 ra[U], rb[U];
        const bool whole = v0 + (U - 1) * stepi < dvi;
#pragma unroll
        for (int u = 0; u < U; ++u) if (whole || v0 + u * stepi < dvi) ra[u] = ld_stream(pa + (v0 + u * stepi));
#pragma unroll
        for (int u = 0; u < U; ++u) if (whole || v0 + u * stepi < dvi) rb[u] = ld_stream(pb + (v0 + u * stepi));
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (whole || v0 + u * stepi < dvi) {
            float a[E::EPV], b[E::EPV], o[E::EPV];
            E::unpack(ra[u], a);
            E::unpack(rb[u], b);
#pragma unroll
            for (int j = 0; j < E::EPV; ++j) o[j] = act_gate<ACT, T>(a[j]) * b[j];
            st_stream(py + (v0 + u * stepi), E::pack(o));
          }
        }
      }
      continue;
    }
    for (long long v0 = static_cast<long long>(blockIdx.x) * step * U + threadIdx.x; v0 < dv;
         v0 += static_cast<long long>(gridDim.x) * step * U) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const long long c = v0 + u * step;
        if (c < dv) E::store1(yr, c, act_gate<ACT, T>(E::load1(xa, c)) * E::load1(xb, c));
      }
    }
  }
}

}  // namespace akg
