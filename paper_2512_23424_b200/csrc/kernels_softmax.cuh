// reg_softmax: register-resident softmax / log-softmax for rows that fit one warp or
// one CTA, with optional additive and causal masks.
//
// Thread t of the G threads of a row owns vectors t, t + G, ..., VPT of them.  With a
// causal mask only the first NK = ceil(live_vecs / G) of those iterations hold live
// data; the row body is compiled once per NK and selected by a CTA-uniform switch, so
// masked iterations cost nothing but their zero-fill stores (no predicated-off work).
// The exponential is evaluated once per live element, against the warp maximum; the
// cross-warp combine costs one exponential per warp.
#pragma once

#include "kernels_reg.cuh"

namespace akg {

// RING = false: the row is read from global memory; RING = true: from the shared-memory
// buffer at `ring_buf` that a bulk copy has filled with the row's live prefix.
template <int OP, typename T, int G, int VPT, int THREADS, int NK, bool RING = false>
__device__ __forceinline__ void softmax_row(const RowParams& p, long long row, int tg, int nvec, int live,
                                            int live_vecs, float (*red)[(G / 32) > 1 ? (G / 32) : 1],
                                            uint32_t ring_buf = 0) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int NW = G / 32;
  constexpr int NKA = NK > 0 ? NK : 1;
  const bool ragged = live_vecs * EPV != live;
  const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + tg * EPV;
  T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + tg * EPV;
  // only the last live iteration can hold vectors beyond the live prefix
  const bool last_ok = (NK > 0) && (tg + (NK - 1) * G < live_vecs);

  uint4 raw[NKA];
#pragma unroll
  for (int k = 0; k < NK; ++k)
    if (k < NK - 1 || last_ok)
      raw[k] = RING ? lds128(ring_buf + static_cast<uint32_t>(tg + k * G) * 16u) : ld_stream(xr + k * G * EPV);
  float v[NKA][EPV];
  float m_t = kNegInf;
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    if (k < NK - 1 || last_ok) {
      E::unpack(raw[k], v[k]);
      if (p.add != nullptr) {
        const T* ar = reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride + tg * EPV;
        float a[EPV];
        E::unpack(ld_stream(ar + k * G * EPV), a);
#pragma unroll
        for (int j = 0; j < EPV; ++j) v[k][j] += a[j];
      }
      if (k == NK - 1 && ragged && tg + k * G == live_vecs - 1) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) if ((tg + k * G) * EPV + j >= live) v[k][j] = kNegInf;
      }
    } else {
#pragma unroll
      for (int j = 0; j < EPV; ++j) v[k][j] = kNegInf;
    }
#pragma unroll
    for (int j = 0; j < EPV; ++j) m_t = fmaxf(m_t, v[k][j]);
  }

  const float m_w = warp_max(m_t);
  const float m_ws = (m_w == kNegInf) ? 0.f : m_w;        // keeps -inf - -inf out of the exponent
  float s_t = 0.f;
  // bf16 storage: one fused multiply-add forms the exponent (its rounding, below 1e-5
  // relative, is far inside the 2^-9 of the bf16 result); fp32 keeps the exact difference
  constexpr bool kFusedExponent = (sizeof(T) == 2);
  const float neg_m_l2 = -m_ws * kLog2e;
#pragma unroll
  for (int k = 0; k < NK; ++k) {
#pragma unroll
    for (int j = 0; j < EPV; ++j) {
      const float e = kFusedExponent ? ex2_approx(fmaf(v[k][j], kLog2e, neg_m_l2)) : exp_diff(v[k][j], m_ws);
      s_t += e;
      if (OP == OP_SOFTMAX) v[k][j] = e;
    }
  }
  const float s_w = warp_sum(s_t);

  float M = m_w, S = s_w, my_factor = 1.f;
  if (NW > 1) {
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = m_w; red[1][threadIdx.x >> 5] = s_w; }
    __syncthreads();
    M = red[0][0];
#pragma unroll
    for (int w = 1; w < NW; ++w) M = fmaxf(M, red[0][w]);
    const float Ms = (M == kNegInf) ? 0.f : M;
    S = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float mw = red[0][w];
      const float f = (mw == M) ? 1.f : exp_diff(mw, Ms);   // equal maxima (also +-inf): factor 1
      S = fmaf(red[1][w], f, S);
    }
    my_factor = (m_w == M) ? 1.f : exp_diff(m_w, Ms);
  }

  const bool dead = (M == kNegInf) && !(S != S);   // only NaN / -inf entries: a NaN row, not a dead one
  const float nan = __int_as_float(0x7fc00000);
  float scale = 0.f, lse_l = 0.f, fill;
  if (OP == OP_SOFTMAX) {
    scale = dead ? 0.f : my_factor * __frcp_rn(S);
    fill = (S != S) ? nan : 0.f;
  } else {
    lse_l = logf(S);
    fill = (S != S) ? nan : kNegInf;
  }

#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    const int idx = tg + k * G;
    float o[EPV];
    if (k < NK && (k < NK - 1 || last_ok)) {
#pragma unroll
      for (int j = 0; j < EPV; ++j) {
        if (OP == OP_SOFTMAX) o[j] = v[k < NK ? k : 0][j] * scale;
        else o[j] = dead ? kNegInf : (v[k < NK ? k : 0][j] - M) - lse_l;
      }
      if (k == NK - 1 && ragged && idx == live_vecs - 1) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) if (idx * EPV + j >= live) o[j] = fill;
      }
    } else {
#pragma unroll
      for (int j = 0; j < EPV; ++j) o[j] = fill;
    }
    if (idx < nvec) st_stream(yr + k * G * EPV, E::pack(o));
  }
}

template <int OP, typename T, int G, int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS, kRegMinBlocks<THREADS>) reg_softmax(const RowParams p) {
  pdl_prologue();
  constexpr int EPV = Elem<T>::EPV;
  constexpr int RPC = THREADS / G;
  constexpr int NW = G / 32;
  static_assert(OP == OP_SOFTMAX || OP == OP_LOG_SOFTMAX, "softmax pair only");
  static_assert(VPT <= 8, "row body is specialised for up to eight iterations");
  __shared__ float red[2][2][NW > 1 ? NW : 1];

  const int tg = threadIdx.x % G;
  const int grp = threadIdx.x / G;
  const int nvec = static_cast<int>(p.cols / EPV);
  int parity = 0;

  for (long long rb = static_cast<long long>(blockIdx.x) * RPC; rb < p.rows;
       rb += static_cast<long long>(gridDim.x) * RPC, parity ^= 1) {
    if (G != THREADS && rb + grp >= p.rows) continue;
    const long long row = balanced_row(p, rb + grp);
    const int live = static_cast<int>(live_cols(p, row));
    const int live_vecs = (live + EPV - 1) / EPV;
    const int nk = (live_vecs + G - 1) / G;             // uniform over the threads of the row
#define AKG_SM_CASE(NK_)                                                                          \
  case NK_:                                                                                       \
    if constexpr (NK_ <= VPT)                                                                     \
      softmax_row<OP, T, G, VPT, THREADS, NK_>(p, row, tg, nvec, live, live_vecs, red[parity]);   \
    break;
    switch (nk) {
      AKG_SM_CASE(0) AKG_SM_CASE(1) AKG_SM_CASE(2) AKG_SM_CASE(3) AKG_SM_CASE(4)
      AKG_SM_CASE(5) AKG_SM_CASE(6) AKG_SM_CASE(7) AKG_SM_CASE(8)
      default: break;
    }
#undef AKG_SM_CASE
  }
}

}  // namespace akg
