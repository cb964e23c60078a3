// Two kernel families:
//   stream_kernel  any alignment, any row length; scalar accesses; one statistics
//                  pass over the row and a second read for the output pass
//   reg_kernel     16-byte aligned rows that fit the register file of one warp or
//                  one CTA: the row is read once with 128-bit loads, kept in
//                  registers, reduced, normalised and written with 128-bit stores
#pragma once

#include "common.cuh"

namespace akg {

// Apply the row scalars to one element (z already masked).
template <int OP>
__device__ __forceinline__ float apply_one(float z, const RowScalars& rs, float scale, float g, float b,
                                           float pre = 1.f) {
  if (OP == OP_SOFTMAX) return z * scale;                      // z holds exp(z - m_local)
  // pre: the fused pre-scale.  A dead row has p = q = 0 (see finalize), so its -inf entries come out as -inf
  if (OP == OP_LOG_SOFTMAX) return fmaf(z - rs.p, pre, -rs.q);
  if (OP == OP_LAYERNORM) return (z - rs.p) * rs.q * g + b;
  return z * rs.q * g;
}

// Value stored in positions that the causal rule masks (never read from memory).
template <int OP> __device__ __forceinline__ float masked_fill(const RowScalars& rs) {
  const float nan = __int_as_float(0x7fc00000);
  if (OP == OP_SOFTMAX) return (rs.q != rs.q) ? nan : 0.f;     // NaN rows are NaN everywhere
  return (rs.q != rs.q) ? nan : kNegInf;
}

// ------------------------------------------------------------------------------------
// reg_kernel: G threads own one row (G = 32: a warp per row, THREADS / 32 rows per CTA;
// G = THREADS: a CTA per row).  Thread t holds vectors t, t + G, ... (VPT of them).
// ------------------------------------------------------------------------------------
template <int OP, typename T, int G, int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS) reg_kernel(const RowParams p) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int N = VPT * EPV;
  constexpr int RPC = THREADS / G;
  constexpr int NW = G / 32;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  static_assert(G == 32 || G == THREADS, "a warp or a CTA per row");
  __shared__ Stat red[2][NW > 1 ? NW : 1];

  const int tg = threadIdx.x % G;
  const int grp = threadIdx.x / G;
  const int nvec = static_cast<int>(p.cols / EPV);
  int parity = 0;

  for (long long rb = static_cast<long long>(blockIdx.x) * RPC; rb < p.rows;
       rb += static_cast<long long>(gridDim.x) * RPC, parity ^= 1) {
    const long long row = rb + grp;
    if (G != THREADS && row >= p.rows) continue;               // warp-uniform

    const int live = SM ? static_cast<int>(live_cols(p, row)) : static_cast<int>(p.cols);
    const int live_vecs = (live + EPV - 1) / EPV;
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys;

    // ---- load: every 16-byte request of this thread is issued before any is used
    uint4 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const int idx = tg + k * G;
      if (idx < live_vecs) raw[k] = ld_stream(xr + static_cast<long long>(idx) * EPV);
    }
    float v[N];
    int n_valid = 0;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const int idx = tg + k * G;
      float f[EPV];
      if (idx < live_vecs) {
        E::unpack(raw[k], f);
      } else {
#pragma unroll
        for (int j = 0; j < EPV; ++j) f[j] = SM ? kNegInf : 0.f;
      }
      if (idx < nvec) n_valid += EPV;
#pragma unroll
      for (int j = 0; j < EPV; ++j) v[k * EPV + j] = f[j];
    }
    if (SM) {
      if (p.add != nullptr) {
        const T* ar = reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
          const int idx = tg + k * G;
          if (idx < live_vecs) {
            float a[EPV];
            E::unpack(ld_stream(ar + static_cast<long long>(idx) * EPV), a);
#pragma unroll
            for (int j = 0; j < EPV; ++j) v[k * EPV + j] = fmaf(a[j], p.inv_scale, v[k * EPV + j]);
          }
        }
      }
      if (live_vecs * EPV != live) {                           // ragged edge of the causal prefix
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
          const int idx = tg + k * G;
          if (idx == live_vecs - 1) {
#pragma unroll
            for (int j = 0; j < EPV; ++j)
              if (idx * EPV + j >= live) v[k * EPV + j] = kNegInf;
          }
        }
      }
    }

    // ---- statistics: thread tile -> warp -> CTA
    float m_local;
    Stat st = tile_stats<OP, N>(v, n_valid, m_local, p.l2e);
    st = (NW > 1) ? cta_reduce<OP, (NW > 1 ? NW : 1)>(st, red[parity], p.l2e) : warp_reduce<OP>(st, p.l2e);
    const RowScalars rs = finalize<OP>(st, p.cols, p.eps);
    float scale = 0.f;
    if (OP == OP_SOFTMAX) scale = (m_local == st.a) ? rs.q : exp_diff(m_local, st.a, p.l2e) * rs.q;

    // ---- normalise and store
    const float fill = SM ? masked_fill<OP>(rs) : 0.f;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const int idx = tg + k * G;
      if (idx < nvec) {
        float o[EPV];
        if (idx < live_vecs) {
          float g[EPV], b[EPV];
#pragma unroll
          for (int j = 0; j < EPV; ++j) { g[j] = 1.f; b[j] = 0.f; }
          if (!SM) {
            if (p.gamma != nullptr)
              E::unpack(ld_cached(reinterpret_cast<const T*>(p.gamma) + static_cast<long long>(idx) * EPV), g);
            if (OP == OP_LAYERNORM && p.beta != nullptr)
              E::unpack(ld_cached(reinterpret_cast<const T*>(p.beta) + static_cast<long long>(idx) * EPV), b);
          }
#pragma unroll
          for (int j = 0; j < EPV; ++j) {
            const bool masked = SM && (idx * EPV + j >= live);
            o[j] = masked ? fill : apply_one<OP>(v[k * EPV + j], rs, scale, g[j], b[j], p.scale);
          }
        } else {
#pragma unroll
          for (int j = 0; j < EPV; ++j) o[j] = fill;
        }
        st_stream(yr + static_cast<long long>(idx) * EPV, E::pack(o));
      }
    }
  }
}

// ------------------------------------------------------------------------------------
// stream_kernel: one CTA per row at a time, scalar accesses at any alignment.
// Pass 1 keeps running statistics per thread (online max / rescaled sum, Welford, or
// a sum of squares); pass 2 re-reads the row (served by L2 for all but huge rows).
// With a residual (normalisations), both passes form x + res; the sum is stored in pass 2
// only, element by element after its operands were read, so it may alias x or res.
// ------------------------------------------------------------------------------------
template <int OP, typename T, int THREADS>
__global__ void __launch_bounds__(THREADS) stream_kernel(const RowParams p) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int NW = THREADS / 32;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  __shared__ Stat red[2][NW];
  int parity = 0;

  for (long long row = blockIdx.x; row < p.rows; row += gridDim.x, parity ^= 1) {
    const long long live = SM ? live_cols(p, row) : p.cols;
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys;
    const T* ar = (SM && p.add != nullptr)
                      ? reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride
                      : nullptr;
    const T* rr = (!SM && p.res != nullptr) ? reinterpret_cast<const T*>(p.res) + row * p.rs : nullptr;
    T* sr = (!SM && p.res != nullptr && p.sum != nullptr) ? reinterpret_cast<T*>(p.sum) + row * p.ss : nullptr;

    Stat st = stat_identity<OP>();
    for (long long c = threadIdx.x; c < live; c += THREADS) {
      float z = E::load1(xr, c);
      if (!SM && rr != nullptr) z += E::load1(rr, c);
      if (SM) {
        if (ar != nullptr) z = fmaf(E::load1(ar, c), p.inv_scale, z);
        const float mn = fmaxf(st.a, z);
        const float ms = (mn == kNegInf) ? 0.f : mn;
        st.b = st.b * exp_diff(st.a, ms, p.l2e) + exp_diff(z, ms, p.l2e);
        st.a = mn;
      } else if (OP == OP_LAYERNORM) {
        st.a += 1.f;
        const float d = z - st.b;
        st.b += __fdividef(d, st.a);
        st.c += d * (z - st.b);
      } else {
        st.a += z * z;
      }
    }
    st = cta_reduce<OP, NW>(st, red[parity], p.l2e);
    const RowScalars rs = finalize<OP>(st, p.cols, p.eps);
    const float fill = SM ? masked_fill<OP>(rs) : 0.f;

    for (long long c = threadIdx.x; c < p.cols; c += THREADS) {
      float o;
      if (c < live) {
        float z = E::load1(xr, c);
        if (SM && ar != nullptr) z = fmaf(E::load1(ar, c), p.inv_scale, z);
        if (OP == OP_SOFTMAX) {
          // exp(z - M) / S; a dead row (no live entry) has q = 0 and p = 0
          o = exp_diff(z, rs.p, p.l2e) * rs.q;
        } else {
          if (!SM && rr != nullptr) {
            z += E::load1(rr, c);
            if (sr != nullptr) E::store1(sr, c, z);
          }
          const float g = (!SM && p.gamma != nullptr) ? E::load1(p.gamma, c) : 1.f;
          const float b = (OP == OP_LAYERNORM && p.beta != nullptr) ? E::load1(p.beta, c) : 0.f;
          o = apply_one<OP>(z, rs, 0.f, g, b, p.scale);
        }
      } else {
        o = fill;
      }
      E::store1(yr, c, o);
    }
  }
}

}  // namespace akg
