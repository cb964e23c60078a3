// axis_reg_kernel: the non-last-axis operators with the strip resident in registers
// (reduce <= nf * R) - the common case of the paper's RMSNorm sketch, whose reduced axis is
// a feature axis of a few dozen entries (Unified Sketch figure, Section 3.2.1).
//
// A CTA is nf x nc warps: warp (wf, wc) owns the 32 * W columns of column block wc and
// the rows f = wf, wf + nf, ... (at most R of them) of the reduced axis.  Every thread
// issues its R row loads back to back and folds them into per-column partial statistics.
// The nf warps of a column block then share the merge instead of repeating it: each takes
// 32 * W / nf columns, combines the nf partials of a column, derives its two scalars
// (max and 1 / sum, mean and 1 / std, ...) once, and publishes them through shared memory.
// With nf == 1 a thread owns whole columns and shared memory is not touched.  The values
// are normalised from the registers they were loaded into, so HBM and L2 see each element
// once in each direction.  nf and nc are launch arguments (blockDim.x = 32 * nf * nc): one
// instantiation per R serves every length of the reduced axis up to 16 * R.  The grid is
// (strips of one outer index, outer indices); no thread divides anything.
#pragma once

#include "kernels_reg.cuh"

namespace akg {

template <typename T, bool VEC> struct AxisRaw;

template <typename T> struct AxisRaw<T, true> {
  using E = Elem<T>;
  using Raw = uint4;
  static constexpr int W = E::EPV;
  static __device__ __forceinline__ Raw load(const T* p) { return ld_stream(p); }
  static __device__ __forceinline__ Raw fill(float v) {
    float t[W];
#pragma unroll
    for (int j = 0; j < W; ++j) t[j] = v;
    return E::pack(t);
  }
  static __device__ __forceinline__ void unpack(const Raw& r, float (&f)[W]) { E::unpack(r, f); }
  static __device__ __forceinline__ Raw pack(const float (&f)[W]) { return E::pack(f); }
  static __device__ __forceinline__ void store(T* p, const Raw& r) { st_stream(p, r); }
};

template <typename T> struct AxisRaw<T, false> {
  using E = Elem<T>;
  using Raw = float;                        // a bf16 value widens exactly
  static constexpr int W = 1;
  static __device__ __forceinline__ Raw load(const T* p) { return E::load1(p, 0); }
  static __device__ __forceinline__ Raw fill(float v) { return v; }
  static __device__ __forceinline__ void unpack(const Raw& r, float (&f)[1]) { f[0] = r; }
  static __device__ __forceinline__ Raw pack(const float (&f)[1]) { return f[0]; }
  static __device__ __forceinline__ void store(T* p, const Raw& r) { E::store1(p, 0, r); }
};

constexpr int kAxisMaxWarps = 16;

// Shared memory of one CTA in floats: partials [KS][nf * nc][32 W], then scalars [2][nc][32 W].
__host__ __device__ constexpr unsigned axis_reg_smem_floats(int ks, int nf, int nc, int w) {
  return nf > 1 ? static_cast<unsigned>((ks * nf * nc + 2 * nc) * 32 * w) : 0u;
}

// The two scalars of a column from its merged statistics:
//   softmax     : p = M (0 for a column without live entry), q = 1 / S (0 for such a column)
//   log-softmax : p = M, q = ln S (both 0 for such a column: x - 0 - 0 = -inf)
//   LayerNorm   : p = mean, q = 1 / sqrt(M2 / F + eps)
//   RMSNorm     : q = 1 / sqrt(sum of squares / F + eps)
template <int OP>
__device__ __forceinline__ void axis_scalars(float a, float b, float inv_f, float eps, float& p, float& q) {
  if (OpTraits<OP>::kSoftmaxLike) {
    const bool dead = (a == kNegInf) && !(b != b);         // only NaN / -inf entries: a NaN column
    p = dead ? 0.f : a;
    q = dead ? 0.f : (OP == OP_SOFTMAX ? __frcp_rn(b) : logf(b));
  } else if (OP == OP_LAYERNORM) {
    p = a;
    q = rsqrt_refined(fmaf(b, inv_f, eps));
  } else {
    p = 0.f;
    q = rsqrt_refined(fmaf(a, inv_f, eps));
  }
}

// Phase 1 of a strip: load this thread's rows and fold them into per-column partials
// ((m, s), (mean, M2) or the sum of squares).  FULL: all R rows exist and the columns are
// inside the array, so nothing is predicated (the case of every thread but those of a
// ragged last warp-row or column block).
template <int OP, typename T, bool VEC, int R, bool FULL>
__device__ __forceinline__ void axis_reg_load(const T* px, long long xstep, bool active, int nt,
                                              typename AxisRaw<T, VEC>::Raw (&raw)[R],
                                              float (&sa)[AxisRaw<T, VEC>::W], float (&sb)[AxisRaw<T, VEC>::W]) {
  using A = AxisRaw<T, VEC>;
  constexpr int W = A::W;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  constexpr bool KEEP = (OP == OP_SOFTMAX) && (sizeof(T) == 4);
#pragma unroll
  for (int r = 0; r < R; ++r, px += xstep) {
    if (FULL) raw[r] = A::load(px);
    else raw[r] = (active && r < nt) ? A::load(px) : A::fill(SM ? kNegInf : 0.f);
  }
  if (SM) {
#pragma unroll
    for (int j = 0; j < W; ++j) sa[j] = kNegInf;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) sa[j] = fmaxf(sa[j], v[j]);
    }
    float ms[W];
#pragma unroll
    for (int j = 0; j < W; ++j) { ms[j] = (sa[j] == kNegInf) ? 0.f : sa[j]; sb[j] = 0.f; }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) { v[j] = exp_diff(v[j], ms[j]); sb[j] += v[j]; }
      if (KEEP) raw[r] = A::pack(v);
    }
  } else if (OP == OP_LAYERNORM) {
#pragma unroll
    for (int j = 0; j < W; ++j) { sa[j] = 0.f; sb[j] = 0.f; }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) sa[j] += v[j];             // rows not held are zeros
    }
    const float inv_nt = FULL ? (1.0f / R) : ((nt > 0) ? __frcp_rn(static_cast<float>(nt)) : 0.f);
#pragma unroll
    for (int j = 0; j < W; ++j) sa[j] *= inv_nt;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (FULL || r < nt) {
        float v[W];
        A::unpack(raw[r], v);
#pragma unroll
        for (int j = 0; j < W; ++j) { const float d = v[j] - sa[j]; sb[j] = fmaf(d, d, sb[j]); }
      }
    }
  } else {
#pragma unroll
    for (int j = 0; j < W; ++j) { sa[j] = 0.f; sb[j] = 0.f; }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) sa[j] = fmaf(v[j], v[j], sa[j]);
    }
  }
}

// Phase 3 of a strip: normalise the rows held in registers with the columns' scalars
// (cp, cq) and store them.  gp / bp point at gamma[wf] / beta[wf] (or are nullptr).
template <int OP, typename T, bool VEC, int R, bool FULL>
__device__ __forceinline__ void axis_reg_store(T* py, long long ystep, bool active, int nt, int nf,
                                               const T* gp, const T* bp,
                                               const typename AxisRaw<T, VEC>::Raw (&raw)[R],
                                               const float (&cp)[AxisRaw<T, VEC>::W],
                                               const float (&cq)[AxisRaw<T, VEC>::W]) {
  using A = AxisRaw<T, VEC>;
  using E = Elem<T>;
  constexpr int W = A::W;
  constexpr bool KEEP = (OP == OP_SOFTMAX) && (sizeof(T) == 4);
#pragma unroll
  for (int r = 0; r < R; ++r, py += ystep) {
    if (FULL || (active && r < nt)) {
      float g = 1.f, be = 0.f;
      if (!OpTraits<OP>::kSoftmaxLike) {
        if (gp != nullptr) g = E::load1(gp, r * nf);
        if (OP == OP_LAYERNORM && bp != nullptr) be = E::load1(bp, r * nf);
      }
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) {
        if (OP == OP_SOFTMAX) v[j] = (KEEP ? v[j] : exp_diff(v[j], cp[j])) * cq[j];
        else if (OP == OP_LOG_SOFTMAX) v[j] = (v[j] - cp[j]) - cq[j];
        else if (OP == OP_LAYERNORM) v[j] = (v[j] - cp[j]) * cq[j] * g + be;
        else v[j] = v[j] * cq[j] * g;
      }
      A::store(py, A::pack(v));
    }
  }
}

// nbase, nrem: reduce / nf and reduce % nf (warp-row i holds nbase + (i < nrem) rows).
template <int OP, typename T, bool VEC, int R>
__global__ void __launch_bounds__(32 * kAxisMaxWarps, 2)
axis_reg_kernel(const AxisParams p, const unsigned strips_per_outer, const int nf, const int nc,
                const int nbase, const int nrem) {
  pdl_prologue();
  using A = AxisRaw<T, VEC>;
  using Raw = typename A::Raw;
  constexpr int W = A::W;
  constexpr int CW = 32 * W;                 // columns of one column block
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  constexpr int KS = (OP == OP_RMSNORM) ? 1 : 2;
  // fp32 softmax keeps exp(x - m_local) in the registers the values came in; bf16 cannot
  // (a second rounding), it evaluates the exponential again for the output
  constexpr bool KEEP = (OP == OP_SOFTMAX) && (sizeof(T) == 4);
  extern __shared__ __align__(16) float axis_smem[];

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int wc = warp / nf;
  const int wf = warp - wc * nf;
  const int nw = nf * nc;
  float* part0 = axis_smem;                                 // [nw][CW]
  float* part1 = axis_smem + (KS - 1) * nw * CW;            // [nw][CW] (aliases part0 when KS == 1)
  float* fin0 = axis_smem + KS * nw * CW;                   // [nc][CW]
  float* fin1 = fin0 + nc * CW;
  const int nt = min(R, nbase + (wf < nrem ? 1 : 0));       // rows this thread holds
  const float inv_f = 1.0f / static_cast<float>(p.reduce);
  const long long xstep = p.xsf * nf, ystep = p.ysf * nf;
  const T* gp = (!SM && p.gamma != nullptr) ? reinterpret_cast<const T*>(p.gamma) + wf : nullptr;
  const T* bp = (OP == OP_LAYERNORM && p.beta != nullptr) ? reinterpret_cast<const T*>(p.beta) + wf : nullptr;

  for (long long b = blockIdx.y; b < p.outer; b += gridDim.y) {
    for (unsigned sc = blockIdx.x; sc < strips_per_outer; sc += gridDim.x) {
      const long long col0 = (static_cast<long long>(sc) * nc + wc) * CW + lane * W;
      const bool active = col0 < p.inner;
      const bool full = active && nt == R;
      const T* xb = reinterpret_cast<const T*>(p.x) + b * p.xso + wf * p.xsf + col0;
      T* yb = reinterpret_cast<T*>(p.y) + b * p.yso + wf * p.ysf + col0;

      Raw raw[R];
      float sa[W], sb[W];
      if (full) axis_reg_load<OP, T, VEC, R, true>(xb, xstep, active, nt, raw, sa, sb);
      else axis_reg_load<OP, T, VEC, R, false>(xb, xstep, active, nt, raw, sa, sb);

      // ---- the two scalars of every column
      float cp[W], cq[W];
      if (nf > 1) {
#pragma unroll
        for (int j = 0; j < W; ++j) {
          part0[warp * CW + lane * W + j] = sa[j];
          if (KS == 2) part1[warp * CW + lane * W + j] = sb[j];
        }
        __syncthreads();
        const float* q0 = part0 + wc * nf * CW;
        const float* q1 = part1 + wc * nf * CW;
        for (int c = wf * 32 + lane; c < CW; c += 32 * nf) {
          float a = 0.f, bb = 0.f;
          if (SM) {
            a = kNegInf;
            for (int i = 0; i < nf; ++i) a = fmaxf(a, q0[i * CW + c]);
            const float ms = (a == kNegInf) ? 0.f : a;
            for (int i = 0; i < nf; ++i) bb = fmaf(q1[i * CW + c], exp_diff(q0[i * CW + c], ms), bb);
          } else if (OP == OP_LAYERNORM) {
            for (int i = 0; i < nf; ++i) a = fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)), q0[i * CW + c], a);
            a *= inv_f;
            for (int i = 0; i < nf; ++i) {
              const float d = q0[i * CW + c] - a;
              bb += fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)) * d, d, q1[i * CW + c]);
            }
          } else {
            for (int i = 0; i < nf; ++i) a += q0[i * CW + c];
          }
          float sp, sq;
          axis_scalars<OP>(a, bb, inv_f, p.eps, sp, sq);
          fin0[wc * CW + c] = sp;
          fin1[wc * CW + c] = sq;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < W; ++j) { cp[j] = fin0[wc * CW + lane * W + j]; cq[j] = fin1[wc * CW + lane * W + j]; }
      } else {
#pragma unroll
        for (int j = 0; j < W; ++j) axis_scalars<OP>(sa[j], sb[j], inv_f, p.eps, cp[j], cq[j]);
      }
      if (KEEP) {
#pragma unroll
        for (int j = 0; j < W; ++j) cq[j] *= exp_diff(sa[j], cp[j]);     // exp(m_local - M) / S
      }

      if (full) axis_reg_store<OP, T, VEC, R, true>(yb, ystep, active, nt, nf, gp, bp, raw, cp, cq);
      else axis_reg_store<OP, T, VEC, R, false>(yb, ystep, active, nt, nf, gp, bp, raw, cp, cq);
    }
  }
}

}  // namespace akg
