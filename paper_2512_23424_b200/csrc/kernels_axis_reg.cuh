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
#include "kernels_split.cuh"

namespace akg {

// How a thread holds one row of its columns (MODE):
//   0  one element, widened to float (any alignment)
//   1  one 16-byte vector as loaded (4 floats / 8 packed bf16); bf16 is unpacked at each use
//   2  bf16 only: one 8-byte vector widened to 4 floats at the load - the register picture of
//      fp32 mode 1, so a bf16 value is unpacked once and softmax evaluates one exponential
//      per element; rows are 256-byte segments per warp
template <typename T, int MODE> struct AxisRaw;

template <> struct AxisRaw<__nv_bfloat16, 2> {
  using T = __nv_bfloat16;
  using Raw = float4;
  static constexpr int W = 4;
  static constexpr bool kFloatRaw = true;
  static __device__ __forceinline__ Raw load(const T* p) {
    uint32_t a, b;
    asm volatile("ld.global.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(a), "=r"(b) : "l"(p) : "memory");
    return make_float4(__uint_as_float(a << 16), __uint_as_float(a & 0xffff0000u),
                       __uint_as_float(b << 16), __uint_as_float(b & 0xffff0000u));
  }
  static __device__ __forceinline__ Raw fill(float v) { return make_float4(v, v, v, v); }
  static __device__ __forceinline__ void unpack(const Raw& r, float (&f)[4]) { f[0] = r.x; f[1] = r.y; f[2] = r.z; f[3] = r.w; }
  static __device__ __forceinline__ Raw pack(const float (&f)[4]) { return make_float4(f[0], f[1], f[2], f[3]); }
  static __device__ __forceinline__ void store(T* p, const Raw& r) {
    const uint32_t a = Elem<T>::pack2(r.x, r.y), b = Elem<T>::pack2(r.z, r.w);
    asm volatile("st.global.cs.v2.u32 [%0], {%1, %2};" :: "l"(p), "r"(a), "r"(b) : "memory");
  }
};

template <typename T> struct AxisRaw<T, 1> {
  using E = Elem<T>;
  using Raw = uint4;
  static constexpr int W = E::EPV;
  static constexpr bool kFloatRaw = (sizeof(T) == 4);
  static __device__ __forceinline__ Raw load(const T* p) { return ld_stream(p); }
  static __device__ __forceinline__ Raw load_hint(const T* p, uint64_t policy) { return ld_hint(p, policy); }
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

template <typename T> struct AxisRaw<T, 0> {
  using E = Elem<T>;
  using Raw = float;                        // a bf16 value widens exactly
  static constexpr int W = 1;
  static constexpr bool kFloatRaw = true;
  static __device__ __forceinline__ Raw load(const T* p) { return E::load1(p, 0); }
  static __device__ __forceinline__ Raw load_hint(const T* p, uint64_t) { return E::load1(p, 0); }
  static __device__ __forceinline__ Raw fill(float v) { return v; }
  static __device__ __forceinline__ void unpack(const Raw& r, float (&f)[1]) { f[0] = r; }
  static __device__ __forceinline__ Raw pack(const float (&f)[1]) { return f[0]; }
  static __device__ __forceinline__ void store(T* p, const Raw& r) { E::store1(p, 0, r); }
};

constexpr int kAxisMaxWarps = 16;

// Shared memory of one CTA in floats: partials [KS][nf * nc][32 W], then scalars [2][nc][32 W].
constexpr int kAxisAffineFloats = 2 * kAxisMaxWarps * 8;     // gamma and beta of up to 16 warp-rows x 8 rows
__host__ __device__ constexpr unsigned axis_reg_smem_floats(int ks, int nf, int nc, int w) {
  return nf > 1 ? static_cast<unsigned>((ks * nf * nc + 2 * nc) * 32 * w + kAxisAffineFloats) : 0u;
}

// The two scalars of a column from its merged statistics:
//   softmax     : p = C = round(M log2e) (0 for a column without live entry), q = 1 / S (0 for
//                 such a column)
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

// Merge the nf partials of one column (q0[i * CW], q1[i * CW]: partial i) and derive the
// column's two scalars.  Warp-row i holds nbase + (i < nrem) rows of the reduced axis.
template <int OP, int CW>
__device__ __forceinline__ void axis_merge_column(const float* q0, const float* q1, int nf, int nbase, int nrem,
                                                  float inv_f, float eps, float& sp, float& sq) {
  float a = 0.f, bb = 0.f;
  if (OpTraits<OP>::kSoftmaxLike) {
    a = kNegInf;
#pragma unroll 4
    for (int i = 0; i < nf; ++i) a = fmaxf(a, q0[i * CW]);
    const float ms = (a == kNegInf) ? 0.f : a;
#pragma unroll 4
    for (int i = 0; i < nf; ++i)
      bb = fmaf(q1[i * CW], OP == OP_SOFTMAX ? ex2_approx(q0[i * CW] - ms) : exp_diff(q0[i * CW], ms), bb);
  } else if (OP == OP_LAYERNORM) {
    // The mean as the first partial mean plus the weighted mean of the differences from it: summing the partial
    // means themselves rounds at the magnitude of count x |mean| and the rounded 1 / F biases the quotient, which
    // together put 1e-6 |mean| into the mean of a thousand rows (results off by 2e-5 where mean / std = 30).
    const float ref = q0[0];
    if (nrem == 0) {                       // equal counts: mean of means, M2 = sum M2_i + n sum d_i^2
#pragma unroll 4
      for (int i = 0; i < nf; ++i) a += q0[i * CW] - ref;
      const float nb = static_cast<float>(nbase);
      a = fmaf(a, nb * inv_f, ref);
      float dd = 0.f;
#pragma unroll 4
      for (int i = 0; i < nf; ++i) {
        const float d = q0[i * CW] - a;
        bb += q1[i * CW];
        dd = fmaf(d, d, dd);
      }
      bb = fmaf(nb, dd, bb);
    } else {
      for (int i = 0; i < nf; ++i) a = fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)), q0[i * CW] - ref, a);
      a = fmaf(a, inv_f, ref);
      for (int i = 0; i < nf; ++i) {
        const float d = q0[i * CW] - a;
        bb += fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)) * d, d, q1[i * CW]);
      }
    }
  } else {
#pragma unroll 4
    for (int i = 0; i < nf; ++i) a += q0[i * CW];
  }
  axis_scalars<OP>(a, bb, inv_f, eps, sp, sq);
}

// Phase 1 of a strip: load this thread's rows and fold them into per-column partials
// ((m, s), (mean, M2) or the sum of squares).  FULL: all R rows exist and the columns are
// inside the array, so nothing is predicated (the case of every thread but those of a
// ragged last warp-row or column block).
template <int OP, typename T, int MODE, int R, bool FULL>
__device__ __forceinline__ void axis_reg_load(const T* px, long long xstep, bool active, int nt,
                                              typename AxisRaw<T, MODE>::Raw (&raw)[R],
                                              float (&sa)[AxisRaw<T, MODE>::W], float (&sb)[AxisRaw<T, MODE>::W]) {
  using A = AxisRaw<T, MODE>;
  constexpr int W = A::W;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  constexpr bool KEEP = (OP == OP_SOFTMAX) && A::kFloatRaw;
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
    // softmax works in the base-2 domain: its partial maximum is c = round(m log2e), and every
    // exponential is exp2(x log2e - c) in one multiply-add.  Partials are later rescaled by
    // exp2(c - C) with the same rounded numbers, so the rounding of m log2e cancels exactly
    // between numerator and denominator.  log-softmax keeps (x - m) exact instead.
    float ms[W];
#pragma unroll
    for (int j = 0; j < W; ++j) {
      if (OP == OP_SOFTMAX) sa[j] *= kLog2e;
      ms[j] = (sa[j] == kNegInf) ? 0.f : sa[j];
      if (OP == OP_SOFTMAX) ms[j] = -ms[j];
      sb[j] = 0.f;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) {
        v[j] = (OP == OP_SOFTMAX) ? ex2_approx(fmaf(v[j], kLog2e, ms[j])) : exp_diff(v[j], ms[j]);
        sb[j] += v[j];
      }
      if (KEEP) raw[r] = A::pack(v);
    }
  } else if (OP == OP_LAYERNORM && sizeof(T) == 2) {
    // 16-bit storage: one sweep of sums shifted by the thread's first row, k = x[0]:
    //   mean = k + S1 / n,  M2 = S2 - S1^2 / n  with S1 = sum (x - k), S2 = sum (x - k)^2.
    // k lies among the data, so S2 exceeds M2 by n (mean - k)^2 only and the subtraction costs a
    // few of fp32's bits, far inside the 2^-9 of the stored result; it saves an unpack and an
    // operation per element against the exact two sweeps that fp32 storage keeps.
    float k[W];
    A::unpack(raw[0], k);
#pragma unroll
    for (int j = 0; j < W; ++j) { sa[j] = 0.f; sb[j] = 0.f; }
#pragma unroll
    for (int r = 1; r < R; ++r) {
      if (FULL || r < nt) {
        if constexpr (MODE == 1 && sizeof(T) == 2) {
          // packed row: the stored values enter the subtraction as they are (Elem::sub_wide), no unpack
          const uint32_t ws[4] = {raw[r].x, raw[r].y, raw[r].z, raw[r].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            unsigned short h0, h1;
            halves(ws[i], h0, h1);
            const float d0 = Elem<T>::sub_wide(h0, k[2 * i]), d1 = Elem<T>::sub_wide(h1, k[2 * i + 1]);
            sa[2 * i] += d0; sb[2 * i] = fmaf(d0, d0, sb[2 * i]);
            sa[2 * i + 1] += d1; sb[2 * i + 1] = fmaf(d1, d1, sb[2 * i + 1]);
          }
        } else {
          float v[W];
          A::unpack(raw[r], v);
#pragma unroll
          for (int j = 0; j < W; ++j) { const float d = v[j] - k[j]; sa[j] += d; sb[j] = fmaf(d, d, sb[j]); }
        }
      }
    }
    const float inv_nt = FULL ? (1.0f / R) : ((nt > 0) ? __frcp_rn(static_cast<float>(nt)) : 0.f);
#pragma unroll
    for (int j = 0; j < W; ++j) {
      const float m = sa[j] * inv_nt;                         // mean - k
      sb[j] = fmaxf(fmaf(-sa[j], m, sb[j]), 0.f);
      sa[j] = (FULL || nt > 0) ? k[j] + m : 0.f;
    }
  } else if (OP == OP_LAYERNORM) {
    // fp32 storage: the exact two sweeps, the mean as the thread's first row plus the mean of the differences
    // from it.  (The plain sum of R values rounds at R |mean| and the rounded 1 / nt biases the quotient: with
    // 3 to 16 rows per column and mean / std = 30 the results were off by three to five times what the
    // rounding of the mean itself costs.)
    float k[W];
    A::unpack(raw[0], k);
#pragma unroll
    for (int j = 0; j < W; ++j) { sa[j] = 0.f; sb[j] = 0.f; }
#pragma unroll
    for (int r = 1; r < R; ++r) {
      if (FULL || r < nt) {
        float v[W];
        A::unpack(raw[r], v);
#pragma unroll
        for (int j = 0; j < W; ++j) sa[j] += v[j] - k[j];
      }
    }
    const float inv_nt = FULL ? (1.0f / R) : ((nt > 0) ? __frcp_rn(static_cast<float>(nt)) : 0.f);
#pragma unroll
    for (int j = 0; j < W; ++j) sa[j] = (FULL || nt > 0) ? fmaf(sa[j], inv_nt, k[j]) : 0.f;
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
template <int OP, typename T, int MODE, int R, bool FULL>
__device__ __forceinline__ void axis_reg_store(T* py, long long ystep, bool active, int nt, int nf,
                                               const T* gp, const T* bp, const float* gs, const float* bs,
                                               const typename AxisRaw<T, MODE>::Raw (&raw)[R],
                                               const float (&cp)[AxisRaw<T, MODE>::W],
                                               const float (&cq)[AxisRaw<T, MODE>::W]) {
  using A = AxisRaw<T, MODE>;
  using E = Elem<T>;
  constexpr int W = A::W;
  constexpr bool KEEP = (OP == OP_SOFTMAX) && A::kFloatRaw;
  // softmax from packed values: exp2(x log2e - C) / S with ncp = -C; 16-bit LayerNorm: (x - mean) rstd as
  // one fused multiply-add with ncp = -mean rstd (rounding 2^-24 |mean| rstd, far inside the stored 2^-9)
  constexpr bool kFusedCentre = (OP == OP_LAYERNORM) && (sizeof(T) == 2);
  float ncp[W];
#pragma unroll
  for (int j = 0; j < W; ++j) ncp[j] = kFusedCentre ? -cp[j] * cq[j] : -cp[j];
#pragma unroll
  for (int r = 0; r < R; ++r, py += ystep) {
    if (FULL || (active && r < nt)) {
      float g = 1.f, be = 0.f;
      if (!OpTraits<OP>::kSoftmaxLike) {
        if (gs != nullptr) {                               // staged once per CTA: one shared load, constant offset
          g = gs[r];
          if (OP == OP_LAYERNORM) be = bs[r];
        } else {
          if (gp != nullptr) g = E::load1(gp, r * nf);
          if (OP == OP_LAYERNORM && bp != nullptr) be = E::load1(bp, r * nf);
        }
      }
      float v[W];
      A::unpack(raw[r], v);
#pragma unroll
      for (int j = 0; j < W; ++j) {
        if (OP == OP_SOFTMAX) v[j] = (KEEP ? v[j] : ex2_approx(fmaf(v[j], kLog2e, ncp[j]))) * cq[j];
        else if (OP == OP_LOG_SOFTMAX) v[j] = (v[j] - cp[j]) - cq[j];
        else if (OP == OP_LAYERNORM) v[j] = kFusedCentre ? fmaf(fmaf(v[j], cq[j], ncp[j]), g, be)
                                                         : (v[j] - cp[j]) * cq[j] * g + be;
        else v[j] = v[j] * cq[j] * g;
      }
      A::store(py, A::pack(v));
    }
  }
}

// nbase, nrem: reduce / nf and reduce % nf (warp-row i holds nbase + (i < nrem) rows).
template <int OP, typename T, int MODE, int R>
__global__ void __launch_bounds__(32 * kAxisMaxWarps, 2)
axis_reg_kernel(const AxisParams p, const unsigned strips_per_outer, const int nf, const int nc,
                const int nbase, const int nrem) {
  pdl_prologue();
  using A = AxisRaw<T, MODE>;
  using Raw = typename A::Raw;
  constexpr int W = A::W;
  constexpr int CW = 32 * W;                 // columns of one column block
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  constexpr int KS = (OP == OP_RMSNORM) ? 1 : 2;
  // fp32 softmax keeps exp(x - m_local) in the registers the values came in; bf16 cannot
  // (a second rounding), it evaluates the exponential again for the output
  constexpr bool KEEP = (OP == OP_SOFTMAX) && A::kFloatRaw;
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
  // The affine scalars of the reduced axis are the same for every strip: with several warp-rows they are staged
  // once per CTA in shared memory as floats, [warp-row][row], so that the store phase reads them with one shared
  // load at a constant offset (a 16-bit global load with a 64-bit index each cost five instructions per row and
  // scalar: one instruction per element of the 16-bit LayerNorm).  The strip loop's first barrier orders them.
  float* aff = fin1 + nc * CW;                              // [2][nf * R]
  const float* gs = nullptr;
  const float* bs = nullptr;
  if (!SM && nf > 1 && nf * R <= kAxisAffineFloats / 2) {
    for (int i = threadIdx.x; i < nf * R; i += blockDim.x) {
      const int w = i / R, r = i - w * R;
      const long long f = w + static_cast<long long>(r) * nf;
      aff[i] = (p.gamma != nullptr && f < p.reduce) ? Elem<T>::load1(p.gamma, f) : 1.f;
      if (OP == OP_LAYERNORM) aff[nf * R + i] = (p.beta != nullptr && f < p.reduce) ? Elem<T>::load1(p.beta, f) : 0.f;
    }
    gs = aff + wf * R;
    bs = aff + nf * R + wf * R;
  }

  for (long long b = blockIdx.y; b < p.outer; b += gridDim.y) {
    for (unsigned sc = blockIdx.x; sc < strips_per_outer; sc += gridDim.x) {
      const long long col0 = (static_cast<long long>(sc) * nc + wc) * CW + lane * W;
      const bool active = col0 < p.inner;
      const bool full = active && nt == R;
      const T* xb = reinterpret_cast<const T*>(p.x) + b * p.xso + wf * p.xsf + col0;
      T* yb = reinterpret_cast<T*>(p.y) + b * p.yso + wf * p.ysf + col0;

      Raw raw[R];
      float sa[W], sb[W];
      if (full) axis_reg_load<OP, T, MODE, R, true>(xb, xstep, active, nt, raw, sa, sb);
      else axis_reg_load<OP, T, MODE, R, false>(xb, xstep, active, nt, raw, sa, sb);

      // ---- the two scalars of every column
      float cp[W], cq[W];
      if (nf > 1) {
#pragma unroll
        for (int j = 0; j < W; ++j) {
          part0[warp * CW + lane * W + j] = sa[j];
          if (KS == 2) part1[warp * CW + lane * W + j] = sb[j];
        }
        __syncthreads();
        for (int c = wf * 32 + lane; c < CW; c += 32 * nf) {
          float sp, sq;
          axis_merge_column<OP, CW>(part0 + wc * nf * CW + c, part1 + wc * nf * CW + c, nf, nbase, nrem, inv_f, p.eps,
                                    sp, sq);
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
        for (int j = 0; j < W; ++j) cq[j] *= ex2_approx(sa[j] - cp[j]);  // exp2(c_local - C) / S
      }

      if (full) axis_reg_store<OP, T, MODE, R, true>(yb, ystep, active, nt, nf, gp, bp, gs, bs, raw, cp, cq);
      else axis_reg_store<OP, T, MODE, R, false>(yb, ystep, active, nt, nf, gp, bp, gs, bs, raw, cp, cq);
    }
  }
}

}  // namespace akg
