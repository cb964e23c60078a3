// axis_kernel: the four operators over a NON-last axis of x[outer, reduce, inner] (inner
// contiguous) for a reduced axis too long to hold in registers - the general case of the
// layout of the paper's RMSNorm sketch (Unified Sketch figure, Section 3.2.1: X[B, F, D1, D2]
// reduced over F, inner = D1 * D2).
//
// Threads own columns, not rows.  A CTA of 8 warps takes a strip of LC lanes x W contiguous
// columns (W = one 16-byte vector, or one element on the unaligned path) of one outer index;
// a warp spans LC lanes of columns and 32 / LC consecutive rows, so the CTA walks the reduced
// axis 256 / LC rows at a time.  LC is a launch argument: long reduced axes take narrow
// strips, so that the strips in flight stay in L2 between the passes.  Pass 1 keeps running
// statistics per column in registers, block-wise over UB rows loaded back to back (online
// max / rescaled sum, Chan's merge of block mean / M2, sum of squares); the 256 / LC row
// slots of a column are merged through shared memory, each column by one thread, which also
// derives the column's two scalars; pass 2 re-reads the strip from L2, normalises and
// stores.  HBM sees one read and one write per element.
#pragma once

#include "kernels_axis_reg.cuh"
#include "kernels_split.cuh"

namespace akg {

constexpr int kAxisThreads = 256;

// Online statistics of one thread's columns.  softmax keeps the maximum m and, in the base-2
// domain, c = round(m log2e) and s = sum exp2(x log2e - c) (see axis_reg_load); log-softmax
// keeps m and s = sum exp(x - m); LayerNorm keeps mean and M2 of the n rows folded so far
// (n is the same for every column of a thread); RMSNorm keeps the sum of squares.
template <int OP, int W> struct AxisRun {
  float a[W], b[W], c[W];
  float n;
  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < W; ++j) { a[j] = OpTraits<OP>::kSoftmaxLike ? kNegInf : 0.f; b[j] = 0.f; c[j] = kNegInf; }
    n = 0.f;
  }
  // fold `cnt` rows (v[u][j], u < cnt; all UB when FULL)
  template <int UB, bool FULL> __device__ __forceinline__ void fold(const float (&v)[UB][W], int cnt) {
    if (OpTraits<OP>::kSoftmaxLike) {
#pragma unroll
      for (int j = 0; j < W; ++j) {
        float bm = kNegInf;
#pragma unroll
        for (int u = 0; u < UB; ++u) if (FULL || u < cnt) bm = fmaxf(bm, v[u][j]);
        const float mn = fmaxf(a[j], bm);
        const float ms = (mn == kNegInf) ? 0.f : mn;
        if (OP == OP_SOFTMAX) {
          const float cn = ms * kLog2e;
          float acc = b[j] * ex2_approx(c[j] - cn);          // c = -inf while nothing is live: factor 0
#pragma unroll
          for (int u = 0; u < UB; ++u) if (FULL || u < cnt) acc += ex2_approx(fmaf(v[u][j], kLog2e, -cn));
          b[j] = acc; c[j] = (mn == kNegInf) ? kNegInf : cn;
        } else {
          float acc = b[j] * exp_diff(a[j], ms);
#pragma unroll
          for (int u = 0; u < UB; ++u) if (FULL || u < cnt) acc += exp_diff(v[u][j], ms);
          b[j] = acc;
        }
        a[j] = mn;
      }
    } else if (OP == OP_LAYERNORM) {
      const float k = FULL ? static_cast<float>(UB) : static_cast<float>(cnt);
      const float inv_k = FULL ? (1.0f / UB) : __frcp_rn(k);
      const float nn = n + k;
      const float wk = k * __frcp_rn(nn);                     // share of the new block
#pragma unroll
      for (int j = 0; j < W; ++j) {
        float sum = 0.f;
#pragma unroll
        for (int u = 0; u < UB; ++u) if (FULL || u < cnt) sum += v[u][j];
        const float bmean = sum * inv_k;
        float m2 = 0.f;
#pragma unroll
        for (int u = 0; u < UB; ++u) if (FULL || u < cnt) { const float d = v[u][j] - bmean; m2 = fmaf(d, d, m2); }
        const float d = bmean - a[j];
        a[j] = fmaf(d, wk, a[j]);
        b[j] += fmaf(d * d, n * wk, m2);
      }
      n = nn;
    } else {
#pragma unroll
      for (int j = 0; j < W; ++j)
#pragma unroll
        for (int u = 0; u < UB; ++u) if (FULL || u < cnt) a[j] = fmaf(v[u][j], v[u][j], a[j]);
    }
  }
};

// Merge the ns row slots of one column (q0[i * cw], q1[i * cw]) into the column's two scalars.
// Slot i holds nbase + (i < nrem) rows.
template <int OP>
__device__ __forceinline__ void axis_merge_slots(const float* q0, const float* q1, int ns, int cw, int nbase, int nrem,
                                                 float inv_f, float eps, float& sp, float& sq) {
  float a = 0.f, bb = 0.f;
  if (OpTraits<OP>::kSoftmaxLike) {
    a = kNegInf;
#pragma unroll 4
    for (int i = 0; i < ns; ++i) a = fmaxf(a, q0[i * cw]);
    const float ms = (a == kNegInf) ? 0.f : a;
#pragma unroll 4
    for (int i = 0; i < ns; ++i)
      bb = fmaf(q1[i * cw], OP == OP_SOFTMAX ? ex2_approx(q0[i * cw] - ms) : exp_diff(q0[i * cw], ms), bb);
  } else if (OP == OP_LAYERNORM) {
    // (the first slot's mean plus the weighted mean of the differences from it: see axis_merge_column)
    const float ref = q0[0];
    for (int i = 0; i < ns; ++i) a = fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)), q0[i * cw] - ref, a);
    a = fmaf(a, inv_f, ref);
    for (int i = 0; i < ns; ++i) {
      const float d = q0[i * cw] - a;
      bb += fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)) * d, d, q1[i * cw]);
    }
  } else {
#pragma unroll 4
    for (int i = 0; i < ns; ++i) a += q0[i * cw];
  }
  axis_scalars<OP>(a, bb, inv_f, eps, sp, sq);
}

// lc_shift: log2 of the lanes of a warp that lie along the columns (the other 32 >> lc_shift
// lie along rows).  nbase, nrem: reduce / slots and reduce % slots, slots = 256 >> lc_shift.
template <int OP, typename T, int MODE>
#ifndef AKG_AXIS_MINB
#define AKG_AXIS_MINB 4
#endif
__global__ void __launch_bounds__(kAxisThreads, AKG_AXIS_MINB)
axis_kernel(const AxisParams p, const unsigned strips_per_outer, const int lc_shift, const int nbase, const int nrem) {
  pdl_prologue();
  using A = AxisRaw<T, MODE>;
  using E = Elem<T>;
  using Raw = typename A::Raw;
  constexpr int W = A::W;
#ifndef AKG_AXIS_UB
#define AKG_AXIS_UB 4
#endif
  constexpr int UB = (W >= 4) ? AKG_AXIS_UB : 8;   // rows per block = loads in flight per thread
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  __shared__ __align__(16) float part[2][kAxisThreads * W];
  __shared__ __align__(16) float fin[2][32 * W];

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int lc = 1 << lc_shift;
  const int lcol = lane & (lc - 1);
  const int slot = warp * (32 >> lc_shift) + (lane >> lc_shift);     // row slot of this thread
  const int ns = kAxisThreads >> lc_shift;                             // row slots of the CTA
  const int cw = lc * W;                                               // columns of a strip
  const int F = static_cast<int>(p.reduce);
  const float inv_f = 1.0f / static_cast<float>(F);
  const long long xstep = p.xsf * ns, ystep = p.ysf * ns;
  const uint64_t keep = l2_policy_keep();
  const uint64_t drop = l2_policy_drop();
  const T* gp = (!SM && p.gamma != nullptr) ? reinterpret_cast<const T*>(p.gamma) : nullptr;
  const T* bp = (OP == OP_LAYERNORM && p.beta != nullptr) ? reinterpret_cast<const T*>(p.beta) : nullptr;

  for (long long b = blockIdx.y; b < p.outer; b += gridDim.y) {
    for (unsigned sc = blockIdx.x; sc < strips_per_outer; sc += gridDim.x) {
      const long long col0 = static_cast<long long>(sc) * cw + lcol * W;
      const bool active = col0 < p.inner;
      const T* xb = reinterpret_cast<const T*>(p.x) + b * p.xso + slot * p.xsf + col0;
      T* yb = reinterpret_cast<T*>(p.y) + b * p.yso + slot * p.ysf + col0;

      // ---- pass 1: running statistics of this thread's columns over its rows
      AxisRun<OP, W> run;
      run.init();
      if (active) {
        const T* px = xb;
        int f = slot;
        for (; f + (UB - 1) * ns < F; f += UB * ns) {
          Raw raw[UB];
#pragma unroll
          for (int u = 0; u < UB; ++u, px += xstep) raw[u] = A::load_hint(px, keep);
          float v[UB][W];
#pragma unroll
          for (int u = 0; u < UB; ++u) A::unpack(raw[u], v[u]);
          run.template fold<UB, true>(v, UB);
        }
        if (f < F) {
          const int cnt = (F - f + ns - 1) / ns;              // 1 .. UB - 1 rows left
          float v[UB][W];
#pragma unroll
          for (int u = 0; u < UB; ++u, px += xstep) {
            if (u < cnt) A::unpack(A::load_hint(px, keep), v[u]);
            else A::unpack(A::fill(0.f), v[u]);
          }
          run.template fold<UB, false>(v, cnt);
        }
      }
#pragma unroll
      for (int j = 0; j < W; ++j) {
        part[0][slot * cw + lcol * W + j] = (OP == OP_SOFTMAX) ? run.c[j] : run.a[j];
        part[1][slot * cw + lcol * W + j] = run.b[j];
      }
      __syncthreads();

      // ---- one thread per column merges the row slots and derives the column's scalars
      if (static_cast<int>(threadIdx.x) < cw) {
        float sp, sq;
        axis_merge_slots<OP>(&part[0][threadIdx.x], &part[1][threadIdx.x], ns, cw, nbase, nrem, inv_f, p.eps, sp, sq);
        fin[0][threadIdx.x] = sp;
        fin[1][threadIdx.x] = sq;
      }
      __syncthreads();
      float cp[W], cq[W];
#pragma unroll
      for (int j = 0; j < W; ++j) { cp[j] = fin[0][lcol * W + j]; cq[j] = fin[1][lcol * W + j]; }

      // ---- pass 2: second read (L2), normalise, store
      if (active) {
        const T* px = xb;
        T* py = yb;
        for (int f = slot; f < F; f += UB * ns) {
          const bool whole = f + (UB - 1) * ns < F;
          Raw raw[UB];
#pragma unroll
          for (int u = 0; u < UB; ++u, px += xstep)
            if (whole || f + u * ns < F) raw[u] = A::load_hint(px, drop);
#pragma unroll
          for (int u = 0; u < UB; ++u, py += ystep) {
            const int fu = f + u * ns;
            if (whole || fu < F) {
              float g = 1.f, be = 0.f;
              if (!SM) {
                if (gp != nullptr) g = E::load1(gp, fu);
                if (OP == OP_LAYERNORM && bp != nullptr) be = E::load1(bp, fu);
              }
              float v[W];
              A::unpack(raw[u], v);
#pragma unroll
              for (int j = 0; j < W; ++j) {
                if (OP == OP_SOFTMAX) v[j] = ex2_approx(fmaf(v[j], kLog2e, -cp[j])) * cq[j];
                else if (OP == OP_LOG_SOFTMAX) v[j] = (v[j] - cp[j]) - cq[j];
                else if (OP == OP_LAYERNORM) v[j] = (v[j] - cp[j]) * cq[j] * g + be;
                else v[j] = v[j] * cq[j] * g;
              }
              A::store(py, A::pack(v));
            }
          }
        }
      }
      // `part` and `fin` are rewritten by the next strip only after the barriers above
    }
  }
}

}  // namespace akg
