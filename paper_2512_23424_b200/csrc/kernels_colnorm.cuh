// BatchNorm-style column normalisation (BatchNorm is among the operators of Section 3.6): every
// column of x[rows, cols] is normalised with its own mean and biased variance over the rows and
// a per-column affine.  The reduction runs across rows, so a column's statistics come from every
// part of the matrix: two kernels on one stream, with a small workspace between them.
//   col_stat_kernel    grid (column strips, row blocks): per-column (mean, M2) of the block's rows,
//                      written to workspace[block][column]; its loads mark their lines "keep in L2"
//   col_finish_kernel  a warp per column merges the blocks' pairs (counts known from the geometry) and
//                      leaves (mean, 1 / std) in workspace[0][column]: once per column, not once per CTA
//                      of the third kernel (147 row blocks x 4 strips each merged all 147 pairs of their
//                      256 columns before: 40 M warp instructions against 16 M of the statistics kernel)
//   col_apply_kernel   the first kernel's grid, walked in REVERSE block order: the blocks the statistics
//                      kernel read last are the ones still in L2, so a matrix somewhat larger than L2 is
//                      still re-read from there for the most part; normalises its block of rows
// x is read twice; the second read is served by L2 as far as the matrix fits there.  Threads own
// columns (a warp lies 1 << lc_shift lanes along the columns and the rest along rows), as in the
// non-last-axis kernels, whose loaders and running statistics are reused.
#pragma once

#include "kernels_axis.cuh"

namespace akg {

constexpr int kColUB = 4;

template <typename T, int MODE>
__global__ void __launch_bounds__(kAxisThreads, 4) col_stat_kernel(const ColParams p) {
  pdl_prologue();
  using A = AxisRaw<T, MODE>;
  using Raw = typename A::Raw;
  constexpr int W = A::W;
  constexpr int UB = kColUB;
  __shared__ __align__(16) float part[2][kAxisThreads * W];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int lc = 1 << p.lc_shift;
  const int lcol = lane & (lc - 1);
  const int slot = warp * (32 >> p.lc_shift) + (lane >> p.lc_shift);
  const int ns = kAxisThreads >> p.lc_shift;
  const int cw = lc * W;
  const long long col0 = static_cast<long long>(blockIdx.x) * cw + lcol * W;
  const bool active = col0 < p.cols;
  const long long r0 = static_cast<long long>(blockIdx.y) * p.rows_per_block;
  const long long r1 = min(p.rows, r0 + p.rows_per_block);
  const long long xstep = p.xs * ns;

  AxisRun<OP_LAYERNORM, W> run;
  run.init();
  // (a matrix far beyond L2 gains nothing from the marks and measured 8 % slower with them: plain priority then)
  const uint64_t keep = p.l2_keep ? l2_policy_keep() : l2_policy_normal();
  if constexpr (sizeof(T) == 2 && MODE == 1) {
    // 16-bit storage: one sweep of sums about the thread's first row of the block, K = x[first]: S1 = sum (x - K),
    // S2 = sum (x - K)^2, mean = K + S1 / n, M2 = S2 - S1^2 / n.  K lies among the data, so the subtraction at the
    // end costs a relative (n + 1) 2^-24 at most (n is a few dozen rows), far inside the 2^-9 of a 16-bit result;
    // the stored values enter the subtraction as they are (Elem::sub_wide).  Three instructions per element instead
    // of the block-wise means, deviations and merges of the fp32 form.
    if (active && r0 + slot < r1) {
      using E = Elem<T>;
      const T* px = reinterpret_cast<const T*>(p.x) + (r0 + slot) * p.xs + col0;
      float k[W], s1[W], s2[W];
      A::unpack(A::load(px), k);
#pragma unroll
      for (int j = 0; j < W; ++j) { s1[j] = 0.f; s2[j] = 0.f; }
      auto add_row = [&](const Raw& raw) {
        const uint32_t ws[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(ws[i], h0, h1);
          const float d0 = E::sub_wide(h0, k[2 * i]), d1 = E::sub_wide(h1, k[2 * i + 1]);
          s1[2 * i] += d0; s2[2 * i] = fmaf(d0, d0, s2[2 * i]);
          s1[2 * i + 1] += d1; s2[2 * i + 1] = fmaf(d1, d1, s2[2 * i + 1]);
        }
      };
      long long f = r0 + slot;
      for (; f + (UB - 1) * ns < r1; f += UB * ns) {
        Raw raw[UB];
#pragma unroll
        for (int u = 0; u < UB; ++u, px += xstep) raw[u] = A::load_hint(px, keep);
#pragma unroll
        for (int u = 0; u < UB; ++u) add_row(raw[u]);
      }
      for (; f < r1; f += ns, px += xstep) add_row(A::load_hint(px, keep));
      const float n = static_cast<float>((r1 - (r0 + slot) + ns - 1) / ns);
      const float inv_n = __frcp_rn(n);
#pragma unroll
      for (int j = 0; j < W; ++j) {
        const float m = s1[j] * inv_n;                        // mean - K
        run.a[j] = k[j] + m;
        run.b[j] = fmaxf(fmaf(-s1[j], m, s2[j]), 0.f);
      }
    }
  } else if (active) {
    const T* px = reinterpret_cast<const T*>(p.x) + (r0 + slot) * p.xs + col0;
    long long f = r0 + slot;
    for (; f + (UB - 1) * ns < r1; f += UB * ns) {
      Raw raw[UB];
#pragma unroll
      for (int u = 0; u < UB; ++u, px += xstep) raw[u] = A::load_hint(px, keep);
      float v[UB][W];
#pragma unroll
      for (int u = 0; u < UB; ++u) A::unpack(raw[u], v[u]);
      run.template fold<UB, true>(v, UB);
    }
    if (f < r1) {
      const int cnt = static_cast<int>((r1 - f + ns - 1) / ns);
      float v[UB][W];
#pragma unroll
      for (int u = 0; u < UB; ++u, px += xstep) {
        if (u < cnt) A::unpack(A::load(px), v[u]);
        else A::unpack(A::fill(0.f), v[u]);
      }
      run.template fold<UB, false>(v, cnt);
    }
  }
#pragma unroll
  for (int j = 0; j < W; ++j) {
    part[0][slot * cw + lcol * W + j] = run.a[j];
    part[1][slot * cw + lcol * W + j] = run.b[j];
  }
  __syncthreads();
  // one thread per column merges the row slots (slot i holds nbase + (i < nrem) rows of the block)
  const long long c = static_cast<long long>(blockIdx.x) * cw + threadIdx.x;
  if (static_cast<int>(threadIdx.x) < cw && c < p.cols) {
    const long long n = r1 - r0;
    const int nbase = static_cast<int>(n / ns), nrem = static_cast<int>(n % ns);
    // the first slot's mean plus the weighted mean of the differences from it: the sum of count x mean itself
    // would round at n |mean| and the rounded 1 / n would bias every block's quotient the same way
    const float ref = part[0][threadIdx.x];
    float mean = 0.f;
    for (int i = 0; i < ns; ++i)
      mean = fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)), part[0][i * cw + threadIdx.x] - ref, mean);
    mean = fmaf(mean, 1.0f / static_cast<float>(n), ref);
    float m2 = 0.f;
    for (int i = 0; i < ns; ++i) {
      const float d = part[0][i * cw + threadIdx.x] - mean;
      m2 += fmaf(static_cast<float>(nbase + (i < nrem ? 1 : 0)) * d, d, part[1][i * cw + threadIdx.x]);
    }
    p.partial[static_cast<long long>(blockIdx.y) * p.cols + c] = make_float2(mean, m2);
  }
}

// A warp per column: lane l takes row blocks l, l + 32, ...  One sweep over the blocks' pairs, with sums taken
// about the first block's mean (ref): S1 = sum n_b (m_b - ref), S2 = sum (M2_b + n_b (m_b - ref)^2), then
// mean = ref + S1 / N and M2 = S2 - N (mean - ref)^2.  The block means differ from the column mean by about
// sigma / sqrt(rows per block), so the term subtracted at the end is a small fraction of M2 and the subtraction
// costs no accuracy that matters; two sweeps (the mean first) read the pairs twice, one dependent trip to L2 more
// in a kernel that is nothing but latency.
__global__ void __launch_bounds__(256) col_finish_kernel(const ColParams p, const int nblk) {
  pdl_prologue();                              // the statistics kernel has completed when this returns
  const int lane = threadIdx.x & 31;
  const long long c = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (c >= p.cols) return;
  const float inv_rows = 1.0f / static_cast<float>(p.rows);
  auto count = [&](int b) {
    return static_cast<float>(min(p.rows, (b + 1) * p.rows_per_block) - b * p.rows_per_block);
  };
  const float ref = p.partial[c].x;            // block 0 always has rows
  float s1 = 0.f, s2 = 0.f;
  for (int b = lane; b < nblk; b += 32) {
    const float2 pb = p.partial[static_cast<long long>(b) * p.cols + c];
    const float n = count(b), d = pb.x - ref;
    s1 = fmaf(n, d, s1);
    s2 += fmaf(n * d, d, pb.y);
  }
  s1 = warp_sum(s1);
  s2 = warp_sum(s2);
  const float dm = s1 * inv_rows;              // mean - ref
  const float mean = ref + dm;
  const float var = fmaxf(fmaf(-s1, dm, s2), 0.f) * inv_rows;
  __syncwarp();                                // every lane has read the column's pairs
  if (lane == 0) {
    p.partial[c] = make_float2(mean, rsqrt_refined(var + p.eps));
    if (p.mean_out != nullptr) p.mean_out[c] = mean;
    if (p.var_out != nullptr) p.var_out[c] = var;
  }
}


template <typename T, int MODE>
__global__ void __launch_bounds__(kAxisThreads, 4) col_apply_kernel(const ColParams p) {
  pdl_prologue();                              // the merge kernel has completed when this returns
  using A = AxisRaw<T, MODE>;
  using E = Elem<T>;
  using Raw = typename A::Raw;
  constexpr int W = A::W;
  constexpr int UB = kColUB;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int lc = 1 << p.lc_shift;
  const int lcol = lane & (lc - 1);
  const int slot = warp * (32 >> p.lc_shift) + (lane >> p.lc_shift);
  const int ns = kAxisThreads >> p.lc_shift;
  const int cw = lc * W;
  const long long blk = static_cast<long long>(gridDim.y) - 1 - blockIdx.y;     // last read, first re-read
  const long long r0 = blk * p.rows_per_block;
  const long long r1 = min(p.rows, r0 + p.rows_per_block);
  const long long col0 = static_cast<long long>(blockIdx.x) * cw + lcol * W;
  if (col0 >= p.cols) return;
  float mean[W], scale[W], shift[W];
#pragma unroll
  for (int j = 0; j < W; ++j) {
    const float2 ms = (col0 + j < p.cols) ? p.partial[col0 + j] : make_float2(0.f, 0.f);
    mean[j] = ms.x;
    const float g = (p.gamma != nullptr && col0 + j < p.cols) ? E::load1(p.gamma, col0 + j) : 1.f;
    shift[j] = (p.beta != nullptr && col0 + j < p.cols) ? E::load1(p.beta, col0 + j) : 0.f;
    scale[j] = ms.y * g;
  }
  const uint64_t drop = p.l2_keep ? l2_policy_drop() : l2_policy_normal();
  const long long xstep = p.xs * ns, ystep = p.ys * ns;
  const T* px = reinterpret_cast<const T*>(p.x) + (r0 + slot) * p.xs + col0;
  T* py = reinterpret_cast<T*>(p.y) + (r0 + slot) * p.ys + col0;
  for (long long f = r0 + slot; f < r1; f += static_cast<long long>(UB) * ns) {
    const bool whole = f + (UB - 1) * ns < r1;
    Raw raw[UB];
#pragma unroll
    for (int u = 0; u < UB; ++u, px += xstep)
      if (whole || f + u * ns < r1) raw[u] = A::load_hint(px, drop);
#pragma unroll
    for (int u = 0; u < UB; ++u, py += ystep) {
      if (whole || f + u * ns < r1) {
        float v[W];
        A::unpack(raw[u], v);
#pragma unroll
        for (int j = 0; j < W; ++j) v[j] = fmaf(v[j] - mean[j], scale[j], shift[j]);
        A::store(py, A::pack(v));
      }
    }
  }
}

}  // namespace akg
