// Cumulative sum / product along the last axis ("cumulative operations" of the reduction
// category, Section 3.6): y[r, c] = x[r, 0] (+ or *) ... (+ or *) x[r, c], inclusive.
//
// One pass: every element is read once and written once.  A CTA of T threads owns a row and
// walks it in chunks of U * T vectors; thread t holds vectors t, t + T, ... of the chunk (so
// loads and stores stay coalesced) and issues its U loads together.  Inside a chunk the order
// of the elements is (u, t, j): each vector is scanned in registers, the vector totals are
// scanned across the lanes of a warp (U independent shuffle scans), the warps' totals go
// through shared memory (one barrier per chunk, two buffers), and every thread adds up what
// precedes its vectors: the carry of the earlier chunks, the totals of the earlier u, the totals
// of the earlier warps of its own u.  fp32 arithmetic throughout; one rounding at the store.
#pragma once

#include "common.cuh"

namespace akg {

struct ScanParams {
  const void* x;
  void* y;
  long long rows, cols, xs, ys;
};

template <bool PROD> __device__ __forceinline__ float scan_op(float a, float b) { return PROD ? a * b : a + b; }
template <bool PROD> __device__ __forceinline__ float scan_identity() { return PROD ? 1.f : 0.f; }

constexpr int kScanU = 4;
constexpr int kScanMaxWarps = 8;

// WARP = true: every warp of the CTA owns rows of its own (short rows: no shared memory and no
// CTA barrier, the warp's total comes from lane 31 by shuffle); WARP = false: the CTA owns a row.
template <bool PROD, typename T, bool VEC, bool WARP = false>
__global__ void __launch_bounds__(32 * kScanMaxWarps, 4) scan_kernel(const ScanParams p) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = VEC ? E::EPV : 1;
  constexpr int U = kScanU;
  __shared__ float wtot[2][U][kScanMaxWarps];
  const int lane = threadIdx.x & 31;
  const int T_ = WARP ? 32 : static_cast<int>(blockDim.x);      // threads per row
  const int tid = WARP ? lane : static_cast<int>(threadIdx.x);  // position among them
  const int NW = T_ >> 5;
  const int warp = WARP ? 0 : static_cast<int>(threadIdx.x >> 5);
  const long long row0 = WARP ? static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5)
                              : static_cast<long long>(blockIdx.x);
  const long long row_step = WARP ? static_cast<long long>(gridDim.x) * (blockDim.x >> 5)
                                  : static_cast<long long>(gridDim.x);
  const long long nvec = (p.cols + EPV - 1) / EPV;              // VEC: cols is a multiple of EPV
  const float id = scan_identity<PROD>();

  // the 16-byte vectors of a chunk are loaded one chunk ahead (the row's next chunk, or the first
  // chunk of the CTA's next row), so that their latency hides behind the scan of the current one
  uint4 ahead[U];
  auto load_chunk = [&](const T* xr, long long base) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const long long i = base + static_cast<long long>(u) * T_ + tid;
      if (i < nvec) ahead[u] = ld_stream(xr + i * EPV);
    }
  };
  if (VEC && row0 < p.rows) load_chunk(reinterpret_cast<const T*>(p.x) + row0 * p.xs, 0);

  for (long long row = row0; row < p.rows; row += row_step) {
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys;
    float carry = id;
    int par = 0;
    for (long long base = 0; base < nvec; base += static_cast<long long>(U) * T_, par ^= 1) {
      float v[U][EPV];
      // ---- load the chunk (vectors beyond the row hold the identity)
      if (VEC) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) raw[u] = ahead[u];
        const long long nbase = base + static_cast<long long>(U) * T_;
        if (nbase < nvec) load_chunk(xr, nbase);
        else if (row + row_step < p.rows) load_chunk(xr + row_step * p.xs, 0);
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const long long i = base + static_cast<long long>(u) * T_ + tid;
          float f[E::EPV];
          if (i < nvec) E::unpack(raw[u], f);
#pragma unroll
          for (int j = 0; j < EPV; ++j) v[u][j] = (i < nvec) ? f[j] : id;
        }
      } else {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const long long i = base + static_cast<long long>(u) * T_ + tid;
          v[u][0] = (i < nvec) ? E::load1(xr, i) : id;
        }
      }
      // ---- scan inside each vector, then the vector totals across the warp
      float incl[U];                                            // inclusive scan of the totals over lanes
#pragma unroll
      for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int j = 1; j < EPV; ++j) v[u][j] = scan_op<PROD>(v[u][j - 1], v[u][j]);
        incl[u] = v[u][EPV - 1];
      }
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const float o = __shfl_up_sync(0xffffffffu, incl[u], d);
          if (lane >= d) incl[u] = scan_op<PROD>(o, incl[u]);
        }
      }
      if (!WARP) {
        if (lane == 31) {
#pragma unroll
          for (int u = 0; u < U; ++u) wtot[par][u][warp] = incl[u];
        }
        __syncthreads();
      }
      // ---- what precedes this thread's vector u: carry, earlier u, earlier warps, earlier lanes
      float before = carry;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        // the warps' totals of this u are combined on their own, so that the carry picks up one
        // operation per u (its rounding error grows with the number of chunks, not of warps)
        float pre = id, tot = id;
        if (WARP) {
          tot = __shfl_sync(0xffffffffu, incl[u], 31);
        } else {
          for (int w = 0; w < NW; ++w) {
            const float t = wtot[par][u][w];
            if (w < warp) pre = scan_op<PROD>(pre, t);
            tot = scan_op<PROD>(tot, t);
          }
        }
        float mine = scan_op<PROD>(before, pre);                // carry, all of the earlier u, earlier warps
        before = scan_op<PROD>(before, tot);
        const float excl = __shfl_up_sync(0xffffffffu, incl[u], 1);
        if (lane > 0) mine = scan_op<PROD>(mine, excl);
        const long long i = base + static_cast<long long>(u) * T_ + tid;
        if (i < nvec) {
          float o[EPV];
#pragma unroll
          for (int j = 0; j < EPV; ++j) o[j] = scan_op<PROD>(mine, v[u][j]);
          if (VEC) {
            float f[E::EPV];
#pragma unroll
            for (int j = 0; j < EPV; ++j) f[j] = o[j];
            st_stream(yr + i * EPV, E::pack(f));
          } else {
            E::store1(yr, i, o[0]);
          }
        }
      }
      carry = before;
    }
    if (!WARP) __syncthreads();                                 // wtot[par] of the next row
  }
}

}  // namespace akg
