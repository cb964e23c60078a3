// Arg-max / arg-min over the last axis ("argmax/argmin" of the reduction category, Section 3.6).
// out[r] = the smallest column index at which row r attains its maximum (minimum); values are
// compared exactly as stored (-0 == +0); a NaN counts as the extreme for both, the first NaN wins.
//
// Read-only and HBM-bound, so the loop does as little as it can per element and never branches: a
// NaN-propagating max (min) over the 8 or 4 values of a vector, and a select that keeps the
// better of that and the thread's best so far together with the vector's index.  The position
// inside the winning vector is looked up once per thread and row.  Threads merge through a 64-bit key (order-preserving image of
// the value in the high word, inverted index in the low word), whose maximum is the winner with
// the lowest index.  G threads own a row: a warp (short rows, several rows per CTA) or the CTA.
#pragma once

#include "common.cuh"

namespace akg {

struct ArgParams {
  const void* x;
  long long* out;
  long long rows, cols, xs;
};

template <bool MIN> __device__ __forceinline__ float nan_ext(float a, float b) {
  float r;
  if (MIN) asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  else asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return r;
}

// does v beat the best so far?  (NaN beats every number; nothing beats a NaN; equals do not beat)
template <bool MIN> __device__ __forceinline__ bool arg_beats(float v, float best) {
  if (best != best) return false;
  if (v != v) return true;
  return MIN ? (v < best) : (v > best);
}

// order-preserving 32-bit image: larger = better candidate; NaN is the largest; -0 maps like +0
template <bool MIN> __device__ __forceinline__ uint32_t arg_key(float v) {
  if (v != v) return 0xffffffffu;
  uint32_t b = __float_as_uint(v + 0.0f);
  b = (b & 0x80000000u) ? ~b : (b | 0x80000000u);            // ascending with the value
  return MIN ? ~b : b;
}

// The 64-bit key of the best candidate among vectors v_begin + tg, v_begin + tg + G, ... < v_end of
// the row at xr (elements when !VEC); 0 if the thread saw nothing.  Larger key = better candidate,
// ties resolved towards the lower index.
// PRE: the caller may already hold the thread's first four vectors (v_begin + tg + u * G, u < 4)
// in `first` (use_first says whether it does), loaded while it worked on the row before.
template <bool MIN, typename T, bool VEC, bool PRE = false>
__device__ __forceinline__ unsigned long long arg_thread_key(const T* xr, long long v_begin, long long v_end,
                                                             int tg, int G, const uint4* first = nullptr,
                                                             bool use_first = false) {
  using E = Elem<T>;
  constexpr int EPV = VEC ? E::EPV : 1;
  constexpr int U = 4;
  // the extreme of nothing: every first value beats it, and it loses every merge
  float best = MIN ? __int_as_float(0x7f800000) : kNegInf;
  long long bvec = -1;                                        // vector (element when !VEC) holding it
  bool seen = false;

  // per vector: its extreme (NaN-propagating), and a branch-free "take it if it improves"
  auto visit = [&](const float (&v)[EPV], long long vec_index) {
    float ext = v[0];
#pragma unroll
    for (int j = 1; j < EPV; ++j) ext = nan_ext<MIN>(ext, v[j]);
    const bool take = !seen || arg_beats<MIN>(ext, best);
    best = take ? ext : best;
    bvec = take ? vec_index : bvec;
    seen = true;
  };

  long long i = v_begin + tg;
  if (VEC) {
    if (PRE && use_first) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float v[E::EPV];
        E::unpack(first[u], v);
        float w[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) w[j] = v[j];
        visit(w, i + u * G);
      }
      i += U * G;
    }
    for (; i + (U - 1) * G < v_end; i += U * G) {
      uint4 raw[U];
#pragma unroll
      for (int u = 0; u < U; ++u) raw[u] = ld_stream(xr + (i + u * G) * EPV);
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float v[E::EPV];
        E::unpack(raw[u], v);
        float w[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) w[j] = v[j];
        visit(w, i + u * G);
      }
    }
  }
  for (; i < v_end; i += G) {
    float w[EPV];
    if (VEC) {
      float v[E::EPV];
      E::unpack(ld_stream(xr + i * EPV), v);
#pragma unroll
      for (int j = 0; j < EPV; ++j) w[j] = v[j];
    } else {
      w[0] = E::load1(xr, i);
    }
    visit(w, i);
  }
  if (!seen) return 0ull;
  // the position inside the winning vector: its first element equal to the extreme (first NaN
  // if the extreme is NaN); one more load per thread and row, served by L2
  long long bidx = bvec * EPV;
  if (VEC) {
    float v[E::EPV];
    E::unpack(ld_stream(xr + bvec * EPV), v);
    int pos = EPV - 1;
#pragma unroll
    for (int j = EPV - 1; j >= 0; --j)
      if ((best != best) ? (v[j] != v[j]) : (v[j] == best)) pos = j;
    bidx += pos;
  }
  return (static_cast<unsigned long long>(arg_key<MIN>(best)) << 32) |
         (0xffffffffull - static_cast<unsigned long long>(bidx));
}

__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long key) {
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) {
    const unsigned long long o = __shfl_xor_sync(0xffffffffu, key, m);
    key = o > key ? o : key;
  }
  return key;
}

template <bool MIN, typename T, int G, int THREADS, bool VEC>
__global__ void __launch_bounds__(THREADS) arg_kernel(const ArgParams p) {
  pdl_prologue();
  constexpr int EPV = VEC ? Elem<T>::EPV : 1;
  constexpr int RPC = THREADS / G;
  constexpr int NW = G / 32;
  __shared__ unsigned long long red[THREADS / 32];
  const int tg = threadIdx.x % G;
  const int grp = threadIdx.x / G;
  const long long nvec = p.cols / EPV;                          // VEC: cols is a multiple of EPV

  if constexpr (VEC && G == THREADS) {
    // a CTA per row, grid-stride: the first four vectors of the CTA's next row are loaded before
    // the current row is searched, so that their latency hides behind it
    const bool can_pre = nvec >= 4 * G;
    long long row = blockIdx.x;
    if (row >= p.rows) return;
    uint4 pre[4];
    if (can_pre) {
      const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs;
#pragma unroll
      for (int u = 0; u < 4; ++u) pre[u] = ld_stream(xr + (static_cast<long long>(tg) + u * G) * EPV);
    }
    for (; row < p.rows; row += gridDim.x) {
      uint4 cur[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) cur[u] = pre[u];
      const long long nrow = row + gridDim.x;
      if (can_pre && nrow < p.rows) {
        const T* xn = reinterpret_cast<const T*>(p.x) + nrow * p.xs;
#pragma unroll
        for (int u = 0; u < 4; ++u) pre[u] = ld_stream(xn + (static_cast<long long>(tg) + u * G) * EPV);
      }
      unsigned long long key = arg_thread_key<MIN, T, VEC, true>(reinterpret_cast<const T*>(p.x) + row * p.xs, 0, nvec,
                                                                 tg, G, cur, can_pre);
      key = warp_max_key(key);
      __syncthreads();                                          // red is reused by the next row
      if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = key;
      __syncthreads();
      key = red[0];
#pragma unroll
      for (int w = 1; w < NW; ++w) key = red[w] > key ? red[w] : key;
      if (tg == 0) p.out[row] = static_cast<long long>(0xffffffffull - (key & 0xffffffffull));
    }
    return;
  }

  for (long long rb = static_cast<long long>(blockIdx.x) * RPC; rb < p.rows; rb += static_cast<long long>(gridDim.x) * RPC) {
    const long long row = rb + grp;
    const bool have = row < p.rows;
    unsigned long long key = 0ull;
    if (have) key = arg_thread_key<MIN, T, VEC>(reinterpret_cast<const T*>(p.x) + row * p.xs, 0, nvec, tg, G);
    key = warp_max_key(key);
    if (NW > 1) {
      __syncthreads();                                          // red is reused by the next row
      if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = key;
      __syncthreads();
      key = red[0];
#pragma unroll
      for (int w = 1; w < NW; ++w) key = red[w] > key ? red[w] : key;
    }
    if (have && tg == 0) p.out[row] = static_cast<long long>(0xffffffffull - (key & 0xffffffffull));
  }
}

// Few, long rows (a batch of vocabulary-sized rows): a row is cut into gridDim.x segments, one
// CTA each, and the segments' keys meet in an atomic maximum on the row's output word, which a
// first kernel has cleared and a last one turns into the index.  Three launches, one stream.
__global__ void arg_clear_kernel(const ArgParams p) {
  pdl_prologue();
  for (long long r = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; r < p.rows;
       r += static_cast<long long>(gridDim.x) * blockDim.x)
    p.out[r] = 0;
}

template <bool MIN, typename T, bool VEC>
__global__ void __launch_bounds__(256) arg_split_kernel(const ArgParams p, const long long seg_vecs) {
  pdl_prologue();
  constexpr int EPV = VEC ? Elem<T>::EPV : 1;
  __shared__ unsigned long long red[8];
  const long long nvec = p.cols / EPV;
  const long long v0 = static_cast<long long>(blockIdx.x) * seg_vecs;
  const long long v1 = min(nvec, v0 + seg_vecs);
  for (long long row = blockIdx.y; row < p.rows; row += gridDim.y) {
    unsigned long long key = arg_thread_key<MIN, T, VEC>(reinterpret_cast<const T*>(p.x) + row * p.xs, v0, v1,
                                                         static_cast<int>(threadIdx.x), 256);
    key = warp_max_key(key);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x == 0) {
      key = red[0];
#pragma unroll
      for (int w = 1; w < 8; ++w) key = red[w] > key ? red[w] : key;
      if (key != 0ull) atomicMax(reinterpret_cast<unsigned long long*>(p.out) + row, key);
    }
  }
}

__global__ void arg_finish_kernel(const ArgParams p) {
  pdl_prologue();
  for (long long r = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; r < p.rows;
       r += static_cast<long long>(gridDim.x) * blockDim.x) {
    const unsigned long long key = reinterpret_cast<const unsigned long long*>(p.out)[r];
    p.out[r] = static_cast<long long>(0xffffffffull - (key & 0xffffffffull));
  }
}

}  // namespace akg
