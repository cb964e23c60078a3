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

#include "tma.cuh"

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


// scan_flat_kernel: the vectorised CTA-per-row form of scan_kernel (below) with its two loops - rows, chunks of a row -
// flattened into one walk through the CTA's chunks: the loads keep running ahead across row ends, the two buffers of
// warp totals alternate from chunk to chunk across rows as well (no extra barrier at a row's end), and the loads can
// run more than one chunk ahead.  (A warp per row measured slower in this form, 0.82 against 0.94 on bf16
// [16384, 8192], and keeps scan_kernel.)
// DEPTH: how many chunks ahead of the one being scanned the vector loads run.  One is enough while four CTAs per SM
// keep the memory system busy.  A few long rows (fewer CTAs than two per SM) are bound by the load latency instead:
// a chunk's loads were issued only one chunk earlier, a chunk is scanned in a fraction of a microsecond, so every
// chunk waited for most of a memory round trip ([256, 262144] fp32: 64 chunks per row at about 1.5 us each).  With
// DEPTH 3 the loads are three chunks ahead (48 KB in flight per CTA, two CTAs per SM).  The chunk loop is unrolled
// DEPTH times so that every buffer of the ring is a fixed set of registers: shifting the ring by register moves
// made each iteration wait for loads still in flight and gained nothing.
template <bool PROD, typename T, int DEPTH>
__global__ void __launch_bounds__(32 * kScanMaxWarps, DEPTH > 1 ? 2 : 4) scan_flat_kernel(const ScanParams p) {
  constexpr bool VEC = true;
  constexpr bool WARP = false;
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
  const long long chunk = static_cast<long long>(U) * T_;
  const float id = scan_identity<PROD>();

  // the 16-byte vectors of a chunk are loaded DEPTH chunks ahead (the row's later chunks, or the first chunks of
  // the CTA's next rows): the loads follow a cursor of their own through the chunks this CTA (or warp) will scan
  uint4 ahead[DEPTH][U];
  long long frow = row0, fbase = 0;
  auto load_next = [&](uint4 (&dst)[U]) {
    if (frow < p.rows) {
      const T* xf = reinterpret_cast<const T*>(p.x) + frow * p.xs;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const long long i = fbase + static_cast<long long>(u) * T_ + tid;
        if (i < nvec) dst[u] = ld_stream(xf + i * EPV);
      }
      fbase += chunk;
      if (fbase >= nvec) { fbase = 0; frow += row_step; }
    }
  };
  if (VEC) {
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) load_next(ahead[d]);
  }

  long long row = row0, base = 0;
  float carry = id;
  int par = 0;
  while (row < p.rows) {
#pragma unroll
    for (int d = 0; d < DEPTH; ++d) {
      if (row >= p.rows) break;                                 // the same for every thread that shares a barrier
      const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs;
      T* yr = reinterpret_cast<T*>(p.y) + row * p.ys;
      float v[U][EPV];
      // ---- the chunk's values (vectors beyond the row hold the identity)
      if (VEC) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) raw[u] = ahead[d][u];
        load_next(ahead[d]);
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
      for (int s = 1; s < 32; s <<= 1) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const float o = __shfl_up_sync(0xffffffffu, incl[u], s);
          if (lane >= s) incl[u] = scan_op<PROD>(o, incl[u]);
        }
      }
      if (!WARP) {
        // (two buffers alternate from chunk to chunk, across rows as well: a thread can write the buffer of
        // chunk k + 2 only after the barrier of chunk k + 1, which every thread reaches after reading chunk k's)
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
      par ^= 1;
      base += chunk;
      if (base >= nvec) { base = 0; row += row_step; carry = id; }
    }
  }
}


// ------------------------------------------------------------------------------------------------
// scan_short_kernel: rows of at most 4 * L vectors (L = 4, 8 or 16 lanes per row, so up to 64 vectors: a
// kilobyte).  A warp per row leaves most lanes without a vector on such rows (bf16 rows of 256 columns
// are 32 vectors: one per lane, three quarters of the chunk empty, and the row's chain of load, scan
// and store is paid for 512 bytes: 0.35 - 0.45 of the copy rate).  Here L lanes own a row and hold up to
// four of its vectors each (lane l of the group: vectors l, l + L, ...), so a warp works on 32 / L rows
// at once with four loads in flight per lane, shuffle scans of log2 L steps inside the group, and the
// next rows of the warp loaded while the current ones are scanned.  No shared memory, no barrier.
// ------------------------------------------------------------------------------------------------
template <bool PROD, typename T, int L>
__global__ void __launch_bounds__(256, 4) scan_short_kernel(const ScanParams p) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int U = kScanU;
  constexpr int RPW = 32 / L;                                   // rows per warp
  const int lane = threadIdx.x & 31;
  const int gl = lane & (L - 1);                                // lane inside the row's group
  const int nvec = static_cast<int>(p.cols / EPV);
  const float id = scan_identity<PROD>();
  const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
  long long row = (static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5)) * RPW + lane / L;
  const long long row_step = warps * RPW;

  uint4 ahead[U];
  auto load_row = [&](long long r) {
    if (r < p.rows) {
      const T* xr = reinterpret_cast<const T*>(p.x) + r * p.xs;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = u * L + gl;
        if (i < nvec) ahead[u] = ld_stream(xr + static_cast<long long>(i) * EPV);
      }
    }
  };
  load_row(row);
  // (the loop bound is the warp's first row, so that every lane of a warp takes part in the shuffles)
  for (long long base = row - lane / L; base < p.rows; base += row_step, row += row_step) {
    float v[U][EPV];
    const bool active = row < p.rows;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = u * L + gl;
      float f[EPV];
      if (active && i < nvec) E::unpack(ahead[u], f);
#pragma unroll
      for (int j = 0; j < EPV; ++j) v[u][j] = (active && i < nvec) ? f[j] : id;
    }
    load_row(row + row_step);
    float incl[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
      for (int j = 1; j < EPV; ++j) v[u][j] = scan_op<PROD>(v[u][j - 1], v[u][j]);
      incl[u] = v[u][EPV - 1];
    }
#pragma unroll
    for (int d = 1; d < L; d <<= 1) {
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const float o = __shfl_up_sync(0xffffffffu, incl[u], d, L);
        if (gl >= d) incl[u] = scan_op<PROD>(o, incl[u]);
      }
    }
    float before = id;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float tot = __shfl_sync(0xffffffffu, incl[u], L - 1, L);
      const float excl = __shfl_up_sync(0xffffffffu, incl[u], 1, L);
      float mine = before;
      if (gl > 0) mine = scan_op<PROD>(mine, excl);
      before = scan_op<PROD>(before, tot);
      const int i = u * L + gl;
      if (active && i < nvec) {
        float o[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) o[j] = scan_op<PROD>(mine, v[u][j]);
        st_stream(yr + static_cast<long long>(i) * EPV, E::pack(o));
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// scan_split_kernel: few, long rows (a CTA per row would leave most SMs idle and walk a megabyte on
// its own).  A cluster of CS CTAs owns a row at a time and CTA k its slice k of slice_vecs vectors:
//   phase 1  the slice's total: streaming loads marked "keep in L2", eight per thread in flight,
//            thread -> warp -> CTA reduction
//   exchange every CTA sends its total to every CTA of the cluster (one 16-byte st.async into the
//            receiver's shared memory, counted on the receiver's mbarrier: the scheme of
//            split_kernel); a CTA's carry-in is the combination, in slice order, of the totals of
//            the slices before its own - a look-back that never leaves the cluster: no flag in
//            global memory, nothing to spin on but the CTA's own mbarrier, and that wait is bounded
//   phase 2  the chunked scan of scan_kernel over the slice, starting from the carry-in; the slice
//            is read again, now from L2 ("evict first"), and stored
// HBM sees one read and one write per element.  Vectorised rows only.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 scan_ld_hint(const void* p, uint64_t pol) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol) : "memory");
  return v;
}

template <bool PROD, typename T>
__global__ void __launch_bounds__(256, 4) scan_split_kernel(const ScanParams p, const int slice_vecs,
                                                           int* status, const unsigned wait_us) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int U = kScanU;
  constexpr int T_ = 256, NW = T_ / 32;
  __shared__ float wtot[2][U][NW];
  __shared__ float red[NW];
  __shared__ __align__(16) float4 inbox[2][kMaxCluster];
  __shared__ __align__(8) uint64_t xbar[2];
  __shared__ int cta_failed;
  const int tid = static_cast<int>(threadIdx.x), lane = tid & 31, warp = tid >> 5;
  const uint32_t cs = cluster_size(), rank = cluster_rank();
  const long long row_step = cluster_count();
  const int nvec = static_cast<int>(p.cols / EPV);
  const int v0 = static_cast<int>(rank) * slice_vecs;
  const int my_vecs = max(0, min(slice_vecs, nvec - v0));
  const float id = scan_identity<PROD>();
  uint64_t keep, drop;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(drop));

  if (tid == 0) {
    cta_failed = 0;
    mbar_init(smem_addr(&xbar[0]), 1);
    mbar_init(smem_addr(&xbar[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (cs > 1) { cluster_arrive(); cluster_wait(); }

  int par = 0;
  uint32_t phases = 0;
  int mv = my_vecs;                        // -1 once a wait ran out: nothing is loaded or stored any more
  for (long long row = cluster_id(); row < p.rows; row += row_step, par ^= 1) {
    if (*reinterpret_cast<volatile int*>(&cta_failed)) mv = -1;
    const uint4* xs = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p.x) + row * p.xs) + v0;
    uint4* ys = reinterpret_cast<uint4*>(reinterpret_cast<T*>(p.y) + row * p.ys) + v0;

    // ---- phase 1: total of the slice
    float t0 = id, t1 = id;
    int v = tid;
    for (; v + 7 * T_ < mv; v += 8 * T_) {
      uint4 raw[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) raw[u] = scan_ld_hint(xs + v + u * T_, keep);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        float f[EPV];
        E::unpack(raw[u], f);
#pragma unroll
        for (int j = 0; j < EPV; j += 2) { t0 = scan_op<PROD>(t0, f[j]); t1 = scan_op<PROD>(t1, f[j + 1]); }
      }
    }
    for (; v < mv; v += T_) {
      float f[EPV];
      E::unpack(scan_ld_hint(xs + v, keep), f);
#pragma unroll
      for (int j = 0; j < EPV; j += 2) { t0 = scan_op<PROD>(t0, f[j]); t1 = scan_op<PROD>(t1, f[j + 1]); }
    }
    float tot = scan_op<PROD>(t0, t1);
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) tot = scan_op<PROD>(tot, __shfl_xor_sync(0xffffffffu, tot, m));
    if (lane == 0) red[warp] = tot;
    __syncthreads();
    tot = red[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) tot = scan_op<PROD>(tot, red[w]);

    // ---- exchange; carry-in = totals of the slices before mine, in slice order
    float carry = id;
    if (cs > 1) {
      if (tid == 0) mbar_expect_tx(smem_addr(&xbar[par]), cs * 16u);
      if (tid < static_cast<int>(cs))
        st_async_f32x4(smem_addr(&inbox[par][rank]), smem_addr(&xbar[par]), static_cast<uint32_t>(tid), tot, 0.f, 0.f, 0.f);
      if (mv >= 0 && !mbar_wait_timed<true>(smem_addr(&xbar[par]), (phases >> par) & 1u, status, wait_us)) {
        mv = -1;
        cta_failed = 1;
      }
      phases ^= 1u << par;
      for (uint32_t k = 0; k < rank; ++k) carry = scan_op<PROD>(carry, inbox[par][k].x);
    }

    // ---- phase 2: scan of the slice from the carry-in (chunks of U * T_ vectors, as scan_kernel)
    int cpar = 0;
    uint4 ahead[U];                        // a chunk's vectors are loaded one chunk ahead
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = u * T_ + tid;
      if (i < mv) ahead[u] = scan_ld_hint(xs + i, drop);
    }
    for (int base = 0; base < my_vecs; base += U * T_, cpar ^= 1) {     // (every thread: the chunks have a barrier)
      float val[U][EPV];
      uint4 raw[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        raw[u] = ahead[u];
        const int i = base + (U + u) * T_ + tid;
        if (i < mv) ahead[u] = scan_ld_hint(xs + i, drop);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = base + u * T_ + tid;
        float f[EPV];
        if (i < mv) E::unpack(raw[u], f);
#pragma unroll
        for (int j = 0; j < EPV; ++j) val[u][j] = (i < mv) ? f[j] : id;
      }
      float incl[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int j = 1; j < EPV; ++j) val[u][j] = scan_op<PROD>(val[u][j - 1], val[u][j]);
        incl[u] = val[u][EPV - 1];
      }
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const float o = __shfl_up_sync(0xffffffffu, incl[u], d);
          if (lane >= d) incl[u] = scan_op<PROD>(o, incl[u]);
        }
      }
      if (lane == 31) {
#pragma unroll
        for (int u = 0; u < U; ++u) wtot[cpar][u][warp] = incl[u];
      }
      __syncthreads();
      float before = carry;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float pre = id, tot_u = id;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          const float t = wtot[cpar][u][w];
          if (w < warp) pre = scan_op<PROD>(pre, t);
          tot_u = scan_op<PROD>(tot_u, t);
        }
        float mine = scan_op<PROD>(before, pre);
        before = scan_op<PROD>(before, tot_u);
        const float excl = __shfl_up_sync(0xffffffffu, incl[u], 1);
        if (lane > 0) mine = scan_op<PROD>(mine, excl);
        const int i = base + u * T_ + tid;
        if (i < mv) {
          float o[EPV];
#pragma unroll
          for (int j = 0; j < EPV; ++j) o[j] = scan_op<PROD>(mine, val[u][j]);
          st_stream(ys + i, E::pack(o));
        }
      }
      carry = before;
    }
    __syncthreads();                       // red[] and wtot[] of the next row
  }
  if (cs > 1) { cluster_arrive(); cluster_wait(); }   // nobody leaves while a peer may still send to it
}

}  // namespace akg
