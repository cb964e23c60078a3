// Ring-fed register kernels (the TMA family for rows that fit one CTA's registers).
//
// Persistent CTAs, one row per CTA at a time.  Thread 0 keeps NBUF bulk copies
// (cp.async.bulk global -> shared, untiled, no multicast) in flight ahead of the row
// being processed; the CTA waits on the row's mbarrier, pulls its vectors into
// registers with 128-bit shared loads and runs the same lean row bodies as the REG
// family.  Load latency is thereby hidden by the ring instead of by occupancy, and the
// ring depth is independent of the register budget.  A buffer is handed back to the
// copy engine as soon as the row body has passed its reduction barrier (every thread
// has read its part by then).
#pragma once

#include "kernels_softmax.cuh"

namespace akg {

constexpr unsigned kRingHeader = 128;          // mbarriers (kMaxBuf x 8 bytes)

struct RowRing {
  uint32_t bars, bufs, buf_bytes;
  int nbuf;

  __device__ __forceinline__ void init(unsigned char* smem, uint32_t row_bytes, int n) {
    bars = smem_addr(smem);
    bufs = smem_addr(smem + kRingHeader);
    buf_bytes = (row_bytes + 127u) & ~127u;
    nbuf = n;
    if (threadIdx.x == 0) {
      for (int b = 0; b < n; ++b) mbar_init(bars + 8u * b, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
  }
  __device__ __forceinline__ uint32_t buf(int b) const { return bufs + static_cast<uint32_t>(b) * buf_bytes; }
  // thread 0 only: start the copy of `bytes` (a multiple of 16; 0 = nothing to fetch)
  __device__ __forceinline__ void issue(const void* src, uint32_t bytes, int b) const {
    const uint32_t bar = bars + 8u * b;
    if (bytes == 0) { mbar_arrive(bar); return; }
    mbar_expect_tx(bar, bytes);
    constexpr uint32_t kChunk = 32768;
    for (uint32_t off = 0; off < bytes; off += kChunk)
      bulk_load(buf(b) + off, reinterpret_cast<const unsigned char*>(src) + off, min(kChunk, bytes - off), bar);
  }
  __device__ __forceinline__ bool wait(int b, uint32_t phase, const RowParams& p) const {
    return mbar_wait_timed(bars + 8u * b, phase, p.status, p.wait_us);
  }
  // thread 0, before a CTA that gave up leaves: no copy may still be on its way into the CTA's shared
  // memory; `pending` buffers starting at b (phase of the first) have one
  __device__ __forceinline__ void drain(int b, uint32_t phase, int pending, const RowParams& p) const {
    for (; pending > 0; --pending) {
      (void)mbar_wait_timed(bars + 8u * b, phase, nullptr, p.wait_us);
      if (++b == nbuf) { b = 0; phase ^= 1u; }
    }
  }
};

template <int OP, typename T, int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS, kRegMinBlocks<THREADS>) ring_norm_full(const RowParams p, const int nbuf) {
  pdl_prologue();
  constexpr int EPV = Elem<T>::EPV;
  constexpr int NW = THREADS / 32;
  constexpr uint32_t kRowBytes = THREADS * VPT * 16u;
  extern __shared__ __align__(128) unsigned char ring_smem[];
  __shared__ float red[2][2][NW];
  RowRing ring;
  ring.init(ring_smem, kRowBytes, nbuf);

  // A wait that runs out (see mbar_wait_timed) makes its thread "dead": it stores nothing any more and
  // waits for nothing, but still runs the row bodies, whose barriers its CTA needs.  The flag in shared
  // memory spreads the state to the whole CTA at the next row (the row body's barrier lies in between),
  // so that a lost copy costs one wait, not one per remaining row.
  __shared__ int cta_dead;
  if (threadIdx.x == 0) cta_dead = 0;
  __syncthreads();
  const long long step = gridDim.x;
  const T* x = reinterpret_cast<const T*>(p.x);
  int in_flight = 0;                                   // thread 0: copies issued and not yet waited for
  if (threadIdx.x == 0 && !p.no_copies) {
    long long r = blockIdx.x;
    for (int b = 0; b < nbuf && r < p.rows; ++b, r += step) { ring.issue(x + r * p.xs, kRowBytes, b); ++in_flight; }
  }
  int b = 0, parity = 0;
  uint32_t phase = 0;
  bool dead = false;
  for (long long row = blockIdx.x; row < p.rows; row += step, parity ^= 1) {
    if (!dead && *reinterpret_cast<volatile int*>(&cta_dead)) dead = true;
    if (!dead) {
      if (ring.wait(b, phase, p)) { if (threadIdx.x == 0) --in_flight; }
      else { dead = true; cta_dead = 1; }
    }
    norm_row_full<OP, T, THREADS, VPT, THREADS, true>(p, row, threadIdx.x, red[parity], ring.buf(b), dead);
    if (threadIdx.x == 0 && !dead && !p.no_copies) {
      const long long next = row + step * nbuf;
      if (next < p.rows) { ring.issue(x + next * p.xs, kRowBytes, b); ++in_flight; }
    }
    if (!dead && ++b == nbuf) { b = 0; phase ^= 1u; }
  }
  if (threadIdx.x == 0 && dead) ring.drain(b, phase, in_flight, p);
  (void)EPV;
}

template <int OP, typename T, int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS, kRegMinBlocks<THREADS>) ring_softmax(const RowParams p, const int nbuf) {
  pdl_prologue();
  constexpr int EPV = Elem<T>::EPV;
  constexpr int NW = THREADS / 32;
  static_assert(VPT <= 8, "row body is specialised for up to eight iterations");
  extern __shared__ __align__(128) unsigned char ring_smem[];
  __shared__ float red[2][2][NW];
  const int nvec = static_cast<int>(p.cols / EPV);
  RowRing ring;
  ring.init(ring_smem, static_cast<uint32_t>(nvec) * 16u, nbuf);

  const long long step = gridDim.x;
  const T* x = reinterpret_cast<const T*>(p.x);
  auto live_bytes = [&](long long r) -> uint32_t {
    const int live = static_cast<int>(live_cols(p, r));
    return static_cast<uint32_t>((live + EPV - 1) / EPV) * 16u;
  };
  int in_flight = 0;                                   // thread 0: copies issued and not yet waited for
  if (threadIdx.x == 0 && !p.no_copies) {
    long long r = blockIdx.x;
    for (int b = 0; b < nbuf && r < p.rows; ++b, r += step) {
      const long long mr = balanced_row(p, r);
      ring.issue(x + mr * p.xs, live_bytes(mr), b);
      ++in_flight;
    }
  }
  int b = 0, parity = 0;
  uint32_t phase = 0;
  bool dead = false;
  for (long long item = blockIdx.x; item < p.rows; item += step, parity ^= 1) {
    const long long row = balanced_row(p, item);
    // (only forced launches reach this kernel: the CTA-wide vote costs it a barrier per row)
    if (__syncthreads_or(ring.wait(b, phase, p) ? 0 : 1)) { dead = true; break; }
    if (threadIdx.x == 0) --in_flight;
    softmax_row_dispatch<OP, T, THREADS, VPT, VPT, THREADS, true>(p, row, threadIdx.x, nvec, red[parity],
                                                                  ring.buf(b));
    if (threadIdx.x == 0 && !p.no_copies) {
      const long long next = item + step * nbuf;
      if (next < p.rows) {
        const long long mr = balanced_row(p, next);
        ring.issue(x + mr * p.xs, live_bytes(mr), b);
        ++in_flight;
      }
    }
    if (++b == nbuf) { b = 0; phase ^= 1u; }
  }
  // a CTA that gave up stores nothing more; the copy it waited for in vain is still counted
  if (threadIdx.x == 0 && dead) ring.drain(b, phase, in_flight, p);
}

}  // namespace akg
