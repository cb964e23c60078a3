// smem_kernel: rows staged in shared memory by the bulk-copy engine (TMA, untiled
// cp.async.bulk, no multicast), for rows that do not fit the register file.
//
// A cluster of CS CTAs (CS = 1 for the "TMA" family, 2..16 for the "CLUSTER" family)
// owns one row at a time; CTA k of the cluster keeps slice k of the row in shared
// memory.  Each CTA has a ring of NBUF slice buffers: while the slice of row i is being
// reduced, normalised and stored, the copies for rows i+1 .. i+NBUF-1 are in flight.
// Per row: wait for the slice -> pass 1 over shared memory (thread-local statistics)
// -> CTA reduction -> partial statistics written into every peer's shared memory
// (distributed shared memory) -> cluster barrier -> pass 2 over shared memory
// (normalise, 128-bit stores) -> refill the buffer.  HBM traffic stays at one read and
// one write per element; 12 bytes per CTA cross the cluster per row.
#pragma once

#include "kernels_basic.cuh"
#include "tma.cuh"

namespace akg {



// Fold one vector of EPV (masked) values into the running thread statistics.
template <int OP, int EPV>
__device__ __forceinline__ void fold_vector(Stat& st, const float (&z)[EPV], float l2e = kLog2e) {
  if (OpTraits<OP>::kSoftmaxLike) {
    float mv = z[0];
#pragma unroll
    for (int j = 1; j < EPV; ++j) mv = fmaxf(mv, z[j]);
    const float mn = fmaxf(st.a, mv);
    const float ms = (mn == kNegInf) ? 0.f : mn;
    float acc = st.b * exp_diff(st.a, ms, l2e);
    // vectors of eight are 16-bit storage: the exponent as one fused multiply-add (its rounding,
    // below 1e-5 relative, is far inside the 2^-9 of the stored result); fp32 keeps the exact difference
    constexpr bool kFused = (EPV == 8);
    const float nms = -ms * l2e;
#pragma unroll
    for (int j = 0; j < EPV; ++j) acc += kFused ? ex2_approx(fmaf(z[j], l2e, nms)) : exp_diff(z[j], ms, l2e);
    st.a = mn; st.b = acc;
  } else if (OP == OP_LAYERNORM) {
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < EPV; ++j) sum += z[j];
    const float mean = sum * (1.0f / EPV);
    float m2 = 0.f;
#pragma unroll
    for (int j = 0; j < EPV; ++j) { const float d = z[j] - mean; m2 += d * d; }
    st = stat_merge<OP>(st, Stat{static_cast<float>(EPV), mean, m2});
  } else {
#pragma unroll
    for (int j = 0; j < EPV; ++j) st.a += z[j] * z[j];
  }
}

// Fold a block of four vectors: one running-maximum update and one rescale for the block
// (softmax pair); the normalisations fold the vectors one after the other.
template <int OP, int EPV>
__device__ __forceinline__ void fold_block(Stat& st, const float (&z)[4][EPV], float l2e = kLog2e) {
  if (OpTraits<OP>::kSoftmaxLike) {
    float mv = z[0][0];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int j = 0; j < EPV; ++j) mv = fmaxf(mv, z[u][j]);
    const float mn = fmaxf(st.a, mv);
    const float ms = (mn == kNegInf) ? 0.f : mn;
    float acc[4] = {st.b * exp_diff(st.a, ms, l2e), 0.f, 0.f, 0.f};
    constexpr bool kFused = (EPV == 8);                    // as in fold_vector
    const float nms = -ms * l2e;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int j = 0; j < EPV; ++j)
        acc[u] += kFused ? ex2_approx(fmaf(z[u][j], l2e, nms)) : exp_diff(z[u][j], ms, l2e);
    st.a = mn; st.b = (acc[0] + acc[1]) + (acc[2] + acc[3]);
  } else if (OP == OP_LAYERNORM) {
    // exact two sweeps over the 4 * EPV values of the block, then one merge with the running
    // statistics (a merge per vector cost a division for every EPV values)
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int j = 0; j < EPV; ++j) { s0 += z[0][j]; s1 += z[1][j]; s2 += z[2][j]; s3 += z[3][j]; }
    const float mean = ((s0 + s1) + (s2 + s3)) * (1.0f / (4 * EPV));
    float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
#pragma unroll
    for (int j = 0; j < EPV; ++j) {
      const float d0 = z[0][j] - mean, d1 = z[1][j] - mean, d2 = z[2][j] - mean, d3 = z[3][j] - mean;
      q0 = fmaf(d0, d0, q0); q1 = fmaf(d1, d1, q1); q2 = fmaf(d2, d2, q2); q3 = fmaf(d3, d3, q3);
    }
    st = stat_merge<OP>(st, Stat{static_cast<float>(4 * EPV), mean, (q0 + q1) + (q2 + q3)});
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u) fold_vector<OP, EPV>(st, z[u], l2e);
  }
}

struct SmemGeom {
  int nbuf;               // ring depth
  int slice_vecs;         // 16-byte vectors per CTA slice (last slice may be shorter)
  unsigned buf_bytes;     // bytes reserved per ring buffer (multiple of 128)
};

constexpr int kXSlots = 4;          // exchange slots of smem_kernel (see its comment)

template <int OP, typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 3 : 1)      // 256 threads: three CTAs per SM, 85 registers
smem_kernel(const RowParams p, const SmemGeom g, const int xmode) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int NW = THREADS / 32;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;

  extern __shared__ __align__(128) unsigned char smem_raw[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);                       // [kMaxBuf]
  uint64_t* xbar = bars + kMaxBuf;                                               // [kXSlots]
  float4 (*inbox)[kMaxCluster] =
      reinterpret_cast<float4 (*)[kMaxCluster]>(smem_raw + kMaxBuf * 8 + kXSlots * 8);       // [kXSlots][kMaxCluster]
  Stat* red = reinterpret_cast<Stat*>(smem_raw + kMaxBuf * 8 + kXSlots * 8 + kXSlots * kMaxCluster * 16);   // [2][NW]
  Stat* peers = red + 2 * NW;                                                     // [2][kMaxCluster]
  constexpr unsigned kHeader = smem_header_bytes(THREADS);
  unsigned char* bufs = smem_raw + kHeader;

  const uint32_t cs = cluster_size();
  const uint32_t rank = cluster_rank();
  const long long first_row = cluster_id();
  const long long row_step = cluster_count();
  const int nvec = static_cast<int>(p.cols / EPV);
  const int v0 = static_cast<int>(rank) * g.slice_vecs;                          // my first vector
  const int my_vecs = max(0, min(g.slice_vecs, nvec - v0));

  // Exchange of the slices' partial statistics.
  // xmode 1 (default): as in split_kernel, one 16-byte st.async per peer that counts on the receiver's
  // mbarrier, so that no cluster barrier (whose release waits for the CTA's global stores of the row
  // before) stands between two rows.  xmode 2 also software-pipelines the row loop over a ring of two and
  // more buffers: the first sweep of row r + 1 and the sending of its partials come BEFORE the wait for the
  // partials of row r, whose latency then hides behind that sweep.
  // A CTA can therefore be up to two rows ahead of a peer's reads, hence four exchange slots
  // (row r uses slot r mod 4): a peer sends row r + 4 only after it has received every CTA's partial of
  // row r + 2, and a CTA sends that after it has read the slot of row r.
  // xmode 0: plain remote stores and a cluster barrier per row, no pipelining (the first version).
  const bool async_x = xmode != 0 && cs > 1;
  // (measured: no gain for one CTA per SM - 166 us against 165 us on configuration 4 - and a loss where several
  // CTAs share an SM and hide each other's waits anyway - bf16 log-softmax 16384 columns 0.66 against 0.85 of
  // the copy rate, because the wait for the NEXT row's copy then delays the stores and the refill of the
  // current one; the order is kept for experiments only)
  const bool pipelined = xmode == 2 && g.nbuf >= 2;
  if (threadIdx.x == 0) {
    for (int b = 0; b < g.nbuf; ++b) mbar_init(smem_addr(&bars[b]), 1);
    for (int k = 0; k < kXSlots; ++k) mbar_init(smem_addr(&xbar[k]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (cs > 1) {            // every CTA of the cluster is running before any remote store
    cluster_arrive();
    cluster_wait();
  }

  // number of live vectors of my slice for a given row
  auto live_in_slice = [&](long long row, int& live) -> int {
    live = SM ? static_cast<int>(live_cols(p, row)) : static_cast<int>(p.cols);
    const int live_vecs = (live + EPV - 1) / EPV;
    return max(0, min(my_vecs, live_vecs - v0));
  };
  auto issue = [&](long long row, int b) {
    int live;
    const int lv = live_in_slice(row, live);
    const uint32_t bar = smem_addr(&bars[b]);
    if (lv == 0) {
      // nothing to fetch (slice fully masked): complete the phase so parities stay in step
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
    } else {
      const uint32_t bytes = static_cast<uint32_t>(lv) * 16u;
      mbar_expect_tx(bar, bytes);
      const unsigned char* src = reinterpret_cast<const unsigned char*>(
          reinterpret_cast<const T*>(p.x) + row * p.xs + static_cast<long long>(v0) * EPV);
      const uint32_t dst = smem_addr(bufs + static_cast<size_t>(b) * g.buf_bytes);
      constexpr uint32_t kChunk = 32768;
      for (uint32_t off = 0; off < bytes; off += kChunk)
        bulk_load(dst + off, src + off, min(kChunk, bytes - off), bar);
    }
  };

  int in_flight = 0;                 // thread 0: slices issued and not yet waited for
  if (threadIdx.x == 0 && !p.no_copies) {
    long long r = first_row;
    for (int b = 0; b < g.nbuf && r < p.rows; ++b, r += row_step) { issue(r, b); ++in_flight; }
  }

  // A wait that runs out makes the whole CTA "dead" (the vote in sweep1): it reads and stores nothing any
  // more and issues no copy, but goes on through its rows for the sake of the cluster exchange, so that
  // no peer waits for a CTA that has left.
  bool dead = false, xfail = false;  // xfail: this thread's wait for the cluster's partials ran out
  long long dead_it = 0;             // the iteration whose wait ran out
  uint32_t xphases = 0;              // bit k: parity of the phase of xbar[k] that the next wait is for

  // ---- first sweep of iteration `it` (row `row`): wait for the slice, thread statistics, CTA reduction,
  // and the CTA's partial on its way to the peers
  auto sweep1 = [&](long long row, long long it) -> Stat {
    const int b = static_cast<int>(it % g.nbuf);
    const uint32_t phase = static_cast<uint32_t>((it / g.nbuf) & 1);
    const int par = static_cast<int>(it & 1);
    int live;
    const int lv = live_in_slice(row, live);
    const uint32_t buf = smem_addr(bufs + static_cast<size_t>(b) * g.buf_bytes);
    const T* ar = (SM && p.add != nullptr)
                      ? reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride
                      : nullptr;
    if (!dead) {
      if (__syncthreads_or((xfail || !mbar_wait_timed(smem_addr(&bars[b]), phase, p.status, p.wait_us)) ? 1 : 0)) {
        dead = true;
        dead_it = it;
      } else if (threadIdx.x == 0) {
        --in_flight;
      }
    }
    // `plain` = no element of the slice is masked: four vectors per step, loads first, one rescale per block
    Stat st = stat_identity<OP>();
    const bool plain = !SM || (ar == nullptr && (v0 + lv) * EPV <= live);
    int v = dead ? lv : static_cast<int>(threadIdx.x);          // a dead CTA folds nothing
    if (plain) {
      for (; v + 3 * THREADS < lv; v += 4 * THREADS) {
        float z[4][EPV];
#pragma unroll
        for (int u = 0; u < 4; ++u) E::unpack(lds128(buf + static_cast<uint32_t>(v + u * THREADS) * 16u), z[u]);
        fold_block<OP, EPV>(st, z, p.l2e);
      }
    }
    for (; v < lv; v += THREADS) {
      float z[EPV];
      E::unpack(lds128(buf + static_cast<uint32_t>(v) * 16u), z);
      if (SM) {
        const int c0 = (v0 + v) * EPV;
        if (ar != nullptr) {
          float a[EPV];
          E::unpack(ld_stream(ar + c0), a);
#pragma unroll
          for (int j = 0; j < EPV; ++j) z[j] = fmaf(a[j], p.inv_scale, z[j]);
        }
        if (c0 + EPV > live) {
#pragma unroll
          for (int j = 0; j < EPV; ++j) if (c0 + j >= live) z[j] = kNegInf;
        }
      }
      fold_vector<OP, EPV>(st, z, p.l2e);
    }
    st = cta_reduce<OP, NW>(st, red + par * NW, p.l2e);
    if (async_x) {
      const int slot = static_cast<int>(it % kXSlots);
      if (threadIdx.x == 0) mbar_expect_tx(smem_addr(&xbar[slot]), cs * 16u);
      if (threadIdx.x < cs)
        st_async_f32x4(smem_addr(&inbox[slot][rank]), smem_addr(&xbar[slot]), threadIdx.x, st.a, st.b, st.c, 0.f);
    } else if (cs > 1) {
      if (threadIdx.x < cs) {
        const uint32_t slot = smem_addr(&peers[par * kMaxCluster + rank]);
        st_remote_f32(slot, threadIdx.x, st.a);
        st_remote_f32(slot + 4, threadIdx.x, st.b);
        st_remote_f32(slot + 8, threadIdx.x, st.c);
      }
      cluster_arrive();
    }
    return st;
  };

  // ---- the row's statistics from the cluster, second sweep (normalise from shared memory, 128-bit
  // stores), and the buffer handed back to the copy engine
  auto sweep2 = [&](long long row, long long it, Stat st) {
    const int b = static_cast<int>(it % g.nbuf);
    const int par = static_cast<int>(it & 1);
    int live;
    const int lv = live_in_slice(row, live);
    const uint32_t buf = smem_addr(bufs + static_cast<size_t>(b) * g.buf_bytes);
    const T* ar = (SM && p.add != nullptr)
                      ? reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride
                      : nullptr;
    const bool plain = !SM || (ar == nullptr && (v0 + lv) * EPV <= live);
    if (async_x) {
      const int slot = static_cast<int>(it % kXSlots);
      // (a dead CTA does not wait; a wait that runs out here makes the CTA dead at the vote of its next sweep1)
      if (!dead && !mbar_wait_timed<true>(smem_addr(&xbar[slot]), (xphases >> slot) & 1u, p.status, p.wait_us))
        xfail = true;
      xphases ^= 1u << slot;
      const float4 f = inbox[slot][threadIdx.x & (cs - 1)];          // cs is a power of two
      st = butterfly_merge<OP>(Stat{f.x, f.y, f.z}, static_cast<int>(cs), p.l2e);
    } else if (cs > 1) {
      cluster_wait();
      Stat r = peers[par * kMaxCluster];
      for (uint32_t k = 1; k < cs; ++k) r = stat_merge<OP>(r, peers[par * kMaxCluster + k], p.l2e);
      st = r;
    }
    const RowScalars rs = finalize<OP>(st, p.cols, p.eps);
    const float fill = SM ? masked_fill<OP>(rs) : 0.f;

    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + static_cast<long long>(v0) * EPV;
    int v = (dead || xfail) ? my_vecs : static_cast<int>(threadIdx.x);      // a dead CTA stores nothing
    if (plain && lv == my_vecs) {
      for (; v + 3 * THREADS < my_vecs; v += 4 * THREADS) {
        float z[4][EPV];
#pragma unroll
        for (int u = 0; u < 4; ++u) E::unpack(lds128(buf + static_cast<uint32_t>(v + u * THREADS) * 16u), z[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c0 = (v0 + v + u * THREADS) * EPV;
          float ga[EPV], be[EPV], o[EPV];
#pragma unroll
          for (int j = 0; j < EPV; ++j) { ga[j] = 1.f; be[j] = 0.f; }
          if (!SM) {
            if (p.gamma != nullptr) E::unpack(ld_cached(reinterpret_cast<const T*>(p.gamma) + c0), ga);
            if (OP == OP_LAYERNORM && p.beta != nullptr)
              E::unpack(ld_cached(reinterpret_cast<const T*>(p.beta) + c0), be);
          }
#pragma unroll
          for (int j = 0; j < EPV; ++j) {
            if (OP == OP_SOFTMAX) o[j] = exp_diff(z[u][j], rs.p, p.l2e) * rs.q;
            else o[j] = apply_one<OP>(z[u][j], rs, 0.f, ga[j], be[j], p.scale);
          }
          st_stream(yr + static_cast<long long>(v + u * THREADS) * EPV, E::pack(o));
        }
      }
    }
    for (; v < my_vecs; v += THREADS) {
      float o[EPV];
      if (v < lv) {
        float z[EPV];
        E::unpack(lds128(buf + static_cast<uint32_t>(v) * 16u), z);
        const int c0 = (v0 + v) * EPV;
        float ga[EPV], be[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) { ga[j] = 1.f; be[j] = 0.f; }
        if (SM) {
          if (ar != nullptr) {
            float a[EPV];
            E::unpack(ld_stream(ar + c0), a);
#pragma unroll
            for (int j = 0; j < EPV; ++j) z[j] = fmaf(a[j], p.inv_scale, z[j]);
          }
        } else {
          if (p.gamma != nullptr) E::unpack(ld_cached(reinterpret_cast<const T*>(p.gamma) + c0), ga);
          if (OP == OP_LAYERNORM && p.beta != nullptr)
            E::unpack(ld_cached(reinterpret_cast<const T*>(p.beta) + c0), be);
        }
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
          if (SM && c0 + j >= live) o[j] = fill;
          else if (OP == OP_SOFTMAX) o[j] = exp_diff(z[j], rs.p, p.l2e) * rs.q;
          else o[j] = apply_one<OP>(z[j], rs, 0.f, ga[j], be[j], p.scale);
        }
      } else {
#pragma unroll
        for (int j = 0; j < EPV; ++j) o[j] = fill;
      }
      st_stream(yr + static_cast<long long>(v) * EPV, E::pack(o));
    }

    // the buffer is free once every thread has read it: refill for row it + nbuf
    __syncthreads();
    if (threadIdx.x == 0 && !dead && !p.no_copies) {
      const long long next = row + row_step * g.nbuf;
      if (next < p.rows) { issue(next, b); ++in_flight; }
    }
  };

  long long it = 0;
  if (first_row < p.rows) {
    if (pipelined) {
      Stat st = sweep1(first_row, 0);
      for (long long row = first_row; row < p.rows; row += row_step, ++it) {
        const long long next = row + row_step;
        Stat stn = st;
        if (next < p.rows) stn = sweep1(next, it + 1);      // (its partials are on their way while ...)
        sweep2(row, it, st);                                 // (... this row waits for its own)
        st = stn;
      }
    } else {
      for (long long row = first_row; row < p.rows; row += row_step, ++it) {
        const Stat st = sweep1(row, it);
        sweep2(row, it, st);
      }
    }
  }
  // no copy may still be on its way into this CTA's shared memory when it leaves
  if (threadIdx.x == 0 && dead) {
    for (long long k = dead_it; in_flight > 0; --in_flight, ++k)
      (void)mbar_wait_timed(smem_addr(&bars[k % g.nbuf]), static_cast<uint32_t>((k / g.nbuf) & 1), nullptr, p.wait_us);
  }
  if (cs > 1) {            // nobody leaves while a peer may still send to it
    cluster_arrive();
    cluster_wait();
  }
}

}  // namespace akg
