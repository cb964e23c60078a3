// split_kernel: long rows without shared-memory residency.
//
// A cluster of CS CTAs owns one row at a time and CTA k streams slice k twice:
//   pass 1  128-bit loads, four per thread in flight, marked "keep in L2"
//           -> thread statistics -> CTA reduction -> partial statistics exchanged
//           through distributed shared memory -> cluster barrier
//   pass 2  the same slice again, now served by the 126 MB L2 (the row was read a few
//           microseconds earlier), marked "evict first" -> normalise -> streaming stores
// The two passes of consecutive rows are interleaved (pass 2 of row r with pass 1 of the
// cluster's next row), see split_kernel.
// HBM therefore still sees one read and one write per element, while nothing limits
// the row length and every SM keeps many loads in flight.  Rows are spread over as many
// clusters as fit the GPU, so the rows resident in L2 between the passes are
// (clusters in flight) x (row bytes), far below the L2 size for the shapes this is
// chosen for (the planner checks it).
#pragma once

#include "kernels_smem.cuh"

namespace akg {

__device__ __forceinline__ uint64_t l2_policy_keep() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_normal() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// Back to normal priority for the 128-byte line at p (which a "keep" load marked evict_last).
__device__ __forceinline__ void l2_demote_line(const void* p) {
  asm volatile("applypriority.global.L2::evict_normal [%0], 128;" :: "l"(p) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_drop() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint4 ld_hint(const void* p, uint64_t pol) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol) : "memory");
  return v;
}

// What one CTA needs to know about its slice of one row.
template <typename T> struct SplitRow {
  const T* xr;      // slice start in x
  T* yr;            // slice start in y
  const T* ar;      // slice start in the additive mask, or nullptr
  int live;         // live columns of the row
  int lv;           // live vectors of this slice
  bool plain;       // no mask reaches the slice's live part: vectors fold without a column test
};

template <int OP, typename T>
__device__ __forceinline__ SplitRow<T> split_row(const RowParams& p, long long row, int v0, int my_vecs) {
  constexpr int EPV = Elem<T>::EPV;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  SplitRow<T> r;
  r.live = SM ? static_cast<int>(live_cols(p, row)) : static_cast<int>(p.cols);
  const int live_vecs = (r.live + EPV - 1) / EPV;
  r.lv = max(0, min(my_vecs, live_vecs - v0));
  r.xr = reinterpret_cast<const T*>(p.x) + row * p.xs + static_cast<long long>(v0) * EPV;
  r.yr = reinterpret_cast<T*>(p.y) + row * p.ys + static_cast<long long>(v0) * EPV;
  r.ar = (SM && p.add != nullptr) ? reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride +
                                        static_cast<long long>(v0) * EPV
                                  : nullptr;
  r.plain = !SM || (r.ar == nullptr && (v0 + r.lv) * EPV <= r.live);
  return r;
}

// Pass 1 over the slice's vectors from `v` on (thread-strided): folds into st.
template <int OP, typename T, int THREADS>
__device__ __forceinline__ void split_pass1(const RowParams& p, const SplitRow<T>& r, int v0, int v, Stat& st,
                                            uint64_t keep) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  if (r.plain) {
    const uint4* px = reinterpret_cast<const uint4*>(r.xr) + v;
    for (; v + 7 * THREADS < r.lv; v += 8 * THREADS, px += 8 * THREADS) {   // eight loads in flight
      uint4 raw[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) raw[u] = ld_hint(px + u * THREADS, keep);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float z[4][EPV];
#pragma unroll
        for (int u = 0; u < 4; ++u) E::unpack(raw[4 * h + u], z[u]);
        fold_block<OP, EPV>(st, z, p.l2e);
      }
    }
    for (; v + 3 * THREADS < r.lv; v += 4 * THREADS, px += 4 * THREADS) {
      uint4 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) raw[u] = ld_hint(px + u * THREADS, keep);
      float z[4][EPV];
#pragma unroll
      for (int u = 0; u < 4; ++u) E::unpack(raw[u], z[u]);
      fold_block<OP, EPV>(st, z, p.l2e);
    }
    if (v < r.lv) {                     // the ragged last step: up to three loads, in flight together
      uint4 raw[3];
#pragma unroll
      for (int u = 0; u < 3; ++u)
        if (v + u * THREADS < r.lv) raw[u] = ld_hint(px + u * THREADS, keep);
#pragma unroll
      for (int u = 0; u < 3; ++u)
        if (v + u * THREADS < r.lv) {
          float z[EPV];
          E::unpack(raw[u], z);
          fold_vector<OP, EPV>(st, z, p.l2e);
        }
    }
    return;
  }
  for (; v < r.lv; v += THREADS) {
    float z[EPV];
    E::unpack(ld_hint(r.xr + static_cast<long long>(v) * EPV, keep), z);
    if (SM) {
      const int c0 = (v0 + v) * EPV;
      if (r.ar != nullptr) {
        float a[EPV];
        E::unpack(ld_hint(r.ar + static_cast<long long>(v) * EPV, keep), a);
#pragma unroll
        for (int j = 0; j < EPV; ++j) z[j] = fmaf(a[j], p.inv_scale, z[j]);
      }
      if (c0 + EPV > r.live) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) if (c0 + j >= r.live) z[j] = kNegInf;
      }
    }
    fold_vector<OP, EPV>(st, z, p.l2e);
  }
}

// One output vector of a slice that no mask reaches.
template <int OP, typename T>
__device__ __forceinline__ uint4 split_apply_plain(const RowParams& p, const RowScalars& rs, const uint4 raw, int c0) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  if constexpr (!SM && sizeof(T) == 2) {
    // 16-bit normalisations with every affine vector present (the usual call): the stored values go
    // into the arithmetic as they are (see Elem::fma_wide), only gamma is unpacked for LayerNorm
    //   RMSNorm   (x * w) * rstd            the product of two 16-bit values is exact in fp32
    //   LayerNorm beta + ((x - mean) * rstd) * gamma
    if (p.gamma != nullptr && (OP != OP_LAYERNORM || p.beta != nullptr)) {
      const uint4 gw = ld_cached(reinterpret_cast<const T*>(p.gamma) + c0);
      const uint32_t xs[4] = {raw.x, raw.y, raw.z, raw.w}, gs[4] = {gw.x, gw.y, gw.z, gw.w};
      uint32_t out[4];
      if constexpr (OP == OP_RMSNORM) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short x0, x1, g0, g1;
          halves(xs[i], x0, x1);
          halves(gs[i], g0, g1);
          out[i] = E::pack2(E::fma_wide(x0, g0, 0.f) * rs.q, E::fma_wide(x1, g1, 0.f) * rs.q);
        }
      } else {
        const uint4 bw = ld_cached(reinterpret_cast<const T*>(p.beta) + c0);
        const uint32_t bs[4] = {bw.x, bw.y, bw.z, bw.w};
        float ga[EPV];
        E::unpack(gw, ga);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short x0, x1, b0, b1;
          halves(xs[i], x0, x1);
          halves(bs[i], b0, b1);
          out[i] = E::pack2(E::add_wide(b0, E::sub_wide(x0, rs.p) * rs.q * ga[2 * i]),
                            E::add_wide(b1, E::sub_wide(x1, rs.p) * rs.q * ga[2 * i + 1]));
        }
      }
      return make_uint4(out[0], out[1], out[2], out[3]);
    }
  }
  if constexpr (OP == OP_RMSNORM && sizeof(T) == 4) {
    // fp32 RMSNorm with its weight present: no defaults to set up and overwrite (the generic form below spends
    // about two instructions per element on them; 65536 columns 0.93 -> 0.96 of the copy rate).  The same
    // shortcut made fp32 LayerNorm slower (0.82 -> 0.72: its gamma and beta loads then sit between the streaming
    // stores, which the compiler may not move them across), so LayerNorm keeps the generic form.
    if (p.gamma != nullptr) {
      const uint4 gw = ld_cached(reinterpret_cast<const T*>(p.gamma) + c0);
      return make_uint4(__float_as_uint(__uint_as_float(raw.x) * rs.q * __uint_as_float(gw.x)),
                        __float_as_uint(__uint_as_float(raw.y) * rs.q * __uint_as_float(gw.y)),
                        __float_as_uint(__uint_as_float(raw.z) * rs.q * __uint_as_float(gw.z)),
                        __float_as_uint(__uint_as_float(raw.w) * rs.q * __uint_as_float(gw.w)));
    }
  }
  float z[EPV], ga[EPV], be[EPV], o[EPV];
  E::unpack(raw, z);
#pragma unroll
  for (int j = 0; j < EPV; ++j) { ga[j] = 1.f; be[j] = 0.f; }
  if (!SM) {
    if (p.gamma != nullptr) E::unpack(ld_cached(reinterpret_cast<const T*>(p.gamma) + c0), ga);
    if (OP == OP_LAYERNORM && p.beta != nullptr) E::unpack(ld_cached(reinterpret_cast<const T*>(p.beta) + c0), be);
  }
  constexpr bool kFused = (sizeof(T) == 2);               // 16-bit storage: exponent as one multiply-add
  const float nml = -rs.p * p.l2e;
#pragma unroll
  for (int j = 0; j < EPV; ++j) {
    if (OP == OP_SOFTMAX) o[j] = (kFused ? ex2_approx(fmaf(z[j], p.l2e, nml)) : exp_diff(z[j], rs.p, p.l2e)) * rs.q;
    else o[j] = apply_one<OP>(z[j], rs, 0.f, ga[j], be[j], p.scale);
  }
  return E::pack(o);
}

// Pass 2 over the slice's vectors from `v` on: second read (L2), normalise, store.
template <int OP, typename T, int THREADS>
__device__ __forceinline__ void split_pass2(const RowParams& p, const SplitRow<T>& r, const RowScalars& rs, int v0,
                                            int my_vecs, int v, uint64_t drop) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  const float fill = SM ? masked_fill<OP>(rs) : 0.f;
  if (r.plain && r.lv == my_vecs) {
    const uint4* px = reinterpret_cast<const uint4*>(r.xr) + v;
    uint4* py = reinterpret_cast<uint4*>(r.yr) + v;
    for (; v + 3 * THREADS < my_vecs; v += 4 * THREADS, px += 4 * THREADS, py += 4 * THREADS) {
      uint4 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) raw[u] = ld_hint(px + u * THREADS, drop);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        st_stream(py + u * THREADS, split_apply_plain<OP, T>(p, rs, raw[u], (v0 + v + u * THREADS) * EPV));
    }
    if (v < my_vecs) {                  // the ragged last step
      uint4 raw[3];
#pragma unroll
      for (int u = 0; u < 3; ++u)
        if (v + u * THREADS < my_vecs) raw[u] = ld_hint(px + u * THREADS, drop);
#pragma unroll
      for (int u = 0; u < 3; ++u)
        if (v + u * THREADS < my_vecs)
          st_stream(py + u * THREADS, split_apply_plain<OP, T>(p, rs, raw[u], (v0 + v + u * THREADS) * EPV));
    }
    return;
  }
  for (; v < my_vecs; v += THREADS) {
    float o[EPV];
    if (v < r.lv) {
      float z[EPV];
      E::unpack(ld_hint(r.xr + static_cast<long long>(v) * EPV, drop), z);
      const int c0 = (v0 + v) * EPV;
      float ga[EPV], be[EPV];
#pragma unroll
      for (int j = 0; j < EPV; ++j) { ga[j] = 1.f; be[j] = 0.f; }
      if (SM) {
        if (r.ar != nullptr) {
          float a[EPV];
          E::unpack(ld_hint(r.ar + static_cast<long long>(v) * EPV, drop), a);
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
        if (SM && c0 + j >= r.live) o[j] = fill;
        else if (OP == OP_SOFTMAX) o[j] = exp_diff(z[j], rs.p, p.l2e) * rs.q;
        else o[j] = apply_one<OP>(z[j], rs, 0.f, ga[j], be[j], p.scale);
      }
    } else {
#pragma unroll
      for (int j = 0; j < EPV; ++j) o[j] = fill;
    }
    st_stream(r.yr + static_cast<long long>(v) * EPV, E::pack(o));
  }
}


// LayerNorm with 16-bit storage folds the next row in ONE sweep: every thread accumulates
// s1 = sum(x - K) and s2 = sum((x - K)^2) about a shift K of its own, the first element it owns in
// the slice, and turns them into (count, mean, M2) once per row.  K being one of the thread's values,
// (mean_t - K)^2 <= M2_t, hence s2 <= (n_t + 1) M2_t and the cancellation in M2_t = s2 - s1^2 / n_t
// costs at most a relative (n_t + 1) 2^-24 (n_t is a few hundred: 1e-5), far inside the 2^-9 of a
// 16-bit result; fp32 storage keeps the exact two sweeps per block of four vectors.  What is saved
// is registers: the two sweeps hold 32 widened values at once and spilled 280 bytes.
template <int OP, typename T> constexpr bool kShiftedStats = (OP == OP_LAYERNORM && sizeof(T) == 2);

// (K, s1, s2) over n values -> (count, mean, M2)
__device__ __forceinline__ Stat shifted_finish(const Stat& acc, int n) {
  if (n <= 0) return Stat{0.f, 0.f, 0.f};
  const float inv = 1.0f / static_cast<float>(n);
  const float m = acc.b * inv;
  return Stat{static_cast<float>(n), acc.a + m, fmaxf(acc.c - acc.b * m, 0.f)};
}

// One unrolled step of the merged loop on vectors v, v + THREADS, ... (four per thread) of two
// unmasked rows: the loads of the cluster's next row (xn: HBM, "keep") and of the current row (xc:
// L2, "drop") are issued by split_step_load; split_step_use normalises and stores the current row
// and folds the next one.  PRED: the step is the slice's last, ragged one, and vector u takes part
// only if v + u * THREADS < my_vecs.
template <int THREADS, bool PRED>
__device__ __forceinline__ void split_step_load(const uint4* xn, const uint4* xc, int v, int my_vecs, uint64_t keep,
                                                uint64_t drop, uint4 (&rn)[4], uint4 (&rc)[4]) {
#pragma unroll
  for (int u = 0; u < 4; ++u)
    if (!PRED || v + u * THREADS < my_vecs) rn[u] = ld_hint(xn + v + u * THREADS, keep);
#pragma unroll
  for (int u = 0; u < 4; ++u)
    if (!PRED || v + u * THREADS < my_vecs) rc[u] = ld_hint(xc + v + u * THREADS, drop);
}

template <int OP, typename T, int THREADS, bool PRED>
__device__ __forceinline__ void split_step_use(const RowParams& p, uint4* yc, const RowScalars& rs, int v0, int v,
                                               int my_vecs, const uint4 (&rn)[4], const uint4 (&rc)[4], Stat& stn,
                                               const uint4* demote = nullptr) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  if (!PRED && demote != nullptr && (threadIdx.x & 7) == 0) {
#pragma unroll
    for (int u = 0; u < 4; ++u) l2_demote_line(demote + v + u * THREADS);
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
    if (!PRED || v + u * THREADS < my_vecs)
      st_stream(yc + v + u * THREADS, split_apply_plain<OP, T>(p, rs, rc[u], (v0 + v + u * THREADS) * EPV));
  if constexpr (kShiftedStats<OP, T>) {
    // 16-bit LayerNorm: one sweep of sums about the thread's shift stn.a (see shifted_finish); the
    // stored values enter the subtraction as they are (Elem::sub_wide)
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (!PRED || v + u * THREADS < my_vecs) {
        const uint32_t ws[4] = {rn[u].x, rn[u].y, rn[u].z, rn[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(ws[i], h0, h1);
          const float d0 = E::sub_wide(h0, stn.a), d1 = E::sub_wide(h1, stn.a);
          stn.b += d0 + d1;
          stn.c = fmaf(d1, d1, fmaf(d0, d0, stn.c));
        }
      }
  } else if constexpr (OP == OP_RMSNORM && sizeof(T) == 2) {
    // 16-bit RMSNorm: x * x + acc in one instruction per element (Elem::fma_wide), two chains
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (!PRED || v + u * THREADS < my_vecs) {
        const uint32_t ws[4] = {rn[u].x, rn[u].y, rn[u].z, rn[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(ws[i], h0, h1);
          s0 = E::fma_wide(h0, h0, s0);
          s1 = E::fma_wide(h1, h1, s1);
        }
      }
    stn.a += s0 + s1;
  } else if (!PRED) {
    float z[4][EPV];
#pragma unroll
    for (int u = 0; u < 4; ++u) E::unpack(rn[u], z[u]);
    fold_block<OP, EPV>(stn, z, p.l2e);
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (v + u * THREADS < my_vecs) {
        float z[EPV];
        E::unpack(rn[u], z);
        fold_vector<OP, EPV>(stn, z, p.l2e);
      }
  }
}

// The row loop is software-pipelined: while a CTA writes row r (pass 2: L2 reads, HBM
// writes) it already folds its slice of the cluster's next row (pass 1: HBM reads), four
// vectors of each per thread and step, so that every warp keeps DRAM reads and writes in
// flight at once and a row costs one trip through the slice instead of two.
//
// Exchange of the slices' partial statistics (xmode 1, the default): every CTA owns two
// mbarriers (rows alternate between them).  After the CTA reduction, thread k < CS sends the
// CTA's partial to CTA k with one 16-byte st.async, which lands in slot [parity][sender] of the
// receiver's shared memory and counts 16 bytes on the receiver's mbarrier; a CTA waits on its
// own mbarrier for CS x 16 bytes.  Nothing waits for the CTA's global stores (a cluster barrier's
// release does: the profile showed it as membar stalls), and the first loads of the next step
// are already in flight while a thread waits for the partials.  Reuse of a slot and of a phase
// two rows later is ordered by the exchange itself: a peer can send row r + 2 only after it has
// received this CTA's partial of row r + 1, which this CTA sends after all its threads have read
// the slots of row r (the CTA reduction's barrier lies in between).
// xmode 0 keeps the first version: plain remote stores and a cluster barrier per row.
//
// L2 priorities (l2mode 0, the default): pass 1 loads mark their lines "evict last", pass 2 loads
// "evict first", and pass 2 also puts each 128-byte line it has consumed back to normal priority
// (applypriority): in a run of back-to-back calls the lines marked by earlier calls otherwise stay
// privileged and take the room of the rows in flight (config 4: 97.3 us without, 95.3 us with the
// demotion).  l2mode 1: pass 1 with normal priority (97.4 us); l2mode 2: marks, no demotion.
//
// Waits are bounded (two seconds of the global timer).  A CTA whose wait runs out sets the status
// word, stops storing and leaves the row loop; its peers run into the same limit one after the
// other.  All CTAs of a cluster meet at a cluster barrier before they exit, so no partial is ever
// sent to a CTA that has left.
#ifndef AKG_SPLIT_MINB16
#define AKG_SPLIT_MINB16 4
#endif
template <typename T, int THREADS> constexpr int kSplitMinBlocks =
    (sizeof(T) == 2 && THREADS == 256) ? AKG_SPLIT_MINB16 : ((1024 / THREADS) > 0 ? (1024 / THREADS) : 1);

template <int OP, typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, kSplitMinBlocks<T, THREADS>)
split_kernel(const RowParams p, const int slice_vecs, const int xmode, const int l2mode) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int NW = THREADS / 32;
  __shared__ Stat red[2][NW];
  __shared__ Stat peers[2][kMaxCluster];
  __shared__ __align__(16) float4 inbox[2][kMaxCluster];
  __shared__ __align__(8) uint64_t xbar[2];

  const uint32_t cs = cluster_size();
  const uint32_t rank = cluster_rank();
  const long long row_step = cluster_count();
  const int nvec = static_cast<int>(p.cols / EPV);
  const int v0 = static_cast<int>(rank) * slice_vecs;
  const int my_vecs = max(0, min(slice_vecs, nvec - v0));
  const uint64_t keep = (l2mode == 1) ? l2_policy_normal() : l2_policy_keep();   // see split_kernel's comment
  const uint64_t drop = l2_policy_drop();
  const bool async_x = (xmode != 0) && cs > 1;

  if (cs > 1) {            // every CTA of the cluster is running (mbarriers set up) before any remote store
    if (threadIdx.x == 0) {
      mbar_init(smem_addr(&xbar[0]), 1);
      mbar_init(smem_addr(&xbar[1]), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_arrive();
    cluster_wait();
  }

  int par = 0;
  uint32_t phases = 0;        // bit k: parity of the phase of xbar[k] that the next wait is for
  // A thread whose wait ran out has mv = -1 vectors to work on from then on (mv is my_vecs otherwise): it
  // loads and stores nothing, waits for nothing, and still passes every barrier and sends its CTA's
  // partials, so that neither its CTA nor its cluster waits for it.  The flag in shared memory takes the
  // rest of the CTA along at the next row.
  __shared__ int cta_failed;
  if (threadIdx.x == 0) cta_failed = 0;
  int mv = my_vecs;
  auto give_up_with_the_cta = [&]() {
    if (*reinterpret_cast<volatile int*>(&cta_failed)) mv = -1;
  };
  // thread statistics of a slice -> this CTA's partial, sent to every CTA of the cluster
  auto send_stats = [&](Stat st) -> Stat {
    st = cta_reduce<OP, NW>(st, red[par], p.l2e);
    if (async_x) {
      if (threadIdx.x == 0) mbar_expect_tx(smem_addr(&xbar[par]), cs * 16u);
      if (threadIdx.x < cs)
        st_async_f32x4(smem_addr(&inbox[par][rank]), smem_addr(&xbar[par]), threadIdx.x, st.a, st.b, st.c, 0.f);
    } else if (cs > 1) {
      if (threadIdx.x < cs) {
        const uint32_t slot = smem_addr(&peers[par][rank]);
        st_remote_f32(slot, threadIdx.x, st.a);
        st_remote_f32(slot + 4, threadIdx.x, st.b);
        st_remote_f32(slot + 8, threadIdx.x, st.c);
      }
      cluster_arrive();
    }
    return st;
  };
  // ... and the statistics of the whole row, in every CTA of the cluster
  auto recv_stats = [&](Stat st) -> Stat {
    if (async_x) {
      if (mv >= 0 && !mbar_wait_timed<true>(smem_addr(&xbar[par]), (phases >> par) & 1u, p.status, p.wait_us)) {
        mv = -1;
        cta_failed = 1;
      }
      phases ^= 1u << par;
      const float4 f = inbox[par][threadIdx.x & (cs - 1)];           // cs is a power of two
      st = butterfly_merge<OP>(Stat{f.x, f.y, f.z}, static_cast<int>(cs), p.l2e);
    } else if (cs > 1) {
      cluster_wait();
      Stat r = peers[par][0];
      for (uint32_t k = 1; k < cs; ++k) r = stat_merge<OP>(r, peers[par][k], p.l2e);
      st = r;
    }
    par ^= 1;
    return st;
  };

  long long row = cluster_id();
  constexpr bool SM = OpTraits<OP>::kSoftmaxLike;
  constexpr bool kEarlyReread = sizeof(T) == 4 || !SM;
  if (row < p.rows && (!SM || (p.add == nullptr && !p.causal))) {
    // ---- no mask anywhere: every slice is whole, and a row's pointers follow from the previous row's
    const long long dx = row_step * p.xs * static_cast<long long>(sizeof(T)) / 16;   // in vectors
    const long long dy = row_step * p.ys * static_cast<long long>(sizeof(T)) / 16;
    const uint4* xc = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p.x) + row * p.xs) + v0;
    uint4* yc = reinterpret_cast<uint4*>(reinterpret_cast<T*>(p.y) + row * p.ys) + v0;
    Stat st = stat_identity<OP>();
    {
      SplitRow<T> first;
      first.xr = reinterpret_cast<const T*>(xc); first.yr = reinterpret_cast<T*>(yc); first.ar = nullptr;
      first.live = static_cast<int>(p.cols); first.lv = mv; first.plain = true;
      split_pass1<OP, T, THREADS>(p, first, v0, threadIdx.x, st, keep);
    }
    st = send_stats(st);
    for (;; row += row_step, xc += dx, yc += dy) {
      give_up_with_the_cta();
      const bool has_next = row + row_step < p.rows;
      const uint4* xn = xc + dx;
      int v = threadIdx.x;
      uint4 rn[4], rc[4];
      const bool first_full = has_next && v + 3 * THREADS < mv;
      if (first_full) {                              // in flight while this thread waits for the partials
#pragma unroll
        for (int u = 0; u < 4; ++u) rn[u] = ld_hint(xn + v + u * THREADS, keep);
        // ... and so are the first re-reads of the current row, which need no statistics to be issued
        // (65536 fp32 columns: softmax 0.87 -> 0.94, LayerNorm 0.79 -> 0.82 of the copy rate; the 16-bit
        // softmax pair has no registers for them: 170 bytes of spills and 2 - 3 % slower)
        if constexpr (kEarlyReread) {
#pragma unroll
          for (int u = 0; u < 4; ++u) rc[u] = ld_hint(xc + v + u * THREADS, drop);
        }
      }
      st = recv_stats(st);
      const RowScalars rs = finalize<OP>(st, p.cols, p.eps);
      if (!has_next) {
        SplitRow<T> last;
        last.xr = reinterpret_cast<const T*>(xc); last.yr = reinterpret_cast<T*>(yc); last.ar = nullptr;
        last.live = static_cast<int>(p.cols); last.lv = mv; last.plain = true;
        split_pass2<OP, T, THREADS>(p, last, rs, v0, mv, v, drop);
        break;
      }
      Stat stn = stat_identity<OP>();
      if (kShiftedStats<OP, T> && v < mv)       // the shift: the first element this thread owns
        stn.a = Elem<T>::load1(xn + v, 0);
      if (first_full && mv >= 0) {
        if constexpr (!kEarlyReread) {
#pragma unroll
          for (int u = 0; u < 4; ++u) rc[u] = ld_hint(xc + v + u * THREADS, drop);
        }
        const uint4* demote = (l2mode == 0 && ((reinterpret_cast<uintptr_t>(xc) & 127u) == 0)) ? xc : nullptr;
        split_step_use<OP, T, THREADS, false>(p, yc, rs, v0, v, mv, rn, rc, stn, demote);
        v += 4 * THREADS;
        for (; v + 3 * THREADS < mv; v += 4 * THREADS) {
          split_step_load<THREADS, false>(xn, xc, v, mv, keep, drop, rn, rc);
          split_step_use<OP, T, THREADS, false>(p, yc, rs, v0, v, mv, rn, rc, stn, demote);
        }
      }
      if (v < mv) {                             // the ragged last step: its loads in flight together
        split_step_load<THREADS, true>(xn, xc, v, mv, keep, drop, rn, rc);
        split_step_use<OP, T, THREADS, true>(p, yc, rs, v0, v, mv, rn, rc, stn);
      }
      if (kShiftedStats<OP, T>) {
        const int t = static_cast<int>(threadIdx.x);
        stn = shifted_finish(stn, t < mv ? ((mv - 1 - t) / THREADS + 1) * Elem<T>::EPV : 0);
      }
      st = send_stats(stn);
    }
  } else if (row < p.rows) {
    // ---- masked rows: slices may be cut short by the causal rule or carry an additive mask
    SplitRow<T> cur = split_row<OP, T>(p, row, v0, mv);
    Stat st = stat_identity<OP>();
    split_pass1<OP, T, THREADS>(p, cur, v0, threadIdx.x, st, keep);
    st = send_stats(st);
    for (;;) {
      give_up_with_the_cta();
      st = recv_stats(st);
      if (mv < 0) { cur.lv = 0; cur.plain = false; }
      const RowScalars rs = finalize<OP>(st, p.cols, p.eps);
      const long long next_row = row + row_step;
      if (next_row >= p.rows) {
        split_pass2<OP, T, THREADS>(p, cur, rs, v0, mv, threadIdx.x, drop);
        break;
      }
      const SplitRow<T> nxt = split_row<OP, T>(p, next_row, v0, mv);
      Stat stn = stat_identity<OP>();
      split_pass2<OP, T, THREADS>(p, cur, rs, v0, mv, threadIdx.x, drop);
      split_pass1<OP, T, THREADS>(p, nxt, v0, threadIdx.x, stn, keep);
      st = send_stats(stn);
      cur = nxt;
      row = next_row;
    }
  }
  if (cs > 1) {            // nobody leaves while a peer may still send to it
    cluster_arrive();
    cluster_wait();
  }
}


}  // namespace akg
