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


// The row loop is software-pipelined: while a CTA writes row r (pass 2: L2 reads, HBM
// writes) it already folds its slice of the cluster's next row (pass 1: HBM reads), four
// vectors of each per thread and step, so that every warp keeps DRAM reads and writes in
// flight at once and a row costs one trip through the slice instead of two.
template <int OP, typename T, int THREADS>
__global__ void __launch_bounds__(THREADS, (1024 / THREADS) > 0 ? (1024 / THREADS) : 1)
split_kernel(const RowParams p, const int slice_vecs) {
  pdl_prologue();
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int NW = THREADS / 32;
  __shared__ Stat red[2][NW];
  __shared__ Stat peers[2][kMaxCluster];

  const uint32_t cs = cluster_size();
  const uint32_t rank = cluster_rank();
  const long long row_step = cluster_count();
  const int nvec = static_cast<int>(p.cols / EPV);
  const int v0 = static_cast<int>(rank) * slice_vecs;
  const int my_vecs = max(0, min(slice_vecs, nvec - v0));
  const uint64_t keep = l2_policy_keep();
  const uint64_t drop = l2_policy_drop();

  if (cs > 1) {            // every CTA of the cluster is running before any remote store
    cluster_arrive();
    cluster_wait();
  }

  int par = 0;
  // thread statistics of a slice -> statistics of the whole row, in every CTA of the cluster
  auto row_stats = [&](Stat st) -> Stat {
    st = cta_reduce<OP, NW>(st, red[par], p.l2e);
    if (cs > 1) {
      if (threadIdx.x < cs) {
        const uint32_t slot = smem_addr(&peers[par][rank]);
        st_remote_f32(slot, threadIdx.x, st.a);
        st_remote_f32(slot + 4, threadIdx.x, st.b);
        st_remote_f32(slot + 8, threadIdx.x, st.c);
      }
      cluster_arrive();
      cluster_wait();
      Stat r = peers[par][0];
      for (uint32_t k = 1; k < cs; ++k) r = stat_merge<OP>(r, peers[par][k], p.l2e);
      st = r;
    }
    par ^= 1;
    return st;
  };

  long long row = cluster_id();
  if (row >= p.rows) return;
  SplitRow<T> cur = split_row<OP, T>(p, row, v0, my_vecs);
  Stat st = stat_identity<OP>();
  split_pass1<OP, T, THREADS>(p, cur, v0, threadIdx.x, st, keep);
  st = row_stats(st);

  for (;;) {
    const RowScalars rs = finalize<OP>(st, p.cols, p.eps);
    const long long next_row = row + row_step;
    const bool has_next = next_row < p.rows;
    int v = threadIdx.x;
    if (!has_next) {
      split_pass2<OP, T, THREADS>(p, cur, rs, v0, my_vecs, v, drop);
      break;
    }
    const SplitRow<T> nxt = split_row<OP, T>(p, next_row, v0, my_vecs);
    Stat stn = stat_identity<OP>();
    if (cur.plain && nxt.plain && cur.lv == my_vecs && nxt.lv == my_vecs) {
      const uint4* pn = reinterpret_cast<const uint4*>(nxt.xr) + v;
      const uint4* px = reinterpret_cast<const uint4*>(cur.xr) + v;
      uint4* py = reinterpret_cast<uint4*>(cur.yr) + v;
      for (; v + 3 * THREADS < my_vecs; v += 4 * THREADS, pn += 4 * THREADS, px += 4 * THREADS, py += 4 * THREADS) {
        uint4 rn[4], rc[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) rn[u] = ld_hint(pn + u * THREADS, keep);
#pragma unroll
        for (int u = 0; u < 4; ++u) rc[u] = ld_hint(px + u * THREADS, drop);
#pragma unroll
        for (int u = 0; u < 4; ++u)
          st_stream(py + u * THREADS, split_apply_plain<OP, T>(p, rs, rc[u], (v0 + v + u * THREADS) * EPV));
        float z[4][EPV];
#pragma unroll
        for (int u = 0; u < 4; ++u) E::unpack(rn[u], z[u]);
        fold_block<OP, EPV>(stn, z, p.l2e);
      }
    }
    // whatever the merged loop left (all of both passes when it did not run)
    split_pass2<OP, T, THREADS>(p, cur, rs, v0, my_vecs, v, drop);
    split_pass1<OP, T, THREADS>(p, nxt, v0, v, stn, keep);
    st = row_stats(stn);
    cur = nxt;
    row = next_row;
  }
}

}  // namespace akg
