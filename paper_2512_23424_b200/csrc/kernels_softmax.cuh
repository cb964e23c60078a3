// reg_softmax: register-resident softmax / log-softmax for rows that fit one warp or
// one CTA, with optional additive and causal masks.
//
// A group of G threads owns a row (a warp, or the whole CTA; the row body also supports
// aligned sub-groups with named barriers); thread t of the group owns vectors t, t + G, ...
// With a causal mask only the first NK = ceil(live_vecs / G) of those iterations hold
// live data; the row body is compiled once per NK and selected by a group-uniform switch,
// so masked iterations cost nothing but their fill stores (no predicated-off work).
// The exponential is evaluated once per live element, against the warp maximum; the
// cross-warp combine costs one exponential per warp.
//
#pragma once

#include "kernels_reg.cuh"

namespace akg {

// Barrier over the G threads of one row group (the whole CTA, or an aligned subset).
template <int G, int THREADS> __device__ __forceinline__ void group_barrier(int group) {
  if (G == THREADS) __syncthreads();
  else asm volatile("bar.sync %0, %1;" :: "r"(group + 1), "r"(G) : "memory");
}

// One row.  G threads per row, VPT live iterations at most, KFILL >= VPT store iterations
// (KFILL * G vectors cover the row), NK live iterations for this row.
// RING = false: the row is read from global memory; RING = true: from the shared-memory
// buffer at `ring_buf` that a bulk copy has filled with the row's live prefix.
// red: [2][THREADS / 32] floats, indexed by the warp's position in the CTA.
// PREF = true: the caller already holds this row's vectors in `pre` (loaded while the row
// before it was computed); once they are unpacked the body loads the live vectors of the
// caller's next row (`next_xr`, `next_live_vecs`) into `pre`, so that their latency is
// covered by this row's arithmetic, barrier and stores.
template <int OP, typename T, int G, int VPT, int KFILL, int THREADS, int NK, bool RING = false, bool PREF = false>
__device__ __forceinline__ void softmax_row(const RowParams& p, long long row, int tg, int nvec, int live,
                                            int live_vecs, float (*red)[THREADS / 32], uint32_t ring_buf = 0,
                                            uint4* pre = nullptr, const T* next_xr = nullptr,
                                            int next_live_vecs = 0) {
  using E = Elem<T>;
  constexpr int EPV = E::EPV;
  constexpr int NW = G / 32;
  constexpr int NKA = NK > 0 ? NK : 1;
  static_assert(NW >= 1 && (NW & (NW - 1)) == 0, "warps per row must be a power of two");
  static_assert(NK <= VPT && VPT <= KFILL, "live iterations fit the register tile");
  const bool ragged = live_vecs * EPV != live;
  const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + tg * EPV;
  T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + tg * EPV;
  // only the last live iteration can hold vectors beyond the live prefix
  const bool last_ok = (NK > 0) && (tg + (NK - 1) * G < live_vecs);

  uint4 raw[NKA];
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    if constexpr (PREF) raw[k] = pre[k];
    else if (k < NK - 1 || last_ok)
      raw[k] = RING ? lds128(ring_buf + static_cast<uint32_t>(tg + k * G) * 16u) : ld_stream(xr + k * G * EPV);
  }
  float v[NKA][EPV];
  float m_t = kNegInf;
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    if (k < NK - 1 || last_ok) {
      E::unpack(raw[k], v[k]);
      if (p.add != nullptr) {
        const T* ar = reinterpret_cast<const T*>(p.add) + add_row(p, row) * p.add_stride + tg * EPV;
        float a[EPV];
        E::unpack(ld_stream(ar + k * G * EPV), a);
#pragma unroll
        for (int j = 0; j < EPV; ++j) v[k][j] = fmaf(a[j], p.inv_scale, v[k][j]);
      }
      if (k == NK - 1 && ragged && tg + k * G == live_vecs - 1) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) if ((tg + k * G) * EPV + j >= live) v[k][j] = kNegInf;
      }
    } else {
#pragma unroll
      for (int j = 0; j < EPV; ++j) v[k][j] = kNegInf;
    }
#pragma unroll
    for (int j = 0; j < EPV; ++j) m_t = fmaxf(m_t, v[k][j]);
  }
  if constexpr (PREF) {
#pragma unroll
    for (int k = 0; k < VPT; ++k)
      if (tg + k * G < next_live_vecs) pre[k] = ld_stream(next_xr + k * G * EPV);
  }

  const float m_w = warp_max(m_t);
  const float m_ws = (m_w == kNegInf) ? 0.f : m_w;        // keeps -inf - -inf out of the exponent
  float s_t = 0.f;
  // bf16 storage: one fused multiply-add forms the exponent (its rounding, below 1e-5
  // relative, is far inside the 2^-9 of the bf16 result); fp32 keeps the exact difference
  constexpr bool kFusedExponent = (sizeof(T) == 2);
  const float l2e = p.l2e;                                  // scale * log2(e): the pre-scale costs nothing
  const float neg_m_l2 = -m_ws * l2e;
#pragma unroll
  for (int k = 0; k < NK; ++k) {
#pragma unroll
    for (int j = 0; j < EPV; ++j) {
      const float e = kFusedExponent ? ex2_approx(fmaf(v[k][j], l2e, neg_m_l2)) : exp_diff(v[k][j], m_ws, l2e);
      s_t += e;
      if (OP == OP_SOFTMAX) v[k][j] = e;
    }
  }
  const float s_w = warp_sum(s_t);

  float M = m_w, S = s_w, my_factor = 1.f;
  if (NW > 1) {
    const int warp_cta = threadIdx.x >> 5;
    const int wbase = warp_cta & ~(NW - 1);                // first warp of this row's group
    if ((threadIdx.x & 31) == 0) { red[0][warp_cta] = m_w; red[1][warp_cta] = s_w; }
    group_barrier<G, THREADS>(warp_cta / NW);
    // lane l takes the pair of the group's warp (l mod NW); xor-butterflies over NW lanes
    // give every lane the row maximum and the rescaled sum
    const float mw = red[0][wbase + (threadIdx.x & (NW - 1))];
    const float sw = red[1][wbase + (threadIdx.x & (NW - 1))];
    M = mw;
#pragma unroll
    for (int m = 1; m < NW && m < 32; m <<= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, m));
    const float Ms = (M == kNegInf) ? 0.f : M;
    S = sw * ((mw == M) ? 1.f : exp_diff(mw, Ms, l2e));          // equal maxima (also +-inf): factor 1
#pragma unroll
    for (int m = 1; m < NW && m < 32; m <<= 1) S += __shfl_xor_sync(0xffffffffu, S, m);
    my_factor = (m_w == M) ? 1.f : exp_diff(m_w, Ms, l2e);
  }

  const bool dead = (M == kNegInf) && !(S != S);   // only NaN / -inf entries: a NaN row, not a dead one
  const float nan = __int_as_float(0x7fc00000);
  float scale = 0.f, lse_l = 0.f, fill;
  if (OP == OP_SOFTMAX) {
    scale = dead ? 0.f : my_factor * __frcp_rn(S);
    fill = (S != S) ? nan : 0.f;
  } else {
    lse_l = logf(S);
    fill = (S != S) ? nan : kNegInf;
  }
  // 16-bit log-softmax: scale x - (scale M + ln S) as one fused multiply-add per element (the
  // rounding of the bracket, 2^-24 of its magnitude, is inside the cancellation allowance of a
  // 16-bit result); fp32 keeps the exact difference x - M
  // a dead row (every entry -inf) must come out as -inf: with the row constants zeroed each
  // element does that by itself (scale (-inf) - 0), and no element needs a select
  // (CTAs of 512 threads and more have no register to spare for the two constants and keep the
  // select: bf16 16384 columns measured 57 % with them against 69 % without)
  constexpr bool kLeanLog = (THREADS <= 256);
  const float m_out = dead ? 0.f : M, lse_out = dead ? 0.f : lse_l;
  const float neg_shift = -fmaf(m_out, p.scale, lse_out);
  // the fill value as stored bits: +0, -inf or quiet NaN in the element type
  const uint32_t fill_word = E::fill_word(fill);
  const uint4 fill_vec = make_uint4(fill_word, fill_word, fill_word, fill_word);

#pragma unroll
  for (int k = 0; k < KFILL; ++k) {
    const int idx = tg + k * G;
    if (k >= NK) {                                           // compile-time: wholly masked iteration
      if (idx < nvec) st_stream(yr + k * G * EPV, fill_vec); // constant bits, no conversion
      continue;
    }
    uint4 out_vec = fill_vec;
    if (k < NK - 1 || last_ok) {
      float o[EPV];
#pragma unroll
      for (int j = 0; j < EPV; ++j) {
        if (OP == OP_SOFTMAX) o[j] = v[k < NK ? k : 0][j] * scale;
        else if (kLeanLog) o[j] = kFusedExponent ? fmaf(v[k < NK ? k : 0][j], p.scale, neg_shift)
                                                 : fmaf(v[k < NK ? k : 0][j] - m_out, p.scale, -lse_out);
        else o[j] = dead ? kNegInf : fmaf(v[k < NK ? k : 0][j] - M, p.scale, -lse_l);
      }
      if (k == NK - 1 && ragged && idx == live_vecs - 1) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) if (idx * EPV + j >= live) o[j] = fill;
      }
      out_vec = E::pack(o);
    }
    if (idx < nvec) st_stream(yr + k * G * EPV, out_vec);    // one store site per live iteration
  }
}

// Pick the body for this row's number of live iterations (uniform over the row's group).
template <int OP, typename T, int G, int VPT, int KFILL, int THREADS, bool RING = false, bool PREF = false>
__device__ __forceinline__ void softmax_row_dispatch(const RowParams& p, long long row, int tg, int nvec,
                                                     float (*red)[THREADS / 32], uint32_t ring_buf = 0,
                                                     uint4* pre = nullptr, const T* next_xr = nullptr,
                                                     int next_live_vecs = 0) {
  constexpr int EPV = Elem<T>::EPV;
  static_assert(VPT <= 8, "row body is specialised for up to eight iterations");
  const int live = static_cast<int>(live_cols(p, row));
  const int live_vecs = (live + EPV - 1) / EPV;
  const int nk = (live_vecs + G - 1) / G;
#define AKG_SM_CASE(NK_)                                                                                      \
  case NK_:                                                                                                   \
    if constexpr (NK_ <= VPT)                                                                                 \
      softmax_row<OP, T, G, VPT, KFILL, THREADS, NK_, RING, PREF>(p, row, tg, nvec, live, live_vecs, red,     \
                                                                  ring_buf, pre, next_xr, next_live_vecs);    \
    break;
  switch (nk) {
    AKG_SM_CASE(0) AKG_SM_CASE(1) AKG_SM_CASE(2) AKG_SM_CASE(3) AKG_SM_CASE(4)
    AKG_SM_CASE(5) AKG_SM_CASE(6) AKG_SM_CASE(7) AKG_SM_CASE(8)
    default: break;
  }
#undef AKG_SM_CASE
}

// Rows of a CTA-per-row launch are prefetched one ahead (see softmax_row) where the extra
// VPT vectors fit the register file: four vectors per thread need 80 registers, which 128-
// and 256-thread CTAs get by giving up a quarter of the resident warps (measured +8 % on
// the causal bf16 workload); wider CTAs keep the 64-register form without prefetch.
template <int THREADS, int VPT> constexpr bool kSoftmaxPref = (VPT <= 2) || (VPT == 4 && THREADS <= 256);
template <int G, int THREADS, int VPT> constexpr int kSoftmaxMinBlocks =
    (G == THREADS && VPT == 4 && THREADS == 128) ? 6
    : (G == THREADS && (VPT == 4 || VPT == 8) && THREADS == 256) ? 3 : kRegMinBlocks<THREADS>;

template <int OP, typename T, int G, int VPT, int THREADS>
__global__ void __launch_bounds__(THREADS, kSoftmaxMinBlocks<G, THREADS, VPT>) reg_softmax(const RowParams p) {
  pdl_prologue();
  constexpr int EPV = Elem<T>::EPV;
  constexpr int NWC = THREADS / 32;
  static_assert(OP == OP_SOFTMAX || OP == OP_LOG_SOFTMAX, "softmax pair only");
  static_assert(G == 32 || G == THREADS, "a warp or a CTA per row");
  __shared__ float red[2][2][NWC];
  const int nvec = static_cast<int>(p.cols / EPV);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if constexpr (G == 32) {
    // a warp per row throughout (rows short enough for one warp's registers)
    for (long long rb = static_cast<long long>(blockIdx.x) * NWC; rb < p.rows;
         rb += static_cast<long long>(gridDim.x) * NWC) {
      if (rb + warp >= p.rows) continue;
      softmax_row_dispatch<OP, T, 32, VPT, VPT, THREADS>(p, balanced_row(p, rb + warp), lane, nvec, red[0]);
    }
  } else {
    // a CTA per row, grid-stride (persistent when the planner caps the grid); the vectors
    // of the CTA's next row are loaded while the current row is computed
    int parity = 0;
    if constexpr (!kSoftmaxPref<THREADS, VPT>) {
      for (long long r = blockIdx.x; r < p.rows; r += gridDim.x, parity ^= 1)
        softmax_row_dispatch<OP, T, THREADS, VPT, VPT, THREADS>(p, balanced_row(p, r), threadIdx.x, nvec, red[parity]);
      return;
    }
    const int tg = threadIdx.x;
    const T* xb = reinterpret_cast<const T*>(p.x) + tg * EPV;
    uint4 pre[VPT];
    long long r = blockIdx.x;
    if (r >= p.rows) return;
    long long row = balanced_row(p, r);
    {
      const int lv = (static_cast<int>(live_cols(p, row)) + EPV - 1) / EPV;
#pragma unroll
      for (int k = 0; k < VPT; ++k)
        if (tg + k * THREADS < lv) pre[k] = ld_stream(xb + row * p.xs + k * THREADS * EPV);
    }
    for (; r < p.rows; r += gridDim.x, parity ^= 1) {
      const long long rn = r + gridDim.x;
      long long row_n = 0;
      int lv_n = 0;
      if (rn < p.rows) {
        row_n = balanced_row(p, rn);
        lv_n = (static_cast<int>(live_cols(p, row_n)) + EPV - 1) / EPV;
      }
      softmax_row_dispatch<OP, T, THREADS, VPT, VPT, THREADS, false, true>(p, row, tg, nvec, red[parity], 0, pre,
                                                                            xb + row_n * p.xs, lv_n);
      row = row_n;
    }
  }
}


// The (maximum, rescaled sum) pairs of the CTAs of a cluster -> the pair of the whole row, in every CTA:
// each CTA sends its pair to every peer with one 16-byte st.async that counts on the receiver's mbarrier
// (the scheme of split_kernel; slot and barrier alternate between two sets from row to row), waits for the
// cluster's pairs with a bounded wait and merges them by a butterfly.  False if the wait ran out.
struct ClusterPairs {
  float4 (*inbox)[kMaxCluster];      // [2][kMaxCluster] in shared memory
  uint64_t* xbar;                    // [2]
  uint32_t cs, rank, phases;
  __device__ __forceinline__ void init(float4 (*ib)[kMaxCluster], uint64_t* xb) {
    inbox = ib; xbar = xb; phases = 0;
    cs = cluster_size(); rank = cluster_rank();
    if (cs > 1) {
      if (threadIdx.x == 0) {
        mbar_init(smem_addr(&xbar[0]), 1);
        mbar_init(smem_addr(&xbar[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      }
      __syncthreads();
      cluster_arrive();            // every CTA of the cluster is running before any remote store
      cluster_wait();
    }
  }
  // every thread of the CTA calls this with the CTA's pair (M, S)
  __device__ __forceinline__ bool merge(float& M, float& S, int par, float l2e, int* status, unsigned wait_us) {
    if (threadIdx.x == 0) mbar_expect_tx(smem_addr(&xbar[par]), cs * 16u);
    if (threadIdx.x < cs) st_async_f32x4(smem_addr(&inbox[par][rank]), smem_addr(&xbar[par]), threadIdx.x, M, S, 0.f, 0.f);
    const bool ok = mbar_wait_timed<true>(smem_addr(&xbar[par]), (phases >> par) & 1u, status, wait_us);
    phases ^= 1u << par;
    const float4 f = inbox[par][threadIdx.x & (cs - 1)];
    const Stat r = butterfly_merge<OP_SOFTMAX>(Stat{f.x, f.y, 0.f}, static_cast<int>(cs), l2e);
    M = r.a; S = r.b;
    return ok;
  }
  __device__ __forceinline__ void finish() const {
    if (cs > 1) { cluster_arrive(); cluster_wait(); }   // nobody leaves while a peer may still send to it
  }
};


// ------------------------------------------------------------------------------------------------
// reg_softmax_packed: the softmax pair on unmasked 16-bit rows of exactly blockDim.x * VPT vectors, the
// row kept PACKED in registers (as reg_norm_packed: four registers per vector, eight vectors per thread in
// 64 registers, half the threads per row of the widened form, eight loads per thread in flight).
//   maximum   packed two-lane maxima over the words (one instruction per two elements)
//   sum       e^(x - m_warp) with the stored value widened inside the subtraction (Elem::sub_wide), against
//             the warp's own maximum, so that one barrier serves both reductions
//   output    softmax: the exponential again, against the row maximum, times 1 / S (the widened form keeps
//             the first exponential instead: a second one here costs less than the registers for it);
//             log-softmax: scale (x - M) - ln S
// A CTA per row, grid-stride.  No mask: the planner sends masked calls to the kernels above.
// ------------------------------------------------------------------------------------------------
template <int OP, typename T, int VPT>
__global__ void __launch_bounds__(1024, 1) reg_softmax_packed(const RowParams p) {
  pdl_prologue();
  using E = Elem<T>;
  static_assert(sizeof(T) == 2, "16-bit storage only");
  static_assert(OP == OP_SOFTMAX || OP == OP_LOG_SOFTMAX, "softmax pair only");
  constexpr int EPV = E::EPV;
  __shared__ float red[2][2][32];
  __shared__ __align__(16) float4 inbox[2][kMaxCluster];
  __shared__ __align__(8) uint64_t xbar[2];
  const int G = blockDim.x;
  const int NW = G >> 5;
  const int tg = threadIdx.x;
  const int lane = tg & 31;
  const float l2e = p.l2e;
  // launched with a cluster of CS CTAs, CTA k holds vectors [k, k + 1) * G * VPT of the row (rows too long
  // for one CTA's registers: every element is still read from HBM once and never leaves the registers)
  ClusterPairs cl;
  cl.init(inbox, xbar);
  const long long slice = static_cast<long long>(cl.rank) * G * VPT * EPV;
  bool gave_up = false;
  int parity = 0;
  for (long long row = cluster_id(); row < p.rows; row += cluster_count(), parity ^= 1) {
    const T* xr = reinterpret_cast<const T*>(p.x) + row * p.xs + slice + tg * EPV;
    T* yr = reinterpret_cast<T*>(p.y) + row * p.ys + slice + tg * EPV;
    uint4 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) raw[k] = ld_stream(xr + static_cast<long long>(k) * G * EPV);
    // ---- maximum
    uint32_t mp = max_pair(static_cast<const T*>(nullptr), raw[0].x, raw[0].y);
    mp = max_pair(static_cast<const T*>(nullptr), mp, max_pair(static_cast<const T*>(nullptr), raw[0].z, raw[0].w));
#pragma unroll
    for (int k = 1; k < VPT; ++k) {
      const uint32_t a = max_pair(static_cast<const T*>(nullptr), raw[k].x, raw[k].y);
      const uint32_t b = max_pair(static_cast<const T*>(nullptr), raw[k].z, raw[k].w);
      mp = max_pair(static_cast<const T*>(nullptr), mp, max_pair(static_cast<const T*>(nullptr), a, b));
    }
    unsigned short m0, m1;
    halves(mp, m0, m1);
    const float m_w = warp_max(fmaxf(E::add_wide(m0, 0.f), E::add_wide(m1, 0.f)));
    const float m_ws = (m_w == kNegInf) ? 0.f : m_w;        // keeps -inf - -inf out of the exponent
    // ---- sum of exponentials against the warp's maximum (a NaN element makes the sum NaN)
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        unsigned short h0, h1;
        halves(w[i], h0, h1);
        s0 += ex2_approx(E::sub_wide(h0, m_ws) * l2e);
        s1 += ex2_approx(E::sub_wide(h1, m_ws) * l2e);
      }
    }
    const float s_w = warp_sum(s0 + s1);
    // ---- the warps' pairs: lane l takes warp l's (nothing beyond the CTA's warps)
    float M = m_w, S = s_w;
    if (NW > 1) {
      if (lane == 0) { red[parity][0][tg >> 5] = m_w; red[parity][1][tg >> 5] = s_w; }
      __syncthreads();
      const float mw = lane < NW ? red[parity][0][lane] : kNegInf;
      const float sw = lane < NW ? red[parity][1][lane] : 0.f;
      M = warp_max(mw);
      const float Ms = (M == kNegInf) ? 0.f : M;
      S = warp_sum(sw * ((mw == M) ? 1.f : exp_diff(mw, Ms, l2e)));      // equal maxima (also +-inf): factor 1
    }
    if (cl.cs > 1 && !gave_up && !cl.merge(M, S, parity, l2e, p.status, p.wait_us)) gave_up = true;
    if (gave_up) continue;                                // (no CTA barrier follows in this row: see below)
    const bool dead = (M == kNegInf) && !(S != S);        // only NaN / -inf entries: a NaN row, not a dead one
    const float Mo = (M == kNegInf) ? 0.f : M;
    if (OP == OP_SOFTMAX) {
      const float inv = dead ? 0.f : __frcp_rn(S);
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(w[i], h0, h1);
          o[i] = E::pack2(ex2_approx(E::sub_wide(h0, Mo) * l2e) * inv, ex2_approx(E::sub_wide(h1, Mo) * l2e) * inv);
        }
        st_stream(yr + static_cast<long long>(k) * G * EPV, make_uint4(o[0], o[1], o[2], o[3]));
      }
    } else {
      // a dead row: M and ln S are taken as 0, and scale (-inf - 0) - 0 = -inf for every element by itself
      const float neg_lse = dead ? 0.f : -logf(S);
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          unsigned short h0, h1;
          halves(w[i], h0, h1);
          o[i] = E::pack2(fmaf(E::sub_wide(h0, Mo), p.scale, neg_lse), fmaf(E::sub_wide(h1, Mo), p.scale, neg_lse));
        }
        st_stream(yr + static_cast<long long>(k) * G * EPV, make_uint4(o[0], o[1], o[2], o[3]));
      }
    }
  }
  cl.finish();
}

// ------------------------------------------------------------------------------------------------
// reg_softmax_flex: the fp32 counterpart of reg_softmax_packed - the softmax pair on unmasked fp32 rows of
// exactly blockDim.x * VPT vectors, blockDim.x any multiple of 32, so that a row takes the fewest threads
// that hold it with up to eight vectors each (12288 columns: 384 threads of eight instead of a ragged CTA of
// 512).  Values in registers, one exponential per element (softmax keeps it for the output), one barrier.
// ------------------------------------------------------------------------------------------------
template <int OP, int VPT>
__global__ void __launch_bounds__(1024, 1) reg_softmax_flex(const RowParams p) {
  pdl_prologue();
  using E = Elem<float>;
  static_assert(OP == OP_SOFTMAX || OP == OP_LOG_SOFTMAX, "softmax pair only");
  constexpr int EPV = E::EPV;
  constexpr int N = VPT * EPV;
  __shared__ float red[2][2][32];
  __shared__ __align__(16) float4 inbox[2][kMaxCluster];
  __shared__ __align__(8) uint64_t xbar[2];
  const int G = blockDim.x;
  const int NW = G >> 5;
  const int tg = threadIdx.x;
  const int lane = tg & 31;
  const float l2e = p.l2e;
  ClusterPairs cl;                    // a cluster of CS CTAs per row, as in reg_softmax_packed
  cl.init(inbox, xbar);
  const long long slice = static_cast<long long>(cl.rank) * G * VPT * EPV;
  bool gave_up = false;
  int parity = 0;
  for (long long row = cluster_id(); row < p.rows; row += cluster_count(), parity ^= 1) {
    const float* xr = reinterpret_cast<const float*>(p.x) + row * p.xs + slice + tg * EPV;
    float* yr = reinterpret_cast<float*>(p.y) + row * p.ys + slice + tg * EPV;
    uint4 raw[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) raw[k] = ld_stream(xr + static_cast<long long>(k) * G * EPV);
    float v[N];
    float m_t = kNegInf;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
      float f[EPV];
      E::unpack(raw[k], f);
#pragma unroll
      for (int j = 0; j < EPV; ++j) { v[k * EPV + j] = f[j]; m_t = fmaxf(m_t, f[j]); }
    }
    const float m_w = warp_max(m_t);
    const float m_ws = (m_w == kNegInf) ? 0.f : m_w;        // keeps -inf - -inf out of the exponent
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int i = 0; i < N; i += 2) {
      const float e0 = exp_diff(v[i], m_ws, l2e), e1 = exp_diff(v[i + 1], m_ws, l2e);
      s0 += e0;
      s1 += e1;
      if (OP == OP_SOFTMAX) { v[i] = e0; v[i + 1] = e1; }
    }
    const float s_w = warp_sum(s0 + s1);
    float M = m_w, S = s_w, my_factor = 1.f;
    if (NW > 1) {
      if (lane == 0) { red[parity][0][tg >> 5] = m_w; red[parity][1][tg >> 5] = s_w; }
      __syncthreads();
      const float mw = lane < NW ? red[parity][0][lane] : kNegInf;
      const float sw = lane < NW ? red[parity][1][lane] : 0.f;
      M = warp_max(mw);
      const float Ms = (M == kNegInf) ? 0.f : M;
      S = warp_sum(sw * ((mw == M) ? 1.f : exp_diff(mw, Ms, l2e)));      // equal maxima (also +-inf): factor 1
      my_factor = (m_w == M) ? 1.f : exp_diff(m_w, Ms, l2e);
    }
    if (cl.cs > 1) {
      if (!gave_up && !cl.merge(M, S, parity, l2e, p.status, p.wait_us)) gave_up = true;
      my_factor = (m_w == M) ? 1.f : exp_diff(m_w, (M == kNegInf) ? 0.f : M, l2e);
    }
    if (gave_up) continue;
    const bool dead = (M == kNegInf) && !(S != S);        // only NaN / -inf entries: a NaN row, not a dead one
    if (OP == OP_SOFTMAX) {
      const float scale = dead ? 0.f : my_factor * __frcp_rn(S);
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        float o[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) o[j] = v[k * EPV + j] * scale;
        st_stream(yr + static_cast<long long>(k) * G * EPV, E::pack(o));
      }
    } else {
      // a dead row: M and ln S are taken as 0, and scale (-inf - 0) - 0 = -inf for every element by itself
      const float Mo = dead ? 0.f : M, neg_lse = dead ? 0.f : -logf(S);
#pragma unroll
      for (int k = 0; k < VPT; ++k) {
        float o[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) o[j] = fmaf(v[k * EPV + j] - Mo, p.scale, neg_lse);
        st_stream(yr + static_cast<long long>(k) * G * EPV, E::pack(o));
      }
    }
  }
  cl.finish();
}

}  // namespace akg
