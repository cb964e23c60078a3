// Device-side building blocks shared by every kernel family of the row-operator
// library: parameter block, element packing, streaming loads / stores, and the
// per-operator statistics (online max / rescaled sum for the softmax pair,
// count-mean-M2 with Chan's merge for LayerNorm, sum of squares for RMSNorm).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace akg {

enum Op : int { OP_SOFTMAX = 0, OP_LOG_SOFTMAX = 1, OP_LAYERNORM = 2, OP_RMSNORM = 3 };
enum DType : int { DT_F32 = 0, DT_BF16 = 1, DT_F16 = 2 };

// One operator call.  Strides in elements.  gamma doubles as the RMSNorm weight.
struct RowParams {
  const void* x;
  void* y;
  long long rows, cols, xs, ys;
  const void* gamma;
  const void* beta;
  float eps;
  const void* add;          // additive mask or nullptr
  long long add_rows, add_stride;
  int causal;
  long long period, offset;
  int period_pow2;          // 1: period is a power of two (row & (period - 1))
  int add_mode;             // 0: row % add_rows, 1: add_rows == 1, 2: add_rows >= rows
  int interleave;           // 1: visit the rows of a causal period short/long alternately
  long long row_base;       // global index of row 0 (mask rules use row + row_base); 0 unless chunked
  int* status;              // device status word (bounded waits report here)
  unsigned wait_us;         // limit of a bounded wait in microseconds; 0 = two seconds
  int no_copies;            // test only: the ring kernels issue no bulk copy, so every wait runs out
  // fused residual add (normalisations only): the operator runs on x + res; the sum is also
  // stored to `sum` unless that is nullptr.  res == nullptr: plain operator.
  const void* res;
  long long rs;             // row stride of res
  void* sum;
  long long ss;             // row stride of sum
  // fused pre-scale of the softmax pair: the operator runs on scale * x (+ additive mask).
  // The kernels keep x unscaled (for scale > 0 the maximum sits at the same place) and fold the
  // scale into the constant of the exponential: l2e = scale * log2(e).  The additive mask is
  // taken as add * inv_scale; log-softmax multiplies its difference by scale at the end.
  float l2e, scale, inv_scale;
};

// One call over a non-last axis: x[outer, reduce, inner], inner contiguous.
struct AxisParams {
  const void* x;
  void* y;
  long long outer, reduce, inner;
  long long xso, xsf, yso, ysf;       // outer / reduce strides in elements (inner stride is 1)
  const void* gamma;                  // [reduce] or nullptr (RMSNorm weight / LayerNorm gamma)
  const void* beta;                   // [reduce] or nullptr
  float eps;
};

// One gated-activation call: x[rows, 2 d] (gate | factor), y[rows, d].
struct ActParams {
  const void* x;
  void* y;
  long long rows, d;                  // d: output columns
  long long xs, ys;                   // row strides in elements
};

// One BatchNorm-style column normalisation: x, y [rows, cols]; per-column gamma / beta.
struct ColParams {
  const void* x;
  void* y;
  long long rows, cols, xs, ys;
  const void* gamma;
  const void* beta;
  float eps;
  float2* partial;                    // workspace [row blocks][cols]: (mean, M2) of each block
  float* mean_out;                    // [cols] or nullptr
  float* var_out;                     // [cols] or nullptr
  long long rows_per_block;           // a multiple of the CTA's row slots
  int lc_shift;                       // log2 of the lanes of a warp that lie along the columns
  int l2_keep;                        // 1: the matrix is small enough for L2 priorities to pay (see kernels_colnorm.cuh)
};

// Shared-memory ring kernels: limits and the size of the bookkeeping area that
// precedes the ring buffers (mbarriers, CTA reduction slots, cluster exchange slots).
constexpr int kMaxCluster = 16;
constexpr int kMaxBuf = 16;
constexpr unsigned kMaxDynSmem = 232448;      // 227 KiB opt-in limit per CTA
// layout: ring mbarriers [kMaxBuf] | exchange mbarriers [4] | inbox of the st.async exchange
// [4][kMaxCluster] x 16 bytes | CTA reduction slots [2][warps] | remote-store slots [2][kMaxCluster]
__host__ __device__ constexpr unsigned smem_header_bytes(int threads) {
  return (kMaxBuf * 8u + 4u * 8u + 4u * kMaxCluster * 16u + (2u * (threads / 32) + 2u * kMaxCluster) * 12u + 127u) & ~127u;
}

// Programmatic dependent launch.  Every kernel starts with this: it waits until the
// kernel launched before it on the stream has completed and its writes are visible
// (so stream order is kept exactly), then lets the kernel launched after it begin to
// place its CTAs while this one drains.  Both instructions do nothing when the launch
// did not ask for programmatic serialisation.  What is gained is the launch latency
// between back-to-back kernels (about 2.5 us on B200, a tenth of a 20 us kernel).
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegInf = -__builtin_huge_valf();

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// e^(a - b) for a <= b (or NaN / inf operands, which propagate as IEEE says)
__device__ __forceinline__ float exp_diff(float a, float b) { return ex2_approx((a - b) * kLog2e); }
// e^(scale (a - b)) with l2e = scale * log2(e)
__device__ __forceinline__ float exp_diff(float a, float b, float l2e) { return ex2_approx((a - b) * l2e); }

// 128-bit streaming accesses: the row data is touched once, keep it out of L1.
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
// streaming store (evict-first in L2): measured against the default and the .cg forms on the four large
// configurations, it is 1 - 2 % ahead in the register kernels and 7 % in the two-pass kernel, whose second pass
// needs the L2 room the output lines would take
__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// read-only, cached (gamma / beta / weight are reused by every row)
__device__ __forceinline__ uint4 ld_cached(const void* p) {
  return __ldg(reinterpret_cast<const uint4*>(p));
}

template <typename T> struct Elem;

template <> struct Elem<float> {
  static constexpr int EPV = 4;                    // elements per 16-byte vector
  static constexpr int DT = DT_F32;
  static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y);
    f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
  }
  static __device__ __forceinline__ uint4 pack(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]),
                      __float_as_uint(f[2]), __float_as_uint(f[3]));
  }
  static __device__ __forceinline__ float load1(const void* base, long long i) {
    return reinterpret_cast<const float*>(base)[i];
  }
  static __device__ __forceinline__ void store1(void* base, long long i, float v) {
    reinterpret_cast<float*>(base)[i] = v;
  }
  // the stored bits of v, replicated to fill a 32-bit word (for constant fills)
  static __device__ __forceinline__ uint32_t fill_word(float v) { return __float_as_uint(v); }
};

template <> struct Elem<__nv_bfloat16> {
  static constexpr int EPV = 8;
  static constexpr int DT = DT_BF16;
  static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);            // low half = even element
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);   // round-to-nearest-even, once
    return *reinterpret_cast<uint32_t*>(&h);
  }
  static __device__ __forceinline__ uint4 pack(const float (&f)[8]) {
    return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
  }
  static __device__ __forceinline__ float load1(const void* base, long long i) {
    return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(base)[i]) << 16);
  }
  static __device__ __forceinline__ void store1(void* base, long long i, float v) {
    reinterpret_cast<__nv_bfloat16*>(base)[i] = __float2bfloat16_rn(v);
  }
  static __device__ __forceinline__ uint32_t fill_word(float v) { return pack2(v, v); }
  // Mixed-precision arithmetic of sm_100: a 16-bit operand is widened inside the instruction, which
  // runs on the FMA pipe, so the value never has to be unpacked by a shift / mask on the ALU pipe.
  // `h` is one stored element (either half of a packed word, see halves()).
  static __device__ __forceinline__ float sub_wide(unsigned short h, float c) {            // h - c
    float d; asm("sub.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(c)); return d;
  }
  static __device__ __forceinline__ float add_wide(unsigned short h, float c) {            // h + c
    float d; asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(c)); return d;
  }
  static __device__ __forceinline__ float fma_wide(unsigned short a, unsigned short b, float c) {   // a * b + c
    float d; asm("fma.rn.f32.bf16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c)); return d;
  }
};

// element-wise maximum of two packed pairs (a NaN operand is ignored, as fmaxf does)
__device__ __forceinline__ uint32_t max_pair(const __nv_bfloat16*, uint32_t a, uint32_t b) {
  uint32_t d; asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}
__device__ __forceinline__ uint32_t max_pair(const __half*, uint32_t a, uint32_t b) {
  uint32_t d; asm("max.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}

// the two 16-bit halves of a packed word (low half = even element)
__device__ __forceinline__ void halves(uint32_t w, unsigned short& lo, unsigned short& hi) {
  asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
}

// IEEE half (the paper's float16 regime, Section 4.1): same vector shape as bf16, hardware
// conversions in both directions, one rounding (nearest-even) at the store.
template <> struct Elem<__half> {
  static constexpr int EPV = 8;
  static constexpr int DT = DT_F16;
  static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      f[2 * i] = p.x;
      f[2 * i + 1] = p.y;
    }
  }
  static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
  }
  static __device__ __forceinline__ uint4 pack(const float (&f)[8]) {
    return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
  }
  static __device__ __forceinline__ float load1(const void* base, long long i) {
    return __half2float(reinterpret_cast<const __half*>(base)[i]);
  }
  static __device__ __forceinline__ void store1(void* base, long long i, float v) {
    reinterpret_cast<__half*>(base)[i] = __float2half_rn(v);
  }
  static __device__ __forceinline__ uint32_t fill_word(float v) { return pack2(v, v); }
  static __device__ __forceinline__ float sub_wide(unsigned short h, float c) {
    float d; asm("sub.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(c)); return d;
  }
  static __device__ __forceinline__ float add_wide(unsigned short h, float c) {
    float d; asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(h), "f"(c)); return d;
  }
  static __device__ __forceinline__ float fma_wide(unsigned short a, unsigned short b, float c) {
    float d; asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c)); return d;
  }
};

template <int OP> struct OpTraits {
  static constexpr bool kSoftmaxLike = (OP == OP_SOFTMAX || OP == OP_LOG_SOFTMAX);
};

// Number of leading live columns of a row (the rest is masked by the causal rule).
__device__ __forceinline__ long long live_cols(const RowParams& p, long long row) {
  if (!p.causal) return p.cols;
  const long long g = row + p.row_base;
  const long long rp = p.period_pow2 ? (g & (p.period - 1)) : (g % p.period);
  long long l = rp + p.offset + 1;
  return l < 0 ? 0 : (l > p.cols ? p.cols : l);
}

// Under a causal mask the live length grows with the row's position in its period, so
// neighbouring rows cost the same and an SM would see all-short then all-long rows.
// With p.interleave set (period a power of two, rows a multiple of it) work item i of a
// period is mapped to row i/2 (i even) or period-1-i/2 (i odd): CTAs resident together
// then mix short and long rows, and load-heavy and store-heavy work overlap.  Rows are
// independent, so any one-to-one order is valid.
__device__ __forceinline__ long long balanced_row(const RowParams& p, long long i) {
  if (!p.interleave) return i;
  const long long r = i & (p.period - 1);
  const long long h = r >> 1;
  return (i - r) + ((r & 1) ? (p.period - 1 - h) : h);
}

// Row of the additive mask that row `row` uses.
__device__ __forceinline__ long long add_row(const RowParams& p, long long row) {
  return p.add_mode == 1 ? 0 : (p.add_mode == 2 ? row + p.row_base : (row + p.row_base) % p.add_rows);
}

// ---------------------------------------------------------------------------------
// Per-row statistics.  Field use:
//   softmax pair : a = running max m, b = sum of exp(z - m)
//   LayerNorm    : a = count, b = mean, c = sum of squared deviations (M2)
//   RMSNorm      : a = sum of squares
// ---------------------------------------------------------------------------------
struct Stat { float a, b, c; };

template <int OP> __device__ __forceinline__ Stat stat_identity() {
  if (OpTraits<OP>::kSoftmaxLike) return Stat{kNegInf, 0.f, 0.f};
  return Stat{0.f, 0.f, 0.f};
}

template <int OP> __device__ __forceinline__ Stat stat_merge(const Stat& x, const Stat& y, float l2e = kLog2e) {
  Stat r;
  if (OpTraits<OP>::kSoftmaxLike) {
    // (m, s) (+) (m', s') = (M, s e^(m-M) + s' e^(m'-M)); equal maxima (also both
    // -inf, or both +inf) take factor 1 so that no inf - inf is formed here.
    const float M = fmaxf(x.a, y.a);
    const float fx = (x.a == M) ? 1.f : exp_diff(x.a, M, l2e);
    const float fy = (y.a == M) ? 1.f : exp_diff(y.a, M, l2e);
    r.a = M; r.b = x.b * fx + y.b * fy; r.c = 0.f;
  } else if (OP == OP_LAYERNORM) {
    // Chan's pairwise update of (count, mean, M2)
    const float n = x.a + y.a;
    const float w = (n > 0.f) ? __fdividef(y.a, n) : 0.f;
    const float d = y.b - x.b;
    r.a = n; r.b = x.b + d * w; r.c = x.c + y.c + d * d * x.a * w;
  } else {
    r.a = x.a + y.a; r.b = 0.f; r.c = 0.f;
  }
  return r;
}

// 1 / sqrt(a): hardware approximation plus one Newton step (about 1 ulp).
__device__ __forceinline__ float rsqrt_refined(float a) {
  float r = rsqrtf(a);
  if (a > 0.f && a < __int_as_float(0x7f800000)) r = r * (1.5f - 0.5f * a * r * r);
  return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  return v;
}

// Sum of n values (n a power of two, at most 32) held one per lane, lane l holding entry l mod n; every
// lane gets the same bits (an xor butterfly adds the same pairs in every lane).
__device__ __forceinline__ float lanes_sum(float v, int n) {
  for (int m = 1; m < n; m <<= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
  return v;
}

__device__ __forceinline__ float lanes_max(float v, int n) {
  for (int m = 1; m < n; m <<= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, m));
  return v;
}

// (maximum, rescaled sum) of n softmax partials held one per lane: the maximum first, then every partial
// rescaled once, then the sum - two butterflies and one exponential per lane instead of log2 n ordered merges
// with two exponentials each (those merges were 0.4 special-function and 2.3 instructions in all per element of
// the two-pass kernel on configuration 4, on the path between a row's two passes).  Equal maxima (also both
// -inf, or both +inf) take factor 1, so that no inf - inf is formed; a NaN maximum cannot occur (fmaxf drops
// NaN), a NaN partial sum makes the row NaN.
template <int FULL_WARP> __device__ __forceinline__ Stat softmax_merge_lanes(const Stat& s, int n, float l2e) {
  float M = s.a;
  if (FULL_WARP) {
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, m));
  } else {
    M = lanes_max(M, n);
  }
  const float Ms = (M == kNegInf) ? 0.f : M;
  const float w = s.b * ((s.a == M) ? 1.f : exp_diff(s.a, Ms, l2e));
  return Stat{M, FULL_WARP ? warp_sum(w) : lanes_sum(w, n), 0.f};
}

// (count, mean, M2) of n partial statistics held one per lane (as lanes_sum), all at once instead of by
// pairwise Chan merges: N = sum n_i, mean = ref + sum n_i (mean_i - ref) / N, M2 = sum (M2_i + n_i (mean_i - mean)^2),
// ref being the first entry's mean: the sums run over differences of means, so the error of the merged mean
// scales with the spread of the partial means, not with their magnitude (as in the pairwise update).
// Three butterflies of sums replace log2 n merges with a division each; the per-row reductions of the
// two-pass cluster kernel were 590 warp instructions per warp and row-slice with pairwise merges, two fifths
// of all its LayerNorm instructions (fp32, 65536 columns).
template <int FULL_WARP> __device__ __forceinline__ Stat layernorm_merge_lanes(const Stat& s, int n) {
  const int first = FULL_WARP ? 0 : static_cast<int>(threadIdx.x & 31u & ~static_cast<unsigned>(n - 1));
  const float ref = __shfl_sync(0xffffffffu, s.b, first);
  const float w = s.a * (s.b - ref);
  const float cnt = FULL_WARP ? warp_sum(s.a) : lanes_sum(s.a, n);
  const float sum = FULL_WARP ? warp_sum(w) : lanes_sum(w, n);
  // (the fast division's two ulps apply to the correction term only; a correctly rounded division here, on
  // the path between a row's two passes, cost the two-pass kernel 6 % on fp32 LayerNorm)
  const float mean = (cnt > 0.f) ? ref + __fdividef(sum, cnt) : 0.f;
  const float d = s.b - mean;
  const float m2 = fmaf(s.a * d, d, s.c);
  return Stat{cnt, mean, FULL_WARP ? warp_sum(m2) : lanes_sum(m2, n)};
}

template <int OP> __device__ __forceinline__ Stat stat_shfl_xor(const Stat& s, int lane_mask) {
  Stat r;
  r.a = __shfl_xor_sync(0xffffffffu, s.a, lane_mask);
  r.b = (OP != OP_RMSNORM) ? __shfl_xor_sync(0xffffffffu, s.b, lane_mask) : 0.f;
  r.c = (OP == OP_LAYERNORM) ? __shfl_xor_sync(0xffffffffu, s.c, lane_mask) : 0.f;
  return r;
}

template <int OP> __device__ __forceinline__ Stat warp_reduce(Stat s, float l2e = kLog2e) {
  if constexpr (OP == OP_LAYERNORM) return layernorm_merge_lanes<1>(s, 32);
  if constexpr (OP == OP_RMSNORM) return Stat{warp_sum(s.a), 0.f, 0.f};
  if constexpr (OpTraits<OP>::kSoftmaxLike) return softmax_merge_lanes<1>(s, 32, l2e);
#pragma unroll
  for (int m = 16; m >= 1; m >>= 1) s = stat_merge<OP>(s, stat_shfl_xor<OP>(s, m), l2e);
  return s;
}

// Merge n statistics (n a power of two, at most 32) held one per lane, lane l holding entry l mod n, by a
// butterfly of log2 n steps.  Both partners of a step merge (entry of the lower lane, entry of the higher
// lane) in that order, so every lane ends with the same bits; a serial merge of 16 entries is a chain of 15
// dependent merges (two exponentials each for the softmax pair), this one of four.
template <int OP> __device__ __forceinline__ Stat butterfly_merge(Stat s, int n, float l2e = kLog2e) {
  if constexpr (OP == OP_LAYERNORM) return layernorm_merge_lanes<0>(s, n);
  if constexpr (OP == OP_RMSNORM) return Stat{lanes_sum(s.a, n), 0.f, 0.f};
  if constexpr (OpTraits<OP>::kSoftmaxLike) return softmax_merge_lanes<0>(s, n, l2e);
  const int lane = threadIdx.x & 31;
  for (int k = 1; k < n; k <<= 1) {
    const Stat o = stat_shfl_xor<OP>(s, k);
    const bool upper = (lane & k) != 0;                    // the operands are ordered, the merge is evaluated once
    const Stat lo{upper ? o.a : s.a, upper ? o.b : s.b, 0.f}, hi{upper ? s.a : o.a, upper ? s.b : o.b, 0.f};
    s = stat_merge<OP>(lo, hi, l2e);
  }
  return s;
}

// Reduce over a whole CTA of NW warps.  `slots` points at NW Stat entries of shared
// memory reserved for this call; callers alternate between two slot sets on
// successive rows so one barrier per row is enough.  Every thread gets the result,
// combined in the same order, hence bit-identical across the CTA.
template <int OP, int NW> __device__ __forceinline__ Stat cta_reduce(Stat s, Stat* slots, float l2e = kLog2e) {
  s = warp_reduce<OP>(s, l2e);
  if (NW == 1) return s;
  if ((threadIdx.x & 31) == 0) slots[threadIdx.x >> 5] = s;
  __syncthreads();
  if constexpr ((NW & (NW - 1)) == 0 && NW <= 32) {
    return butterfly_merge<OP>(slots[threadIdx.x & (NW - 1)], NW, l2e);
  } else {
    Stat r = slots[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) r = stat_merge<OP>(r, slots[w], l2e);
    return r;
  }
}

// Row scalars derived from the reduced statistics.
//   softmax     : p = M (row max, or 0 if no live entry), q = 1 / S (0 if no live entry)
//   log-softmax : p = M, q = ln S (both 0 if no live entry); dead = no live entry
//   LayerNorm   : p = mean, q = 1 / sqrt(var + eps)
//   RMSNorm     : q = 1 / sqrt(mean square + eps)
struct RowScalars { float p, q; bool dead; };

template <int OP> __device__ __forceinline__ RowScalars finalize(const Stat& s, long long cols, float eps) {
  RowScalars r;
  r.dead = false;
  if (OP == OP_SOFTMAX) {
    r.dead = (s.a == kNegInf) && !(s.b != s.b);   // a row of only NaN / -inf is a NaN row
    r.p = r.dead ? 0.f : s.a;
    r.q = r.dead ? 0.f : 1.0f / s.b;
  } else if (OP == OP_LOG_SOFTMAX) {
    r.dead = (s.a == kNegInf) && !(s.b != s.b);   // a row of only NaN / -inf is a NaN row
    r.p = r.dead ? 0.f : s.a;                     // zeroed for a dead row: pre (-inf - 0) - 0 = -inf without a select
    r.q = r.dead ? 0.f : logf(s.b);
  } else if (OP == OP_LAYERNORM) {
    r.p = s.b;
    r.q = rsqrt_refined(fmaf(s.c, __frcp_rn(static_cast<float>(cols)), eps));
  } else {
    r.p = 0.f;
    r.q = rsqrt_refined(fmaf(s.a, __frcp_rn(static_cast<float>(cols)), eps));
  }
  return r;
}

// Statistics of a register tile of N already-masked values (n_valid of them count).
// For softmax the values are replaced by exp(z - m_local) so that the exponential
// is evaluated once per element; the caller later scales by exp(m_local - M) / S.
template <int OP, int N>
__device__ __forceinline__ Stat tile_stats(float (&v)[N], int n_valid, float& m_local, float l2e = kLog2e) {
  Stat s = stat_identity<OP>();
  m_local = 0.f;
  if (OpTraits<OP>::kSoftmaxLike) {
    float m = kNegInf;
#pragma unroll
    for (int i = 0; i < N; ++i) m = fmaxf(m, v[i]);
    const float ms = (m == kNegInf) ? 0.f : m;      // keeps -inf - -inf out of the exponent
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const float e = exp_diff(v[i], ms, l2e);
      acc += e;
      if (OP == OP_SOFTMAX) v[i] = e;
    }
    s.a = m; s.b = acc; m_local = m;
  } else if (OP == OP_LAYERNORM) {
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) sum += (i < n_valid) ? v[i] : 0.f;
    const float n = static_cast<float>(n_valid);
    const float mean = (n_valid > 0) ? sum / n : 0.f;
    float m2 = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) { const float d = v[i] - mean; m2 += (i < n_valid) ? d * d : 0.f; }
    s.a = n; s.b = mean; s.c = m2;
  } else {
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) ss += (i < n_valid) ? v[i] * v[i] : 0.f;
    s.a = ss;
  }
  return s;
}

}  // namespace akg
