// C ABI of the row-operator library: argument validation, kernel-family choice,
// launch.  No device memory is allocated here and nothing synchronises.
#include <atomic>
#include <climits>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/akg.h"
#include "launch.cuh"

namespace akg {
namespace {

thread_local char t_error[256] = "";
thread_local char t_kernel[96] = "";
thread_local size_t t_host_up = 0, t_host_down = 0;   // bytes the last host-buffer call copied each way
std::atomic<int> g_forced_variant{V_AUTO};
std::atomic<int> g_tune_reg_threads{0};   // 0 = planner's choice
std::atomic<int> g_tune_reg_vpt{0};
std::atomic<int> g_tune_reg_group{0};     // 0 = planner's choice, 32 = warp per row, 1 = CTA per row
std::atomic<int> g_tune_grid_cap{0};      // 0 = one CTA per row group
std::atomic<int> g_tune_cluster_size{0};  // shared-memory ring family: CTAs per row
std::atomic<int> g_tune_smem_nbuf{0};     //   ring depth limit
std::atomic<int> g_tune_smem_threads{0};  //   CTA size (256 / 512 / 1024)
std::atomic<int> g_tune_smem_ctas{0};     //   CTAs per SM the ring is sized for
std::atomic<int> g_tune_reg_general{0};   // 1 = never take the predicate-free normalisation kernel
std::atomic<int> g_tune_cluster_mode{0};  // 0 = planner's choice, 1 = row resident in shared memory, 2 = two-pass split
std::atomic<int> g_tune_tma_mode{0};      // 0 = planner's choice, 1 = ring-fed register kernel, 2 = shared-memory passes
std::atomic<int> g_tune_interleave{0};    // 1 = visit causal rows short/long alternately (default: storage order)
std::atomic<int> g_tune_pdl{0};           // 2 = launch without programmatic stream serialisation
std::atomic<int> g_tune_reg_flex{0};      // 2 = never the runtime-thread-count normalisation kernel, 5 = never its packed 16-bit form
std::atomic<int> g_tune_packed_vpt{0};    // packed 16-bit form: vectors per thread (0 = planner's choice)
std::atomic<int> g_tune_axis_r{0};        // non-last axis: rows per thread (2 / 4 / 8), -1 = two-pass kernel only
std::atomic<int> g_tune_axis_nc{0};       //   column blocks per CTA
std::atomic<int> g_tune_axis_lc{0};       //   two-pass kernel: 1 + log2 of the lanes along the columns
std::atomic<int> g_tune_host_chunks{0};   // host-buffer pipeline: chunks per call (0 = default)
std::atomic<int> g_tune_host_min_kib{0};  //   smallest chunk in KiB (0 = default)
std::atomic<int> g_tune_host_full_upload{0};  //   1 = upload the masked columns of causal rows too
std::atomic<int> g_tune_split_exchange{0};  // two-pass split kernel: 1 = cluster barrier per row instead of st.async + mbarrier
std::atomic<int> g_tune_split_l2{0};        //   L2 priority scheme (see split_kernel)
std::atomic<int> g_tune_test_wait_us{0};    // test only: limit of the kernels' bounded waits in microseconds (0 = two seconds)
std::atomic<int> g_tune_test_no_copies{0};  // test only: 1 = the ring kernels issue no bulk copy, so that their waits run out
std::atomic<int> g_tune_axis_mode{0};     //   1 = 16-byte vectors, 2 = bf16 8-byte vectors widened, 3 = elements

__device__ int g_status_word = 0;

akg_status fail(akg_status st, const char* fmt, const char* a = "", long long b = 0) {
  std::snprintf(t_error, sizeof t_error, fmt, a, b);
  return st;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool valid_dtype(int dtype) { return dtype == AKG_F32 || dtype == AKG_BF16 || dtype == AKG_F16; }
const char* dtype_name(int dtype) { return dtype == AKG_F32 ? "f32" : (dtype == AKG_F16 ? "f16" : "bf16"); }

struct Call {
  int op;
  const void* x; void* y;
  int64_t rows, cols, xs, ys;
  int dtype;
  const akg_mask* mask;
  const void* gamma; const void* beta;
  float eps;
  void* stream;
  int64_t row_base = 0;      // global index of row 0 (host-buffer chunks)
  float scale = 1.f;         // fused pre-scale of the softmax pair
};

akg_status validate(const Call& c, const char* name) {
  if (!valid_dtype(c.dtype)) return fail(AKG_ERR_INVALID_ARG, "%s: unknown dtype", name);
  if (c.rows < 0 || c.cols < 0) return fail(AKG_ERR_INVALID_ARG, "%s: negative rows or cols", name);
  const bool norm = (c.op == OP_LAYERNORM || c.op == OP_RMSNORM);
  if (norm && !(c.eps >= 0.f)) return fail(AKG_ERR_INVALID_ARG, "%s: eps must be >= 0 and not NaN", name);
  if (norm && std::isinf(c.eps)) return fail(AKG_ERR_INVALID_ARG, "%s: eps must be finite", name);
  if (c.mask != nullptr) {
    const akg_mask& m = *c.mask;
    if (m.causal != 0 && m.causal != 1) return fail(AKG_ERR_INVALID_ARG, "%s: mask.causal must be 0 or 1", name);
    if (m.causal && m.causal_period < 1) return fail(AKG_ERR_INVALID_ARG, "%s: mask.causal_period must be >= 1", name);
    if (m.additive != nullptr && (m.add_rows < 1 || m.add_row_stride < c.cols))
      return fail(AKG_ERR_INVALID_ARG, "%s: additive mask needs add_rows >= 1 and add_row_stride >= cols", name);
  }
  if (c.rows == 0 || c.cols == 0) return AKG_OK;
  if (c.x == nullptr || c.y == nullptr) return fail(AKG_ERR_INVALID_ARG, "%s: x and y must not be NULL", name);
  if (c.xs < c.cols || c.ys < c.cols) return fail(AKG_ERR_INVALID_ARG, "%s: row stride smaller than cols", name);
  if (c.cols > INT_MAX / 2) return fail(AKG_ERR_UNSUPPORTED, "%s: cols above 2^30 - 1", name);
  const int64_t es = (c.dtype == AKG_F32) ? 4 : 2;
  // extent of each matrix in bytes; reject anything that would overflow pointer arithmetic
  const long double lim = 9.0e18L;
  if (static_cast<long double>(c.rows) * c.xs * es > lim || static_cast<long double>(c.rows) * c.ys * es > lim)
    return fail(AKG_ERR_INVALID_ARG, "%s: rows * stride overflows", name);
  const uintptr_t x0 = reinterpret_cast<uintptr_t>(c.x), y0 = reinterpret_cast<uintptr_t>(c.y);
  const uintptr_t x1 = x0 + static_cast<uintptr_t>(((c.rows - 1) * c.xs + c.cols) * es);
  const uintptr_t y1 = y0 + static_cast<uintptr_t>(((c.rows - 1) * c.ys + c.cols) * es);
  const bool overlap = x0 < y1 && y0 < x1;
  if (overlap && !(x0 == y0 && c.xs == c.ys)) {
    // Two column windows of one buffer (x = buf[:, :cols], y = buf[:, cols:], equal strides, as in a
    // fused gate / up or q / k / v layout) interleave without sharing an element: with d the distance of
    // the bases modulo the row pitch, the windows are disjoint iff cols <= d and d + cols <= pitch.
    bool disjoint_windows = false;
    if (c.xs == c.ys) {
      const uintptr_t pitch = static_cast<uintptr_t>(c.xs * es), width = static_cast<uintptr_t>(c.cols * es);
      const uintptr_t d = (x0 > y0 ? x0 - y0 : y0 - x0) % pitch;
      disjoint_windows = d >= width && d + width <= pitch;
    }
    if (!disjoint_windows)
      return fail(AKG_ERR_INVALID_ARG, "%s: x and y overlap without being the same matrix", name);
  }
  return AKG_OK;
}

bool is_pow2(long long v) { return v > 0 && (v & (v - 1)) == 0; }

// SMs of the current device (cached per device; 148 if the query fails).
int sm_count() {
  static std::atomic<int> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 148; }
  int n = cache[dev].load();
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      n = 148;
    }
    cache[dev].store(n);
  }
  return n;
}

int pow2_ceil(int v) { int r = 1; while (r < v) r <<= 1; return r; }

// Can the vectorised families run this call?  (16-byte aligned rows and vectors.)
bool vector_ok(const Call& c) {
  const int64_t es = (c.dtype == AKG_F32) ? 4 : 2;
  const int64_t epv = 16 / es;
  if (c.cols % epv) return false;
  if (!aligned16(c.x) || !aligned16(c.y)) return false;
  if (c.rows > 1 && ((c.xs * es) % 16 || (c.ys * es) % 16)) return false;
  if (c.gamma && !aligned16(c.gamma)) return false;
  if (c.beta && !aligned16(c.beta)) return false;
  if (c.mask && c.mask->additive) {
    if (!aligned16(c.mask->additive)) return false;
    if (c.mask->add_rows > 1 && (c.mask->add_row_stride * es) % 16) return false;
  }
  return true;
}

// Register-resident plan, or false if the row does not fit.
bool plan_reg(const Call& c, LaunchPlan* plan) {
  const int64_t epv = (c.dtype == AKG_F32) ? 4 : 8;
  const int64_t nvec = c.cols / epv;
  int group = 0, vpt = 0, threads = 0, persist = 0;
  const int t_group = g_tune_reg_group.load(), t_threads = g_tune_reg_threads.load(), t_vpt = g_tune_reg_vpt.load();
  const bool many_rows = c.rows >= 4096;
  const bool want_warp = (t_group == 32) || (t_group == 0 && nvec <= 256 && many_rows);
  const bool norm_op = (c.op == OP_LAYERNORM || c.op == OP_RMSNORM);
  // normalisation rows of exactly 32 x (3, 5, 6, 7) vectors: a warp per row, predicate-free (fp32
  // 768 columns, 16-bit 768 and 1280 columns; more than 40 values per thread would spill)
  const int64_t per_lane = (nvec % 32 == 0) ? nvec / 32 : 0;
  const bool odd_warp_fit = want_warp && t_group == 0 && norm_op && g_tune_reg_general.load() == 0 &&
                            (per_lane == 3 || per_lane == 5 || per_lane == 6 || per_lane == 7) &&
                            (per_lane * epv <= 40 || per_lane == 7);   // 7: the alternative is 224 x 1
  if (odd_warp_fit) {
    group = 32; threads = 128; vpt = static_cast<int>(per_lane);
  } else if (want_warp && t_group == 0 && c.dtype != AKG_F32 && nvec > 128 && (c.op == OP_LAYERNORM || c.op == OP_RMSNORM)) {
    // 16-bit normalisation rows of 1025 .. 2048 columns: a warp per row would hold 64 values per
    // thread and spills (LayerNorm 58 % of the copy rate); a CTA of 128 threads per row measured
    // 70 - 75 % (RMSNorm 91 - 93 %); two warps per row and a packed-register variant were no better
    group = threads = 128; vpt = 2;
    // LayerNorm: grid-stride over 64 CTAs per SM measured 82 % against 71 % with a CTA per row
    if (c.op == OP_LAYERNORM) persist = sm_count() * 64;
  } else if (want_warp && t_group == 0 && c.dtype != AKG_F32 && nvec > 192 && !norm_op) {
    // the 16-bit softmax pair at 1544 .. 2048 columns: eight vectors per lane spill in the warp form
    // (2048 columns: 69 % softmax, 73 % log-softmax against 86 % and 80 % with a CTA of 128 per row)
    group = threads = 128; vpt = 2;
  } else if (want_warp && nvec <= 256 &&
             !(nvec == 192 && !norm_op && c.dtype != AKG_F32 && t_group == 0 && g_tune_reg_general.load() == 0 &&
               g_tune_reg_flex.load() != 2 && g_tune_reg_flex.load() != 5 &&
               (c.mask == nullptr || (c.mask->additive == nullptr && !c.mask->causal)))) {
    // (the unmasked 16-bit softmax pair at 1536 columns goes on to the packed kernel, 64 threads of three vectors:
    // log-softmax 0.82 -> 0.88, softmax 0.86 -> 0.86 against eight widened vectors per lane here)
    group = 32; threads = 128;
    vpt = pow2_ceil(static_cast<int>((nvec + 31) / 32));
  } else if (t_threads > 0 && t_vpt > 0) {
    group = threads = t_threads; vpt = t_vpt;
    if (static_cast<int64_t>(threads) * vpt < nvec) return false;
  } else {
    // widest vectors-per-thread of 4 until the CTA is full, then 8
    if (nvec <= 128) { threads = 128; vpt = 1; }
    else if (nvec <= 256) { threads = 128; vpt = 2; }
    else if (nvec <= 512) { threads = 128; vpt = 4; }
    else if (nvec <= 1024) { threads = 256; vpt = 4; }
    else if (nvec <= 2048 && c.dtype == AKG_F32 && !norm_op) { threads = 256; vpt = 8; }   // fp32 softmax pair: fat threads (5120 columns: 80 % against 71 % as 512 x 4)
    else if (nvec <= 2048) { threads = 512; vpt = 4; }
    else if (nvec <= 4096 && c.dtype == AKG_F32) { threads = 512; vpt = 8; }   // (16-bit rows beyond 2048 vectors: other families)
    else if (nvec <= 8192 && c.dtype == AKG_F32) { threads = 1024; vpt = 8; }
    else if (nvec <= 8192 && nvec % 8 == 0 && (nvec / 8) % 32 == 0 &&
             ((norm_op && c.dtype != AKG_F32) ||
              (!norm_op && (c.mask == nullptr || (c.mask->additive == nullptr && !c.mask->causal)))) &&
             g_tune_reg_general.load() == 0 && g_tune_reg_flex.load() != 2 && g_tune_reg_flex.load() != 5) {
      threads = static_cast<int>(nvec / 8); vpt = 8;     // only as the packed kernel, chosen below
    }
    else return false;
    group = threads;
  }
  const int64_t rpc = threads / group;          // rows per CTA iteration
  int64_t grid = (c.rows + rpc - 1) / rpc;
  int cap = g_tune_grid_cap.load();
  // the softmax pair runs persistent (two resident waves of CTAs, grid-stride over rows):
  // measured a little faster than one CTA per row, most under a causal mask
  // (the cap has to be a multiple of the CTAs resident at once, 1024 / threads per SM, fewer
  // where the kernel trades occupancy for registers: 2.67 waves measured 4 % slower than 2 or 4)
  if (cap == 0 && group == threads && (c.op == OP_SOFTMAX || c.op == OP_LOG_SOFTMAX)) {
    const int resident = (vpt == 4 && threads == 128) ? 6 : ((vpt == 4 || vpt == 8) && threads == 256) ? 3 : 1024 / threads;
    cap = sm_count() * 2 * resident;
  }
  if (cap == 0) cap = persist;
  if (cap > 0 && grid > cap) grid = cap;
  if (grid > INT_MAX) grid = INT_MAX;
  plan->variant = V_REG; plan->threads = threads; plan->group = group; plan->vpt = vpt;
  plan->grid = static_cast<unsigned>(grid); plan->cluster = 1; plan->smem = 0;
  // a row of exactly group * vpt vectors takes the predicate-free normalisation kernel
  plan->stages = (static_cast<int64_t>(group) * vpt == nvec && g_tune_reg_general.load() == 0) ? 1 : 0;
  // otherwise a normalisation row that splits exactly into (a multiple of 32 threads) x vpt
  // vectors takes the runtime-thread-count variant of it (e.g. 5120, 6144, 7168 columns)
  const bool norm = (c.op == OP_LAYERNORM || c.op == OP_RMSNORM);
  // (also preferred over the 512- and 1024-thread exact fits: fatter threads measured faster)
  if (norm && (plan->stages == 0 || threads >= 512 || g_tune_reg_flex.load() == 1) && group == threads &&
      g_tune_reg_general.load() == 0 &&
      !(t_threads > 0 && t_vpt > 0) && g_tune_reg_flex.load() != 2) {
    const int max_vpt = (c.dtype == AKG_F32) ? 8 : 4;
    int best_vpt = 0;
    int64_t best_g = 0;
    // 16-bit rows of 9216 .. 16384 columns: eight vectors per thread in a CTA of up to 256 fat threads
    // (128 registers) instead of 288 .. 512 threads of four
    // (RMSNorm: 12288 columns 69 -> 77 %, 14336: 72 -> 82 %, 16384: 82 % with the ring -> 86 %; LayerNorm level, not taken)
    if (c.dtype != AKG_F32 && c.op == OP_RMSNORM && g_tune_reg_flex.load() != 4 && nvec > 1024 && nvec % 8 == 0 &&
        (nvec / 8) % 32 == 0 && nvec / 8 <= 256) {
      best_vpt = 8; best_g = nvec / 8;
    }
    // fewer, fatter threads measured best (the per-row reduction is paid per thread): take
    // the largest vectors-per-thread that leaves at least 128 threads, else whatever fits
    // (one vector per thread only as a last resort: 1536 16-bit columns ran at 38 - 44 % as 192 x 1)
    for (int v = max_vpt; v >= 3 && best_vpt == 0; --v) {
      if (nvec % v) continue;
      const int64_t g = nvec / v;
      if (g % 32 == 0 && g >= 128 && g <= 1024) { best_vpt = v; best_g = g; }
    }
    for (int v = max_vpt; v >= 1 && best_vpt == 0; --v) {
      if (nvec % v) continue;
      const int64_t g = nvec / v;
      if (g % 32 == 0 && g >= 64 && g <= 1024) { best_vpt = v; best_g = g; }
    }
    if (best_vpt > 0) {
      plan->mode = 2; plan->threads = static_cast<int>(best_g); plan->group = plan->threads; plan->vpt = best_vpt;
      plan->grid = static_cast<unsigned>(c.rows > INT_MAX ? INT_MAX : c.rows);
      // 16-bit rows: grid-stride over 64 CTAs per SM (measured 2 - 12 % ahead of a CTA per row at
      // 1280 - 5120 columns; fp32 rows showed no consistent gain)
      const unsigned flex_cap = g_tune_grid_cap.load() > 0 ? static_cast<unsigned>(g_tune_grid_cap.load())
                                : (c.dtype != AKG_F32 ? static_cast<unsigned>(sm_count()) * 64u : 0u);
      if (flex_cap > 0 && plan->grid > flex_cap) plan->grid = flex_cap;
    }
  }
  // 16-bit normalisation rows with a CTA per row: the packed form of the runtime-thread-count kernel
  // (reg_norm_packed: the row stays packed in registers, eight vectors per thread fit 64 registers).  Measured
  // on bf16 rows of 2048 .. 16384 columns against everything above (fraction of the copy rate): LayerNorm
  // 0.73 - 0.95 -> 0.93 - 0.99, RMSNorm 0.79 - 0.98 (ring-fed: 0.91) -> 0.96 - 1.01.  Vectors per thread:
  // LayerNorm the most that leaves 64 threads (8192 columns: eight 0.95, four 0.88); RMSNorm four while that
  // keeps the CTA at 384 threads or fewer (8192 columns: four 1.01, eight 0.98), else the most (16384: eight
  // 0.97, four 0.89).
  // The unmasked softmax pair has a packed form too (reg_softmax_packed).
  const bool unmasked = c.mask == nullptr || (c.mask->additive == nullptr && !c.mask->causal);
  // ... and so has the unmasked fp32 softmax pair its runtime-thread-count form (reg_softmax_flex).
  if (((norm && c.dtype != AKG_F32) || (!norm && unmasked)) && group == threads && g_tune_reg_general.load() == 0 &&
      !(t_threads > 0 && t_vpt > 0) && g_tune_reg_flex.load() != 2 && g_tune_reg_flex.load() != 5) {
    const int want = g_tune_packed_vpt.load();
    int pv = 0;
    auto fits = [&](int v) {
      if (nvec % v) return false;
      const int64_t g = nvec / v;
      return g % 32 == 0 && g >= 64 && g <= 1024;
    };
    if (want > 0) { if (want >= 2 && want <= 8 && fits(want)) pv = want; }
    else if (c.op == OP_RMSNORM && fits(4) && nvec / 4 <= 384) pv = 4;
    else { for (int v = 8; v >= 2 && pv == 0; --v) if (fits(v)) pv = v; }
    if (pv > 0) {
      plan->mode = 3; plan->stages = 0; plan->vpt = pv; plan->threads = static_cast<int>(nvec / pv); plan->group = plan->threads;
      plan->grid = static_cast<unsigned>(c.rows > INT_MAX ? INT_MAX : c.rows);
      const unsigned pcap = g_tune_grid_cap.load() > 0 ? static_cast<unsigned>(g_tune_grid_cap.load())
                                                       : static_cast<unsigned>(sm_count()) * 64u;
      if (plan->grid > pcap) plan->grid = pcap;
    }
  }
  // (16-bit rows beyond 2048 vectors, and fp32 softmax rows beyond 4096, are in this family only in that form)
  if (plan->mode != 3 && ((c.dtype != AKG_F32 && nvec > 2048) || (c.dtype == AKG_F32 && !norm && nvec > 4096))) return false;
  return true;
}

// Register-resident cluster plan for the unmasked softmax pair: a cluster of cs CTAs per row, CTA k holding
// slice k of the row in registers (eight vectors per thread), the (maximum, sum) pairs exchanged through
// distributed shared memory.  Rows of exactly cs * threads * 8 vectors, threads a multiple of 32.  Among the
// cluster sizes that fit, the smallest whose CTAs have at most 512 threads (two CTAs per SM) and that gives
// the GPU two CTAs per SM; false if none fits.
bool plan_cluster_reg(const Call& c, LaunchPlan* plan) {
  if (c.op != OP_SOFTMAX && c.op != OP_LOG_SOFTMAX) return false;
  if (c.mask != nullptr && (c.mask->additive != nullptr || c.mask->causal)) return false;
  if (g_tune_reg_general.load() != 0 || g_tune_reg_flex.load() == 2 || g_tune_reg_flex.load() == 5) return false;
  const int64_t epv = (c.dtype == AKG_F32) ? 4 : 8;
  const int64_t nvec = c.cols / epv;
  const int t_cs = g_tune_cluster_size.load();
  int best = 0;
  for (int cs = 2; cs <= kMaxCluster; cs *= 2) {
    if (t_cs > 0 && cs != t_cs) continue;
    if (nvec % (cs * 8)) continue;
    const int64_t g = nvec / (cs * 8);
    if (g % 32 || g < 64 || g > 1024) continue;
    if (best == 0) best = cs;                               // the smallest that fits at all
    if (g <= 512 && (c.rows * cs >= 2 * static_cast<int64_t>(sm_count()) || cs == kMaxCluster)) { best = cs; break; }
    if (g <= 512) best = cs;
  }
  if (best == 0) return false;
  const int64_t clusters = std::min<int64_t>(c.rows, INT_MAX / best);
  plan->variant = V_REG; plan->mode = 3; plan->stages = 0; plan->vpt = 8; plan->cluster = best;
  plan->threads = static_cast<int>(nvec / (best * 8)); plan->group = plan->threads;
  plan->grid = static_cast<unsigned>(clusters * best); plan->smem = 0;
  return true;
}

// Shared-memory ring plan with a cluster of cs CTAs per row, cs_min <= cs <= cs_max
// (cs = 1 is the plain TMA ring).  Picks the smallest cluster whose slice leaves room
// for at least two ring buffers, else the smallest with one.  False if nothing fits.
bool plan_smem(const Call& c, int cs_min, int cs_max, LaunchPlan* plan, int want_threads = 0, int want_ctas = 0) {
  const int64_t epv = (c.dtype == AKG_F32) ? 4 : 8;
  const int64_t nvec = c.cols / epv;
  const int t_cs = g_tune_cluster_size.load(), t_nbuf = g_tune_smem_nbuf.load();
  const int t_threads = g_tune_smem_threads.load() > 0 ? g_tune_smem_threads.load() : want_threads;
  const int t_ctas = g_tune_smem_ctas.load() > 0 ? g_tune_smem_ctas.load() : want_ctas;
  if (t_cs > 0) {
    if (t_cs < cs_min || t_cs > cs_max) return false;
    cs_min = cs_max = t_cs;
  }
  int best_cs = 0, best_nbuf = 0, best_threads = 0;
  int64_t best_slice = 0;
  for (int want = 2; want >= 1 && best_cs == 0; --want) {
    for (int cs = cs_min; cs <= cs_max; cs *= 2) {
      const int64_t slice = (nvec + cs - 1) / cs;
      if (slice < 1) continue;
      int threads = t_threads > 0 ? t_threads : (slice <= 1024 ? 256 : (slice <= 8192 ? 512 : 1024));
      if (threads != 256 && threads != 512 && threads != 1024) return false;
      const int64_t buf = (slice * 16 + 127) & ~int64_t(127);
      // rows of up to 32 KiB share an SM between two CTAs so that one row's reduction
      // overlaps the other's copies and stores
      const int ctas = t_ctas > 0 ? t_ctas : ((cs == 1 && buf <= 32768) ? 2 : 1);
      const int64_t budget = static_cast<int64_t>(kMaxDynSmem) / ctas - (ctas > 1 ? 1024 : 0) -
                             smem_header_bytes(threads);
      int64_t nbuf = budget / buf;
      if (nbuf > kMaxBuf) nbuf = kMaxBuf;
      if (t_nbuf > 0 && nbuf > t_nbuf) nbuf = t_nbuf;
      if (nbuf >= want) { best_cs = cs; best_nbuf = static_cast<int>(nbuf); best_threads = threads; best_slice = slice; break; }
    }
  }
  if (best_cs == 0) return false;
  const int64_t buf = (best_slice * 16 + 127) & ~int64_t(127);
  plan->variant = (best_cs == 1) ? V_TMA : V_CLUSTER;
  // clusters, 1: partials exchanged under a cluster barrier; 2 (any cluster size): pipelined row loop
  plan->mode = (best_cs > 1 && g_tune_split_exchange.load() == 1) ? 1 : (g_tune_split_exchange.load() == 2 ? 2 : 0);
  plan->threads = best_threads; plan->group = best_threads; plan->vpt = static_cast<int>(best_slice);
  plan->cluster = best_cs; plan->stages = best_nbuf;
  plan->smem = smem_header_bytes(best_threads) + static_cast<size_t>(best_nbuf) * buf;
  const int cap = g_tune_grid_cap.load();
  plan->grid = cap > 0 ? static_cast<unsigned>((cap / best_cs > 0 ? cap / best_cs : 1) * best_cs) : 0u;
  return true;
}

// Ring-fed register plan: persistent CTAs, a CTA per row, the row prefetched by bulk
// copies into a shared-memory ring.  Normalisations need a row of exactly threads * vpt
// vectors; the softmax pair takes any row that fits.  False if the row does not fit.
bool plan_ring(const Call& c, LaunchPlan* plan) {
  const int64_t epv = (c.dtype == AKG_F32) ? 4 : 8;
  const int64_t nvec = c.cols / epv;
  const bool norm = (c.op == OP_LAYERNORM || c.op == OP_RMSNORM);
  const int t_threads = g_tune_reg_threads.load(), t_vpt = g_tune_reg_vpt.load();
  int threads = 0, vpt = 0;
  if (t_threads > 0 && t_vpt > 0) { threads = t_threads; vpt = t_vpt; }
  else if (nvec <= 128) { threads = 128; vpt = 1; }
  else if (nvec <= 256) { threads = 128; vpt = 2; }
  else if (nvec <= 512) { threads = 128; vpt = 4; }
  else if (nvec <= 1024) { threads = 256; vpt = 4; }
  else if (nvec <= 2048) { threads = 512; vpt = 4; }
  else return false;
  if (threads > 512 || vpt > 4 || static_cast<int64_t>(threads) * vpt < nvec) return false;
  if (norm && static_cast<int64_t>(threads) * vpt != nvec) return false;
  const int64_t buf = (nvec * 16 + 127) & ~int64_t(127);
  // size the ring so that the CTAs the register budget allows (1024 threads per SM) fit
  const int ctas = g_tune_smem_ctas.load() > 0 ? g_tune_smem_ctas.load() : (1024 / threads);
  int64_t nbuf = (static_cast<int64_t>(kMaxDynSmem) + 1024) / ctas - 1024 - 256 - 128;
  nbuf /= buf;
  if (nbuf > kMaxBuf) nbuf = kMaxBuf;
  const int t_nbuf = g_tune_smem_nbuf.load();
  if (t_nbuf > 0 && nbuf > t_nbuf) nbuf = t_nbuf;
  if (nbuf < 1) return false;
  plan->variant = V_TMA; plan->mode = 1; plan->threads = threads; plan->group = threads; plan->vpt = vpt;
  plan->cluster = 1; plan->stages = static_cast<int>(nbuf);
  plan->smem = 128 + static_cast<size_t>(nbuf) * buf;
  const int cap = g_tune_grid_cap.load();
  plan->grid = cap > 0 ? static_cast<unsigned>(cap) : 0u;
  return true;
}

// Two-pass split plan (cluster per row, second pass served by L2): any aligned row.
// The cluster is sized so that every SM gets work even when there are few rows.
bool plan_split(const Call& c, LaunchPlan* plan) {
  const int64_t epv = (c.dtype == AKG_F32) ? 4 : 8;
  const int64_t nvec = c.cols / epv;
  const int t_cs = g_tune_cluster_size.load(), t_threads = g_tune_smem_threads.load();
  const int threads = t_threads > 0 ? t_threads : 256;
  if (threads != 256 && threads != 512 && threads != 1024) return false;
  int cs = t_cs;
  if (cs == 0) {
    // slices of about 4096 vectors (16 per thread) measured best at every row length (65536 fp32
    // columns: 4 CTAs 82 %, 16 CTAs 45 % of the copy rate; 131072: 8 CTAs 84 %, 16 CTAs 64 %);
    // few rows take larger clusters so that there are about two CTAs per SM
    // (fp32 softmax pair and RMSNorm: slices of 1664 .. 3328 vectors instead.  Measured on 2^26 elements, fraction
    // of the copy rate with slices of 4000 - 5120 vectors against 2000 - 2560: 32000 columns 0.76 -> 0.89 - 0.92,
    // 40960: 0.73 -> 0.89 - 0.91, 65536: 0.76 -> 0.88 - 0.93, 81920: 0.75 -> 0.88 - 0.90; 98304 columns, where the
    // old rule already gave 3072, 0.89 - 0.91.  fp32 LayerNorm and the 16-bit types measured the other way round:
    // LayerNorm 65536 columns 0.79 with 4096, 0.76 with 2048; bf16 131072 columns 0.67 against 0.60.
    // What the large slices cost is L2 room: a resident CTA keeps its slice of the current row and of the next
    // one in L2 between the passes, 592 CTAs x 64 KB x 2 = 76 MB, and the second pass starts to miss (ncu, 65536
    // columns: L2 hit rate 20 % and 310 MB read from DRAM with 4096-vector slices, 42 % and 269 MB with 2048;
    // capping the grid at 448 CTAs brought the large slices from 0.77 to 0.85).)
    const bool small_slices = c.dtype == AKG_F32 && c.op != OP_LAYERNORM;
    // (16-bit log-softmax and normalisations: 2300 .. 4600, which moves 81920 and 151936 columns to half the slice:
    // bf16 81920 columns log-softmax 0.69 -> 0.73, LayerNorm 0.63 -> 0.71, RMSNorm 0.69 -> 0.80; 151936: 0.67 -> 0.71,
    // 0.59 -> 0.66, 0.65 -> 0.73; the 16-bit softmax measured level or worse with the smaller slices)
    // 16-bit RMSNorm and log-softmax take the small slices as well (bf16 131072 columns: RMSNorm 0.75 -> 0.80,
    // log-softmax 0.71 -> 0.74; 32000 columns log-softmax 0.73 -> 0.76), but no 16-bit operator gains from a
    // cluster of 16 with slices below 3072 vectors (only 31 such clusters fit the GPU, 496 of its 592 CTA slots:
    // bf16 262144 columns log-softmax 0.66 with 16 CTAs of 2048 vectors against 0.71 with 8 of 4096).
    const bool sixteen = c.dtype != AKG_F32;
    const int64_t min_next = (small_slices || (sixteen && (c.op == OP_RMSNORM || c.op == OP_LOG_SOFTMAX))) ? 1664
                             : ((sixteen && c.op == OP_LAYERNORM) ? 2300 : 3072);
    int by_len = 1, by_fill = 1;
    while (by_len < kMaxCluster &&
           nvec / (2 * by_len) >= ((sixteen && 2 * by_len == kMaxCluster) ? std::max<int64_t>(min_next, 3072) : min_next))
      by_len *= 2;
    if (c.dtype == AKG_F32 && c.op == OP_LAYERNORM && nvec > 4096 && nvec <= 8192) by_len = 2;   // see run()
    while (by_fill < kMaxCluster && c.rows * by_fill < 2 * static_cast<int64_t>(sm_count())) by_fill *= 2;
    cs = std::max(by_len, by_fill);
  }
  if (cs < 1 || cs > kMaxCluster || (cs & (cs - 1))) return false;
  while (cs > 1 && nvec / cs < threads) cs /= 2;          // keep at least one vector per thread
  plan->variant = V_CLUSTER; plan->threads = threads; plan->group = threads;
  // slices of one vector per thread more or less (a slice's ragged last step is predicated, so the
  // CTAs of a cluster get equal work: rounding to whole unrolled steps of four vectors per thread
  // gave 50304 fp32 columns slices of 4096 / 4096 / 4096 / 288 vectors)
  int64_t slice = (nvec + cs - 1) / cs;
  slice = (slice + threads - 1) / threads * threads;
  plan->vpt = static_cast<int>(slice);
  plan->cluster = cs; plan->stages = 0; plan->smem = 0;
  // mode 1: the partials are exchanged under a cluster barrier per row (the first version); otherwise
  // st.async + mbarrier
  plan->mode = g_tune_split_exchange.load() == 1 ? 1 : 0;
  plan->split_l2 = g_tune_split_l2.load();
  const int cap = g_tune_grid_cap.load();
  plan->grid = cap > 0 ? static_cast<unsigned>((cap / cs > 0 ? cap / cs : 1) * cs) : 0u;
  if (cap == 0) {
    // rows in flight must stay resident in L2 between the two passes: at most 64 MB of
    // them, but never fewer clusters than it takes to give every SM a CTA
    const int64_t row_bytes = c.cols * ((c.dtype == AKG_F32) ? 4 : 2);
    int64_t clusters = (int64_t(64) << 20) / (row_bytes > 0 ? row_bytes : 1);
    const int64_t floor_clusters = (160 + cs - 1) / cs;
    if (clusters < floor_clusters) clusters = floor_clusters;
    if (clusters < 4096) plan->grid = static_cast<unsigned>(clusters * cs);   // else: the launcher's own limit is lower
  }
  return true;
}

// Device address of the status word on the current device (cached per device).
int* status_word_ptr() {
  static std::atomic<int*> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  int* ptr = cache[dev].load();
  if (ptr == nullptr) {
    void* sym = nullptr;
    if (cudaGetSymbolAddress(&sym, g_status_word) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    ptr = static_cast<int*>(sym);
    cache[dev].store(ptr);
  }
  return ptr;
}

void plan_stream(const Call& c, LaunchPlan* plan) {
  int64_t grid = c.rows;
  const int cap = g_tune_grid_cap.load();
  if (cap > 0 && grid > cap) grid = cap;
  if (grid > INT_MAX) grid = INT_MAX;
  plan->variant = V_STREAM; plan->threads = 256; plan->group = 256; plan->vpt = 0;
  plan->grid = static_cast<unsigned>(grid); plan->cluster = 1; plan->stages = 0; plan->smem = 0;
}

akg_status run(const Call& c, const char* name) {
  t_error[0] = '\0';
  akg_status st = validate(c, name);
  if (st != AKG_OK) return st;
  if (c.rows == 0 || c.cols == 0) return AKG_OK;

  RowParams p;
  std::memset(&p, 0, sizeof p);
  p.x = c.x; p.y = c.y; p.rows = c.rows; p.cols = c.cols; p.xs = c.xs; p.ys = c.ys;
  p.gamma = c.gamma; p.beta = c.beta; p.eps = c.eps;
  p.period = 1;
  p.add_rows = 1;
  if (c.mask != nullptr) {
    p.add = c.mask->additive;
    if (p.add) {
      p.add_rows = c.mask->add_rows; p.add_stride = c.mask->add_row_stride;
      p.add_mode = (p.add_rows == 1) ? 1 : (p.add_rows >= c.rows ? 2 : 0);
    }
    p.causal = c.mask->causal;
    if (p.causal) {
      p.period = c.mask->causal_period; p.offset = c.mask->causal_offset;
      p.period_pow2 = is_pow2(p.period) ? 1 : 0;
      p.interleave = (p.period_pow2 && p.period >= 4 && c.rows % p.period == 0 &&
                      g_tune_interleave.load() == 1) ? 1 : 0;   // opt-in: measured slower than storage order
    }
  }
  p.status = nullptr;
  p.wait_us = g_tune_test_wait_us.load() > 0 ? static_cast<unsigned>(g_tune_test_wait_us.load()) : 0u;
  p.no_copies = g_tune_test_no_copies.load() == 1 ? 1 : 0;
  p.scale = c.scale; p.inv_scale = 1.0f / c.scale; p.l2e = kLog2e * c.scale;   // scale 1: exactly log2(e)
  p.row_base = c.row_base;
  if (c.row_base != 0) { p.interleave = 0; if (p.add_mode == 2) p.add_mode = 0; }

  const int forced = g_forced_variant.load();
  const bool vec = vector_ok(c);
  // Short rows without an additive mask (up to 64 vectors; normalisation rows below 128 vectors that are not a
  // multiple of a warp): several rows per warp and four vectors per lane, see kernels_short.cuh.
  if (forced == V_AUTO && vec && p.add == nullptr && g_tune_reg_general.load() == 0 &&
      g_tune_reg_group.load() == 0) {
    const int64_t nv = c.cols / ((c.dtype == AKG_F32) ? 4 : 8);
    const bool norm = (c.op == OP_LAYERNORM || c.op == OP_RMSNORM);
    // (the softmax pair also up to 128 vectors in the 16-bit types, 96 in fp32: bf16 1024 columns 96 %
    // of the copy rate against 72 % with a warp per row, fp32 320 columns 94 % against 87 %)
    // under the causal rule only up to 64 vectors: beyond, the warp-per-row kernel's skipping of
    // masked iterations is level or ahead (bf16 1024 columns: 67 % against 58 - 65 %)
    if (nv <= 64 || (norm && nv < 128 && nv % 32 != 0) ||
        (!norm && !p.causal && nv <= (c.dtype == AKG_F32 ? 96 : 128))) {
      int lanes = 4;
      while (lanes < 32 && short_max_vectors(lanes) < nv) lanes *= 2;
      const int64_t rpc = short_rows_per_cta(lanes);
      int64_t ctas = (c.rows + rpc - 1) / rpc;
      const int64_t cap = g_tune_grid_cap.load() > 0 ? g_tune_grid_cap.load() : static_cast<int64_t>(sm_count()) * 32;
      if (ctas > cap) ctas = cap;
      const cudaError_t e = launch_short(c.op, c.dtype, lanes, p, static_cast<unsigned>(ctas),
                                         g_tune_pdl.load() == 2 ? 0 : 1, static_cast<cudaStream_t>(c.stream));
      if (e != cudaSuccess) {
        (void)cudaGetLastError();
        std::snprintf(t_error, sizeof t_error, "%s: launch failed: %s", name, cudaGetErrorString(e));
        return AKG_ERR_CUDA;
      }
      std::snprintf(t_kernel, sizeof t_kernel, "short<%s,l%d,grid%u>", dtype_name(c.dtype), lanes,
                    static_cast<unsigned>(ctas));
      return AKG_OK;
    }
  }

  LaunchPlan plan;
  std::memset(&plan, 0, sizeof plan);
  bool planned = false;
  // Automatic choice (each rule is a measured preference on B200, see the profiles):
  //   every row that fits a CTA's registers -> register kernels (plan_reg; 16-bit rows without a mask in
  //     their packed form, up to 8192 vectors)
  //   longer aligned rows -> two-pass split cluster kernel (second pass from L2)
  //   anything unaligned -> scalar stream kernel
  // (the ring-fed register kernels are no automatic choice any more: bf16 RMSNorm with many rows, their one
  // case, runs at 0.91 - 0.96 of the copy rate through the ring and at 0.98 - 1.01 in the packed register
  // kernel; forcing the TMA family still reaches them)
  // (the kernel that keeps a row in shared memory is no automatic choice either: its best case, 16-bit
  // log-softmax rows of 32 - 40 KB with three CTAs of 256 threads per SM, measured 0.79 - 0.85 of the copy rate
  // against 0.69 - 0.78 in the widened register / two-pass kernels, and 0.96 - 1.0 in the packed register kernel)
  // rows beyond 2048 vectors in the 16-bit types (beyond 4096 for the fp32 softmax pair) measured
  // faster in the two-pass kernel than in one CTA of 640 - 1024 threads: bf16 32768 columns 77 - 79 %
  // against 63 %, fp32 softmax 32768 columns 81 % against 77 % (fp32 normalisations: 82 % against 93 %, kept)
  const int64_t row_vecs = c.cols / ((c.dtype == AKG_F32) ? 4 : 8);
  // (unmasked 16-bit rows stay in registers up to 8192 vectors where the packed kernels fit them: bf16
  // 20480 - 32768 columns LayerNorm 0.86 - 0.92 against 0.74 - 0.77 in the two-pass kernel, RMSNorm 0.94 - 0.96
  // against 0.64 - 0.85 with the row in shared memory, softmax 0.95 - 0.99 against 0.70, log-softmax 0.96
  // against 0.72; 65536 columns 0.71 / 0.85 / 0.70 / 0.72 against 0.69 / 0.75 / 0.69 / 0.71)
  const bool norm_call = c.op == OP_LAYERNORM || c.op == OP_RMSNORM;
  const bool packed_fits = row_vecs <= 8192 &&
                           ((norm_call && c.dtype != AKG_F32) ||
                            (!norm_call && (c.mask == nullptr || (c.mask->additive == nullptr && !c.mask->causal)))) &&
                           row_vecs % 8 == 0 && (row_vecs / 8) % 32 == 0 && g_tune_reg_general.load() == 0 &&
                           !(c.dtype == AKG_F32 && row_vecs > 4096) &&                        // see long_row
                           g_tune_reg_flex.load() != 2 && g_tune_reg_flex.load() != 5 &&
                           // a CTA per row needs rows for about a full wave of threads; fewer rows are cut into
                           // slices by the two-pass cluster kernel
                           c.rows * (row_vecs / 8) >= static_cast<int64_t>(sm_count()) * 1024;
  // (fp32 rows of 4097 .. 6143 vectors would take one CTA of 544 .. 736 fat threads per SM: 20480 columns measured
  // 0.81 - 0.83 there and 0.91 - 0.93 in the two-pass kernel for the softmax pair and RMSNorm; LayerNorm 0.82 against
  // 0.79 and stays; from 6144 vectors on RMSNorm is level in both; the fp32 softmax pair, with its slices sized
  // for L2, is level at 24576 columns and ahead beyond - 28672: 0.91 against 0.90, 32768: 0.95 against 0.92 - so
  // every fp32 softmax row beyond 4096 vectors takes the two-pass kernel)
  const bool thin_cta = c.dtype == AKG_F32 && row_vecs > 4096 && row_vecs < 6144 && c.op != OP_LAYERNORM &&
                        g_tune_reg_flex.load() != 1;
  // (fp32 LayerNorm rows of 4097 .. 8192 vectors, given rows enough to matter: two CTAs of a cluster per row
  // measured 0.83 - 0.87 against 0.79 - 0.83 in one CTA of 576 - 1024 threads; with a few hundred rows the
  // register kernel stays ahead, 0.49 - 0.51 against 0.41 - 0.50)
  const bool ln_two_ctas = c.dtype == AKG_F32 && c.op == OP_LAYERNORM && row_vecs > 4096 && row_vecs <= 8192 &&
                           c.rows >= 1024 && g_tune_reg_flex.load() != 1;
  const bool long_row = forced == V_AUTO && g_tune_cluster_mode.load() != 1 && !packed_fits &&
                        ((c.dtype != AKG_F32 && row_vecs > 2048) || thin_cta || ln_two_ctas ||
                         (c.dtype == AKG_F32 && row_vecs > 4096 && (c.op == OP_SOFTMAX || c.op == OP_LOG_SOFTMAX)));
  // Unmasked softmax rows too long for one CTA's registers, held in the registers of a cluster instead
  // (cluster_mode 3).  Not an automatic choice: one row at a time per CTA leaves the exchange of the pairs
  // exposed (configuration 4: 150 us with 16 CTAs of 512 threads against 95 us in the two-pass kernel, which
  // overlaps the second pass of a row with the first pass of the next; 131072 fp32 columns 0.65 against 0.78).
  // (asked for with a forced cluster size, it also takes rows that one CTA could hold)
  if (!planned && vec && forced == V_AUTO && g_tune_cluster_mode.load() == 3 &&
      (g_tune_cluster_size.load() > 1 || long_row || row_vecs > 8192)) {
    planned = plan_cluster_reg(c, &plan);
    if (planned) p.status = status_word_ptr();
  }
  if (!planned && (forced == V_AUTO || forced == V_REG) && vec && !long_row) {
    planned = plan_reg(c, &plan);
    // fp32 normalisation rows beyond 4096 vectors stay in registers only as an exact fit (the ragged
    // 1024-thread form measured 49 % on 32000 columns)
    if (planned && forced == V_AUTO && g_tune_cluster_mode.load() != 1 && c.dtype == AKG_F32 && row_vecs > 4096 &&
        plan.mode != 2 && plan.mode != 3 && plan.stages != 1) {
      planned = false;
      plan = LaunchPlan{};
    }
  }
  if (!planned && vec) {
    if (forced == V_AUTO) planned = (g_tune_cluster_mode.load() == 1) ? plan_smem(c, 1, kMaxCluster, &plan)
                                                                      : plan_split(c, &plan);
    else if (forced == V_TMA)
      planned = (g_tune_tma_mode.load() != 2 && plan_ring(c, &plan)) || plan_smem(c, 1, 1, &plan);
    else if (forced == V_CLUSTER)
      planned = (g_tune_cluster_mode.load() == 2) ? plan_split(c, &plan) : plan_smem(c, 2, kMaxCluster, &plan);
    if (planned) p.status = status_word_ptr();
  }
  if (!planned && (forced == V_AUTO || forced == V_STREAM)) { plan_stream(c, &plan); planned = true; }
  if (!planned) return fail(AKG_ERR_UNSUPPORTED, "%s: the forced kernel family cannot run this call", name);

  cudaStream_t stream = static_cast<cudaStream_t>(c.stream);
  // programmatic dependent launch hides the launch gap of back-to-back calls; cluster
  // launches measured slower with it (dependent clusters take SMs from the tail), so not there
  plan.pdl = (g_tune_pdl.load() == 2 || ((plan.variant == V_CLUSTER || plan.cluster > 1) && g_tune_pdl.load() != 1)) ? 0 : 1;
  cudaError_t err;
  switch (c.op) {
    case OP_SOFTMAX: err = launch_op<OP_SOFTMAX>(plan, c.dtype, p, stream); break;
    case OP_LOG_SOFTMAX: err = launch_op<OP_LOG_SOFTMAX>(plan, c.dtype, p, stream); break;
    case OP_LAYERNORM: err = launch_op<OP_LAYERNORM>(plan, c.dtype, p, stream); break;
    default: err = launch_op<OP_RMSNORM>(plan, c.dtype, p, stream); break;
  }
  if (err != cudaSuccess) {
    (void)cudaGetLastError();
    std::snprintf(t_error, sizeof t_error, "%s: launch failed: %s", name, cudaGetErrorString(err));
    return AKG_ERR_CUDA;
  }
  const char* dt = dtype_name(c.dtype);
  if (plan.variant == V_REG)
    std::snprintf(t_kernel, sizeof t_kernel, "reg<%s,g%d,t%d,v%d%s%s>", dt, plan.group, plan.threads, plan.vpt,
                  plan.cluster == 16 ? ",cs16" : plan.cluster == 8 ? ",cs8" : plan.cluster == 4 ? ",cs4" : plan.cluster == 2 ? ",cs2" : "",
                  plan.mode == 3 ? (c.dtype == AKG_F32 ? ",flex" : ",packed") : plan.mode == 2 ? ",flex"
                                 : ((plan.stages == 1 && (c.op == OP_LAYERNORM || c.op == OP_RMSNORM)) ? ",full" : ""));
  else if (plan.variant == V_TMA || plan.variant == V_CLUSTER)
    std::snprintf(t_kernel, sizeof t_kernel, "%s<%s,t%d,cs%d,nbuf%d,slice%d>",
                  plan.variant == V_TMA ? (plan.mode == 1 ? "ring" : "tma")
                  : (plan.stages != 0 ? "cluster" : "split"),
                  dt, plan.threads,
                  plan.cluster, plan.stages, plan.vpt);
  else
    std::snprintf(t_kernel, sizeof t_kernel, "stream<%s,t%d>", dt, plan.threads);
  return AKG_OK;
}

// ---- host-buffer pipeline ------------------------------------------------------------
// Three internal streams per device, each owning one slot of the caller's workspace:
// chunk i goes host -> slot (i % 3) -> kernel in place -> host on stream (i % 3), so the
// copy engines (both directions) and the SMs work on different chunks at the same time.
constexpr int kHostSlots = 3;
struct HostPipe {
  cudaStream_t s[kHostSlots];
  cudaEvent_t done[kHostSlots];
  cudaEvent_t start, vectors;
  bool ready = false;
};
std::mutex g_pipe_mu;
HostPipe g_pipes[64];

akg_status cuda_fail(const char* name, cudaError_t err) {
  (void)cudaGetLastError();
  std::snprintf(t_error, sizeof t_error, "%s: %s", name, cudaGetErrorString(err));
  return AKG_ERR_CUDA;
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t host_vector_bytes(int64_t cols, int dtype, bool gamma, bool beta) {
  const size_t one = round_up(static_cast<size_t>(cols) * ((dtype == AKG_F32) ? 4 : 2), 256);
  return one * ((gamma ? 1 : 0) + (beta ? 1 : 0));
}

akg_status run_host(const Call& hc, const char* name, void* workspace, size_t ws_bytes) {
  t_error[0] = '\0';
  akg_status st = validate(hc, name);              // same rules; the pointers are host pointers here
  if (st != AKG_OK) return st;
  if (hc.rows == 0 || hc.cols == 0) return AKG_OK;
  if (hc.mask != nullptr && hc.mask->additive != nullptr)
    return fail(AKG_ERR_UNSUPPORTED, "%s: an additive mask is not supported with host buffers", name);
  if (workspace == nullptr || !aligned16(workspace))
    return fail(AKG_ERR_INVALID_ARG, "%s: workspace must be a 16-byte aligned device pointer", name);
  const size_t es = (hc.dtype == AKG_F32) ? 4 : 2;
  const size_t row_bytes = static_cast<size_t>(hc.cols) * es;
  const size_t vec_bytes = host_vector_bytes(hc.cols, hc.dtype, hc.gamma != nullptr, hc.beta != nullptr);
  if (ws_bytes < vec_bytes + kHostSlots * round_up(row_bytes, 256))
    return fail(AKG_ERR_INVALID_ARG, "%s: workspace too small (see akg_host_workspace_bytes)", name);
  const size_t slot_bytes = ((ws_bytes - vec_bytes) / kHostSlots) & ~static_cast<size_t>(255);
  int64_t chunk_rows = static_cast<int64_t>(slot_bytes / row_bytes);
  // about a dozen chunks so the pipeline fills, but no chunk under 4 MiB (copy efficiency)
  const int64_t nchunks = g_tune_host_chunks.load() > 0 ? g_tune_host_chunks.load() : 12;
  const size_t min_bytes = g_tune_host_min_kib.load() > 0 ? (size_t(g_tune_host_min_kib.load()) << 10) : (size_t(4) << 20);
  int64_t want = (hc.rows + nchunks - 1) / nchunks;
  const int64_t min_rows = static_cast<int64_t>((min_bytes + row_bytes - 1) / row_bytes);
  if (want < min_rows) want = min_rows;
  if (chunk_rows > want) chunk_rows = want;
  // Under a causal mask the kernels never read a row's masked columns, so they are not uploaded either: a
  // chunk that lies inside one causal period needs the columns up to its last row's live length only.  For
  // that, chunks are made a quarter of a period at most (while that is still min_rows or more) and are cut
  // at the period's boundaries.  (Configuration 5: 0.63 GiB instead of 1 GiB per upload.)
  const bool causal = hc.mask != nullptr && hc.mask->causal != 0 && g_tune_host_full_upload.load() == 0;
  const int64_t period = causal ? hc.mask->causal_period : 0;
  if (causal && period / 4 >= min_rows && chunk_rows > period / 4) chunk_rows = period / 4;
  if (chunk_rows < 1) chunk_rows = 1;
  // The first and the last chunks are smaller (an eighth, a quarter, a half of a chunk): the upload of the
  // first chunk and the download of the last one are the only copies nothing else overlaps.
  // (only while the smallest pieces stay at a quarter of the smallest chunk, a megabyte: with pieces of 0.7 MB
  // configuration 2 measured 1.81 ms against 1.77 ms without the ramp)
  const bool ramp = g_tune_host_chunks.load() == 0 && hc.rows >= 6 * chunk_rows && chunk_rows / 8 >= min_rows / 4 &&
                    chunk_rows >= 8;

  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return cuda_fail(name, err);
  if (dev < 0 || dev >= 64) return fail(AKG_ERR_UNSUPPORTED, "%s: device index above 63", name);
  std::lock_guard<std::mutex> lock(g_pipe_mu);
  HostPipe& pipe = g_pipes[dev];
  if (!pipe.ready) {
    for (int k = 0; k < kHostSlots; ++k) {
      if ((err = cudaStreamCreateWithFlags(&pipe.s[k], cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(name, err);
      if ((err = cudaEventCreateWithFlags(&pipe.done[k], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(name, err);
    }
    if ((err = cudaEventCreateWithFlags(&pipe.start, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(name, err);
    if ((err = cudaEventCreateWithFlags(&pipe.vectors, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(name, err);
    pipe.ready = true;
  }
  cudaStream_t user = static_cast<cudaStream_t>(hc.stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  void* d_gamma = nullptr;
  void* d_beta = nullptr;
  size_t off = 0;
  if ((err = cudaEventRecord(pipe.start, user)) != cudaSuccess) return cuda_fail(name, err);
  for (int k = 0; k < kHostSlots; ++k)
    if ((err = cudaStreamWaitEvent(pipe.s[k], pipe.start, 0)) != cudaSuccess) return cuda_fail(name, err);
  if (hc.gamma != nullptr) {
    d_gamma = ws + off; off += round_up(row_bytes, 256);
    if ((err = cudaMemcpyAsync(d_gamma, hc.gamma, row_bytes, cudaMemcpyHostToDevice, pipe.s[0])) != cudaSuccess) return cuda_fail(name, err);
  }
  if (hc.beta != nullptr) {
    d_beta = ws + off; off += round_up(row_bytes, 256);
    if ((err = cudaMemcpyAsync(d_beta, hc.beta, row_bytes, cudaMemcpyHostToDevice, pipe.s[0])) != cudaSuccess) return cuda_fail(name, err);
  }
  if (off > 0) {
    if ((err = cudaEventRecord(pipe.vectors, pipe.s[0])) != cudaSuccess) return cuda_fail(name, err);
    for (int k = 1; k < kHostSlots; ++k)
      if ((err = cudaStreamWaitEvent(pipe.s[k], pipe.vectors, 0)) != cudaSuccess) return cuda_fail(name, err);
  }
  const unsigned char* hx = static_cast<const unsigned char*>(hc.x);
  unsigned char* hy = static_cast<unsigned char*>(hc.y);
  int64_t chunk = 0;
  size_t up_bytes = vec_bytes ? row_bytes * ((hc.gamma != nullptr) + (hc.beta != nullptr)) : 0, down_bytes = 0;
  for (int64_t r0 = 0; r0 < hc.rows; ++chunk) {
    const int k = static_cast<int>(chunk % kHostSlots);
    int64_t n = chunk_rows;
    if (ramp) {                                             // 1/8, 1/8, 1/4, 1/2 of a chunk at either end
      const int64_t left = hc.rows - r0;
      const int64_t head = chunk < 2 ? 8 : (chunk == 2 ? 4 : (chunk == 3 ? 2 : 1));
      n = chunk_rows / head;
      if (left <= chunk_rows / 4) n = std::min<int64_t>(n, (chunk_rows + 7) / 8);
      else if (left <= chunk_rows / 2 + chunk_rows / 4) n = std::min<int64_t>(n, chunk_rows / 4);
      else if (left <= chunk_rows + chunk_rows / 2 + chunk_rows / 4) n = std::min<int64_t>(n, chunk_rows / 2);
    }
    if (n > hc.rows - r0) n = hc.rows - r0;
    size_t up_width = row_bytes;                            // bytes of every row that are uploaded
    if (causal) {
      const int64_t in_period = r0 % period;
      if (in_period + n > period) n = period - in_period;  // a chunk does not cross a period
      const int64_t live = std::max<int64_t>(0, std::min<int64_t>(hc.cols, in_period + n + hc.mask->causal_offset));
      up_width = round_up(static_cast<size_t>(live) * es, 16);
      if (up_width > row_bytes) up_width = row_bytes;
    }
    unsigned char* slot = ws + vec_bytes + static_cast<size_t>(k) * slot_bytes;
    if (up_width == 0) {
      err = cudaSuccess;                                    // every row of the chunk is wholly masked
    } else if (hc.xs == hc.cols && up_width == row_bytes) {
      err = cudaMemcpyAsync(slot, hx + static_cast<size_t>(r0) * row_bytes, static_cast<size_t>(n) * row_bytes,
                            cudaMemcpyHostToDevice, pipe.s[k]);
    } else {
      err = cudaMemcpy2DAsync(slot, row_bytes, hx + static_cast<size_t>(r0) * hc.xs * es, static_cast<size_t>(hc.xs) * es,
                              up_width, static_cast<size_t>(n), cudaMemcpyHostToDevice, pipe.s[k]);
    }
    if (err != cudaSuccess) return cuda_fail(name, err);
    up_bytes += up_width * static_cast<size_t>(n);
    Call dc = hc;
    dc.x = slot; dc.y = slot; dc.rows = n; dc.xs = hc.cols; dc.ys = hc.cols;
    dc.gamma = d_gamma; dc.beta = d_beta; dc.stream = pipe.s[k]; dc.row_base = r0;
    st = run(dc, name);
    if (st != AKG_OK) return st;
    if (hc.ys == hc.cols)
      err = cudaMemcpyAsync(hy + static_cast<size_t>(r0) * row_bytes, slot, static_cast<size_t>(n) * row_bytes,
                            cudaMemcpyDeviceToHost, pipe.s[k]);
    else
      err = cudaMemcpy2DAsync(hy + static_cast<size_t>(r0) * hc.ys * es, static_cast<size_t>(hc.ys) * es, slot, row_bytes,
                              row_bytes, static_cast<size_t>(n), cudaMemcpyDeviceToHost, pipe.s[k]);
    if (err != cudaSuccess) return cuda_fail(name, err);
    down_bytes += row_bytes * static_cast<size_t>(n);
    r0 += n;
  }
  t_host_up = up_bytes;
  t_host_down = down_bytes;
  for (int k = 0; k < kHostSlots; ++k) {
    if ((err = cudaEventRecord(pipe.done[k], pipe.s[k])) != cudaSuccess) return cuda_fail(name, err);
    if ((err = cudaStreamWaitEvent(user, pipe.done[k], 0)) != cudaSuccess) return cuda_fail(name, err);
  }
  return AKG_OK;
}

}  // namespace
}  // namespace akg

using namespace akg;

extern "C" {

akg_status akg_softmax(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                       int64_t y_row_stride, akg_dtype dtype, const akg_mask* mask, void* stream) {
  Call c{OP_SOFTMAX, x, y, rows, cols, x_row_stride, y_row_stride, static_cast<int>(dtype), mask,
         nullptr, nullptr, 0.f, stream};
  return run(c, "akg_softmax");
}

akg_status akg_log_softmax(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                           int64_t y_row_stride, akg_dtype dtype, const akg_mask* mask, void* stream) {
  Call c{OP_LOG_SOFTMAX, x, y, rows, cols, x_row_stride, y_row_stride, static_cast<int>(dtype), mask,
         nullptr, nullptr, 0.f, stream};
  return run(c, "akg_log_softmax");
}

akg_status akg_layernorm(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                         int64_t y_row_stride, akg_dtype dtype, const void* gamma, const void* beta,
                         float eps, void* stream) {
  Call c{OP_LAYERNORM, x, y, rows, cols, x_row_stride, y_row_stride, static_cast<int>(dtype), nullptr,
         gamma, beta, eps, stream};
  return run(c, "akg_layernorm");
}

akg_status akg_rmsnorm(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                       int64_t y_row_stride, akg_dtype dtype, const void* weight, float eps, void* stream) {
  Call c{OP_RMSNORM, x, y, rows, cols, x_row_stride, y_row_stride, static_cast<int>(dtype), nullptr,
         weight, nullptr, eps, stream};
  return run(c, "akg_rmsnorm");
}

akg_status akg_rowop_host(akg_op op, const void* x_host, void* y_host, int64_t rows, int64_t cols,
                          int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype, const void* gamma_host,
                          const void* beta_host, float eps, const akg_mask* mask, void* workspace,
                          size_t workspace_bytes, void* stream) {
  if (op < AKG_OP_SOFTMAX || op > AKG_OP_RMSNORM)
    return fail(AKG_ERR_INVALID_ARG, "%s: unknown operator", "akg_rowop_host");
  const bool softmax_like = (op == AKG_OP_SOFTMAX || op == AKG_OP_LOG_SOFTMAX);
  Call c{static_cast<int>(op), x_host, y_host, rows, cols, x_row_stride, y_row_stride, static_cast<int>(dtype),
         softmax_like ? mask : nullptr, softmax_like ? nullptr : gamma_host,
         op == AKG_OP_LAYERNORM ? beta_host : nullptr, softmax_like ? 0.f : eps, stream};
  return run_host(c, "akg_rowop_host", workspace, workspace_bytes);
}

size_t akg_host_workspace_bytes(int64_t rows, int64_t cols, akg_dtype dtype, int has_gamma, int has_beta) {
  if (rows <= 0 || cols <= 0 || !valid_dtype(dtype)) return 0;
  const size_t row_bytes = static_cast<size_t>(cols) * ((dtype == AKG_F32) ? 4 : 2);
  size_t chunk_rows = (static_cast<size_t>(rows) + 11) / 12;
  const size_t min_rows = ((size_t(4) << 20) + row_bytes - 1) / row_bytes;
  if (chunk_rows < min_rows) chunk_rows = min_rows;
  if (chunk_rows > static_cast<size_t>(rows)) chunk_rows = static_cast<size_t>(rows);
  return host_vector_bytes(cols, dtype, has_gamma != 0, has_beta != 0) +
         kHostSlots * round_up(chunk_rows * row_bytes, 256);
}

const char* akg_status_string(akg_status status) {
  switch (status) {
    case AKG_OK: return "AKG_OK";
    case AKG_ERR_INVALID_ARG: return "AKG_ERR_INVALID_ARG";
    case AKG_ERR_UNSUPPORTED: return "AKG_ERR_UNSUPPORTED";
    case AKG_ERR_CUDA: return "AKG_ERR_CUDA";
    case AKG_ERR_DEVICE_TIMEOUT: return "AKG_ERR_DEVICE_TIMEOUT";
  }
  return "AKG_ERR_UNKNOWN";
}

const char* akg_last_error_string(void) { return t_error; }

int akg_version(void) { return 100; }

akg_status akg_set_variant(akg_variant variant) {
  if (variant < AKG_VARIANT_AUTO || variant > AKG_VARIANT_CLUSTER)
    return fail(AKG_ERR_INVALID_ARG, "%s: unknown variant", "akg_set_variant");
  g_forced_variant.store(static_cast<int>(variant));
  return AKG_OK;
}

akg_status akg_set_tuning(const char* key, int value) {
  if (key == nullptr) return fail(AKG_ERR_INVALID_ARG, "%s: NULL key", "akg_set_tuning");
  if (!std::strcmp(key, "reg_threads")) g_tune_reg_threads.store(value);
  else if (!std::strcmp(key, "reg_vpt")) g_tune_reg_vpt.store(value);
  else if (!std::strcmp(key, "reg_group")) g_tune_reg_group.store(value);
  else if (!std::strcmp(key, "grid_cap")) g_tune_grid_cap.store(value);
  else if (!std::strcmp(key, "cluster_size")) g_tune_cluster_size.store(value);
  else if (!std::strcmp(key, "smem_nbuf")) g_tune_smem_nbuf.store(value);
  else if (!std::strcmp(key, "smem_threads")) g_tune_smem_threads.store(value);
  else if (!std::strcmp(key, "smem_ctas")) g_tune_smem_ctas.store(value);
  else if (!std::strcmp(key, "reg_general")) g_tune_reg_general.store(value);
  else if (!std::strcmp(key, "cluster_mode")) g_tune_cluster_mode.store(value);
  else if (!std::strcmp(key, "tma_mode")) g_tune_tma_mode.store(value);
  else if (!std::strcmp(key, "interleave")) g_tune_interleave.store(value);
  else if (!std::strcmp(key, "pdl")) g_tune_pdl.store(value);
  else if (!std::strcmp(key, "reg_flex")) g_tune_reg_flex.store(value);
  else if (!std::strcmp(key, "packed_vpt")) g_tune_packed_vpt.store(value);
  else if (!std::strcmp(key, "host_chunks")) g_tune_host_chunks.store(value);
  else if (!std::strcmp(key, "host_min_kib")) g_tune_host_min_kib.store(value);
  else if (!std::strcmp(key, "host_full_upload")) g_tune_host_full_upload.store(value);
  else if (!std::strcmp(key, "axis_r")) g_tune_axis_r.store(value);
  else if (!std::strcmp(key, "axis_nc")) g_tune_axis_nc.store(value);
  else if (!std::strcmp(key, "axis_mode")) g_tune_axis_mode.store(value);
  else if (!std::strcmp(key, "axis_lc")) g_tune_axis_lc.store(value);
  else if (!std::strcmp(key, "split_exchange")) g_tune_split_exchange.store(value);
  else if (!std::strcmp(key, "split_l2")) g_tune_split_l2.store(value);
  else if (!std::strcmp(key, "test_wait_us")) g_tune_test_wait_us.store(value);
  else if (!std::strcmp(key, "test_no_copies")) g_tune_test_no_copies.store(value);
  else return fail(AKG_ERR_INVALID_ARG, "akg_set_tuning: unknown key %s", key);
  return AKG_OK;
}

const char* akg_last_kernel_name(void) { return t_kernel; }

akg_status akg_last_host_copy_bytes(size_t* h2d_bytes, size_t* d2h_bytes) {
  if (h2d_bytes != nullptr) *h2d_bytes = t_host_up;
  if (d2h_bytes != nullptr) *d2h_bytes = t_host_down;
  return AKG_OK;
}

akg_status akg_device_status(int* word_out) {
  int word = 0;
  cudaError_t err = cudaMemcpyFromSymbol(&word, g_status_word, sizeof(int));
  if (err == cudaSuccess && word != 0) {
    const int zero = 0;
    err = cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int));
  }
  if (err != cudaSuccess) {
    (void)cudaGetLastError();
    return fail(AKG_ERR_CUDA, "akg_device_status: %s", cudaGetErrorString(err));
  }
  if (word_out) *word_out = word;
  return word == 0 ? AKG_OK : AKG_ERR_DEVICE_TIMEOUT;
}

}  // extern "C"

// ---- operators over a non-last axis ----------------------------------------------------------
extern "C" akg_status akg_rowop_axis(akg_op op, const void* x, void* y, int64_t outer, int64_t reduce,
                                     int64_t inner, int64_t x_outer_stride, int64_t x_reduce_stride,
                                     int64_t y_outer_stride, int64_t y_reduce_stride, akg_dtype dtype,
                                     const void* gamma, const void* beta, float eps, void* stream) {
  const char* name = "akg_rowop_axis";
  akg::t_error[0] = '\0';
  if (op < AKG_OP_SOFTMAX || op > AKG_OP_RMSNORM) return akg::fail(AKG_ERR_INVALID_ARG, "%s: unknown operator", name);
  if (!valid_dtype(dtype)) return akg::fail(AKG_ERR_INVALID_ARG, "%s: unknown dtype", name);
  if (outer < 0 || reduce < 0 || inner < 0) return akg::fail(AKG_ERR_INVALID_ARG, "%s: negative size", name);
  const bool norm = (op == AKG_OP_LAYERNORM || op == AKG_OP_RMSNORM);
  if (norm && (!(eps >= 0.f) || std::isinf(eps)))
    return akg::fail(AKG_ERR_INVALID_ARG, "%s: eps must be finite and >= 0", name);
  if (outer == 0 || reduce == 0 || inner == 0) return AKG_OK;
  if (x == nullptr || y == nullptr) return akg::fail(AKG_ERR_INVALID_ARG, "%s: x and y must not be NULL", name);
  if (x_reduce_stride < inner || y_reduce_stride < inner)
    return akg::fail(AKG_ERR_INVALID_ARG, "%s: reduce stride smaller than inner", name);
  const long double span_x = static_cast<long double>(reduce - 1) * x_reduce_stride + inner;
  const long double span_y = static_cast<long double>(reduce - 1) * y_reduce_stride + inner;
  if (x_outer_stride < span_x || y_outer_stride < span_y)
    return akg::fail(AKG_ERR_INVALID_ARG, "%s: outer stride smaller than one [reduce, inner] slab", name);
  const int64_t es = (dtype == AKG_F32) ? 4 : 2;
  if (static_cast<long double>(outer) * x_outer_stride * es > 9.0e18L ||
      static_cast<long double>(outer) * y_outer_stride * es > 9.0e18L)
    return akg::fail(AKG_ERR_INVALID_ARG, "%s: outer * stride overflows", name);
  if (reduce > INT_MAX / 2 || inner > (int64_t(1) << 40))
    return akg::fail(AKG_ERR_UNSUPPORTED, "%s: reduce above 2^30 - 1 or inner above 2^40", name);
  const uintptr_t x0 = reinterpret_cast<uintptr_t>(x), y0 = reinterpret_cast<uintptr_t>(y);
  const uintptr_t x1 = x0 + static_cast<uintptr_t>(((outer - 1) * x_outer_stride + static_cast<int64_t>(span_x)) * es);
  const uintptr_t y1 = y0 + static_cast<uintptr_t>(((outer - 1) * y_outer_stride + static_cast<int64_t>(span_y)) * es);
  if (x0 < y1 && y0 < x1 && !(x0 == y0 && x_outer_stride == y_outer_stride && x_reduce_stride == y_reduce_stride))
    return akg::fail(AKG_ERR_INVALID_ARG, "%s: x and y overlap without being the same array", name);

  akg::AxisParams p;
  p.x = x; p.y = y; p.outer = outer; p.reduce = reduce; p.inner = inner;
  p.xso = x_outer_stride; p.xsf = x_reduce_stride; p.yso = y_outer_stride; p.ysf = y_reduce_stride;
  p.gamma = norm ? gamma : nullptr;
  p.beta = (op == AKG_OP_LAYERNORM) ? beta : nullptr;
  p.eps = eps;
  const int64_t epv = 16 / es;
  auto multiples_of = [&](int64_t bytes) {
    return (inner * es) % bytes == 0 && reinterpret_cast<uintptr_t>(x) % bytes == 0 &&
           reinterpret_cast<uintptr_t>(y) % bytes == 0 && (x_outer_stride * es) % bytes == 0 &&
           (x_reduce_stride * es) % bytes == 0 && (y_outer_stride * es) % bytes == 0 &&
           (y_reduce_stride * es) % bytes == 0;
  };
  const bool scalar_only = akg::g_forced_variant.load() == akg::V_STREAM;
  const bool vec = !scalar_only && multiples_of(16);
  const int pdl = akg::g_tune_pdl.load() == 2 ? 0 : 1;
  const int tuned = akg::g_tune_grid_cap.load();

  // What a lane holds of a row in the register-resident kernel.  bf16 in 16-byte vectors is
  // unpacked at every use and softmax then needs a second exponential; 8-byte vectors widened
  // to floats avoid both but move 256-byte row segments.  Measured on the sketch's shape:
  // softmax is faster widened, the other three packed.
  int mode = vec ? 1 : 0;
  if (dtype == AKG_BF16 && !scalar_only && multiples_of(8) && (!vec || op == AKG_OP_SOFTMAX)) mode = 2;
  const int t_mode = akg::g_tune_axis_mode.load();
  if (t_mode == 3) mode = 0;
  if (t_mode == 1 && vec) mode = 1;
  if (t_mode == 2 && dtype == AKG_BF16 && !scalar_only && multiples_of(8)) mode = 2;
  const int64_t w = akg::axis_reg_width(static_cast<int>(dtype), mode);

  // Register-resident kernel: nf warps x r rows cover the reduced axis (nf <= 16).  Of the
  // three r, the one that wastes the fewest row slots wins, the larger r on a tie.
  int r_best = 0, nf_best = 0;
  const int t_r = akg::g_tune_axis_r.load();
  for (int r = 8; r >= 2 && t_r >= 0; r >>= 1) {
    if (t_r > 0 && r != t_r) continue;
    const int64_t nf = (reduce + r - 1) / r;
    if (nf > 16) continue;
    if (r_best == 0 || nf * r < static_cast<int64_t>(nf_best) * r_best) { r_best = r; nf_best = static_cast<int>(nf); }
  }
  if (r_best > 0) {
    const int64_t blocks = (inner + 32 * w - 1) / (32 * w);           // column blocks of one outer index
    int64_t nc = std::max(1, 8 / nf_best);                            // about 256 threads
    if (akg::g_tune_axis_nc.load() > 0) nc = std::min<int64_t>(akg::g_tune_axis_nc.load(), 16 / nf_best);
    nc = std::max<int64_t>(1, std::min(nc, blocks));
    const int64_t spo = (blocks + nc - 1) / nc;                       // <= 2^40 / 32 / 4 = 2^33
    // one CTA per strip (more CTAs measured faster than a persistent grid); the loops in the
    // kernel only run when a grid dimension is clipped
    int64_t gx = std::min<int64_t>(spo, tuned > 0 ? tuned : (int64_t(1) << 30));
    if (spo > UINT_MAX) return akg::fail(AKG_ERR_UNSUPPORTED, "%s: inner above 2^37 with a short reduced axis", name);
    const int64_t gy = std::min<int64_t>(outer, 65535);
    const dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(gy));
    const cudaError_t err = akg::launch_axis_reg(static_cast<int>(op), static_cast<int>(dtype), mode, r_best, p, grid,
                                                 static_cast<unsigned>(spo), nf_best, static_cast<int>(nc), pdl,
                                                 static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return akg::cuda_fail(name, err);
    std::snprintf(akg::t_kernel, sizeof akg::t_kernel, "axis_reg<%s,%s,r%d,nf%d,nc%d,grid%ux%u>",
                  dtype_name(dtype), mode == 1 ? "vec" : (mode == 2 ? "wide8" : "scalar"), r_best,
                  nf_best, static_cast<int>(nc), grid.x, grid.y);
    return AKG_OK;
  }

  // Two-pass kernel.  The strips in flight (4 CTAs per SM) are read again from L2 in the second
  // pass: long reduced axes take narrower strips (fewer lanes of a warp along the columns, down
  // to 128-byte row segments) to keep them within 64 MB.
  const int64_t w2 = vec ? epv : 1;
  const int64_t lane_bytes = w2 * es;
  int lc_shift = 5;
  const int min_shift = vec ? 3 : 5;
  while (lc_shift > min_shift &&
         static_cast<long double>(reduce) * (int64_t(1) << lc_shift) * lane_bytes * akg::sm_count() * 4 > 64.0L * 1048576.0L)
    --lc_shift;
  while (lc_shift > 0 && (int64_t(1) << (lc_shift - 1)) * w2 >= inner) --lc_shift;   // no more lanes than columns
  const int t_lc = akg::g_tune_axis_lc.load();
  if (t_lc > 0) lc_shift = std::min(5, t_lc - 1);
  const int64_t cw = (int64_t(1) << lc_shift) * w2;
  const int64_t spo = (inner + cw - 1) / cw;
  if (spo > UINT_MAX) return akg::fail(AKG_ERR_UNSUPPORTED, "%s: inner above 2^32 strips", name);
  const dim3 grid(static_cast<unsigned>(std::min<int64_t>(spo, tuned > 0 ? tuned : (int64_t(1) << 30))),
                  static_cast<unsigned>(std::min<int64_t>(outer, 65535)));
  const cudaError_t err = akg::launch_axis(static_cast<int>(op), static_cast<int>(dtype), vec, p, grid,
                                          static_cast<unsigned>(spo), lc_shift, pdl, static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) return akg::cuda_fail(name, err);
  std::snprintf(akg::t_kernel, sizeof akg::t_kernel, "axis<%s,%s,t256,lc%d,grid%ux%u>", dtype_name(dtype),
                vec ? "vec" : "scalar", 1 << lc_shift, grid.x, grid.y);
  return AKG_OK;
}

// ---- softmax pair with a fused pre-scale -----------------------------------------------------
extern "C" akg_status akg_softmax_scaled(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                                         int64_t y_row_stride, akg_dtype dtype, float scale, const akg_mask* mask,
                                         int log_output, void* stream) {
  using namespace akg;
  const char* name = "akg_softmax_scaled";
  if (!(scale > 0.f) || std::isinf(scale)) {
    t_error[0] = '\0';
    return fail(AKG_ERR_INVALID_ARG, "%s: scale must be finite and > 0", name);
  }
  Call c;
  c.op = log_output ? OP_LOG_SOFTMAX : OP_SOFTMAX;
  c.x = x; c.y = y; c.rows = rows; c.cols = cols; c.xs = x_row_stride; c.ys = y_row_stride;
  c.dtype = static_cast<int>(dtype); c.mask = mask; c.gamma = nullptr; c.beta = nullptr; c.eps = 0.f;
  c.stream = stream; c.scale = scale;
  return run(c, name);
}

// ---- fused residual add + LayerNorm / RMSNorm ----------------------------------------------
extern "C" akg_status akg_add_norm(akg_op op, const void* x, const void* residual, void* y, void* sum_out,
                                   int64_t rows, int64_t cols, int64_t x_row_stride, int64_t res_row_stride,
                                   int64_t y_row_stride, int64_t sum_row_stride, akg_dtype dtype,
                                   const void* gamma, const void* beta, float eps, void* stream) {
  using namespace akg;
  const char* name = "akg_add_norm";
  t_error[0] = '\0';
  if (op != AKG_OP_LAYERNORM && op != AKG_OP_RMSNORM)
    return fail(AKG_ERR_INVALID_ARG, "%s: the operator must be LayerNorm or RMSNorm", name);
  Call c;
  c.op = static_cast<int>(op); c.x = x; c.y = y; c.rows = rows; c.cols = cols; c.xs = x_row_stride; c.ys = y_row_stride;
  c.dtype = static_cast<int>(dtype); c.mask = nullptr; c.gamma = gamma;
  c.beta = (op == AKG_OP_LAYERNORM) ? beta : nullptr; c.eps = eps; c.stream = stream;
  const akg_status st = validate(c, name);
  if (st != AKG_OK) return st;
  if (rows == 0 || cols == 0) return AKG_OK;
  if (residual == nullptr) return fail(AKG_ERR_INVALID_ARG, "%s: residual must not be NULL", name);
  if (res_row_stride < cols || (sum_out != nullptr && sum_row_stride < cols))
    return fail(AKG_ERR_INVALID_ARG, "%s: row stride smaller than cols", name);
  const int64_t es = (dtype == AKG_F32) ? 4 : 2;
  if (static_cast<long double>(rows) * res_row_stride * es > 9.0e18L ||
      static_cast<long double>(rows) * sum_row_stride * es > 9.0e18L)
    return fail(AKG_ERR_INVALID_ARG, "%s: rows * stride overflows", name);
  // An output may be one of the inputs exactly (same base and stride: every element is read
  // before it is written, by the same thread) or disjoint from it; the two outputs are disjoint.
  struct Span { uintptr_t lo, hi; int64_t stride; };
  auto span = [&](const void* ptr, int64_t stride) {
    const uintptr_t lo = reinterpret_cast<uintptr_t>(ptr);
    return Span{lo, lo + static_cast<uintptr_t>(((rows - 1) * stride + cols) * es), stride};
  };
  auto clash = [&](const Span& out, const Span& in) {
    return out.lo < in.hi && in.lo < out.hi && !(out.lo == in.lo && (rows == 1 || out.stride == in.stride));
  };
  const Span sx = span(x, x_row_stride), sr = span(residual, res_row_stride), sy = span(y, y_row_stride);
  if (clash(sy, sr)) return fail(AKG_ERR_INVALID_ARG, "%s: y overlaps residual without being the same matrix", name);
  if (sum_out != nullptr) {
    const Span ss = span(sum_out, sum_row_stride);
    if (clash(ss, sx) || clash(ss, sr))
      return fail(AKG_ERR_INVALID_ARG, "%s: sum_out overlaps an input without being the same matrix", name);
    if (ss.lo < sy.hi && sy.lo < ss.hi) return fail(AKG_ERR_INVALID_ARG, "%s: sum_out overlaps y", name);
  }

  RowParams p;
  std::memset(&p, 0, sizeof p);
  p.x = x; p.y = y; p.rows = rows; p.cols = cols; p.xs = x_row_stride; p.ys = y_row_stride;
  p.gamma = gamma; p.beta = c.beta; p.eps = eps; p.period = 1; p.add_rows = 1;
  p.res = residual; p.rs = res_row_stride; p.sum = sum_out; p.ss = sum_row_stride;
  const int pdl = g_tune_pdl.load() == 2 ? 0 : 1;
  const int cap = g_tune_grid_cap.load();
  unsigned grid = static_cast<unsigned>(rows > INT_MAX ? INT_MAX : rows);
  if (cap > 0 && grid > static_cast<unsigned>(cap)) grid = static_cast<unsigned>(cap);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  const int64_t epv = 16 / es;
  bool vec = vector_ok(c) && g_forced_variant.load() != V_STREAM && aligned16(residual) &&
             (rows == 1 || (res_row_stride * es) % 16 == 0);
  if (sum_out != nullptr) vec = vec && aligned16(sum_out) && (rows == 1 || (sum_row_stride * es) % 16 == 0);
  int vpt = 0;
  int64_t threads = 0;
  if (vec) {
    // a CTA per row, the row in registers: 2 * vpt loads in flight per thread, so four vectors
    // per thread are preferred; at least 128 threads where the row allows
    const int64_t nvec = cols / epv;
    const int order[8] = {4, 3, 2, 1, 8, 7, 6, 5};
    const int t_vpt = g_tune_reg_vpt.load();
    for (int lo : {128, 32}) {
      for (int v : order) {
        if (vpt || (t_vpt > 0 && v != t_vpt) || nvec % v) continue;
        const int64_t g = nvec / v;
        if (g % 32 == 0 && g >= lo && g <= 1024) { vpt = v; threads = g; }
      }
    }
  }
  cudaError_t err;
  if (vpt > 0) {
    err = launch_add_norm(static_cast<int>(op), static_cast<int>(dtype), vpt, static_cast<int>(threads), p, grid, pdl, cs);
    std::snprintf(t_kernel, sizeof t_kernel, "add_flex<%s,t%d,v%d>", dtype_name(dtype),
                  static_cast<int>(threads), vpt);
  } else {
    LaunchPlan plan;
    std::memset(&plan, 0, sizeof plan);
    plan_stream(c, &plan);
    plan.pdl = pdl;
    err = (op == AKG_OP_LAYERNORM) ? launch_op<OP_LAYERNORM>(plan, c.dtype, p, cs) : launch_op<OP_RMSNORM>(plan, c.dtype, p, cs);
    std::snprintf(t_kernel, sizeof t_kernel, "add_stream<%s,t%d>", dtype_name(dtype), plan.threads);
  }
  if (err != cudaSuccess) return cuda_fail(name, err);
  return AKG_OK;
}

// ---- gated activations: SiLU-and-Mul, GELU-and-Mul -----------------------------------------
extern "C" akg_status akg_act_mul(akg_act act, const void* x, void* y, int64_t rows, int64_t d,
                                  int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype, void* stream) {
  using namespace akg;
  const char* name = "akg_act_mul";
  t_error[0] = '\0';
  if (act < AKG_ACT_SILU || act > AKG_ACT_GELU_TANH) return fail(AKG_ERR_INVALID_ARG, "%s: unknown activation", name);
  if (!valid_dtype(dtype)) return fail(AKG_ERR_INVALID_ARG, "%s: unknown dtype", name);
  if (rows < 0 || d < 0) return fail(AKG_ERR_INVALID_ARG, "%s: negative rows or d", name);
  if (rows == 0 || d == 0) return AKG_OK;
  if (x == nullptr || y == nullptr) return fail(AKG_ERR_INVALID_ARG, "%s: x and y must not be NULL", name);
  if (d > (int64_t(1) << 40)) return fail(AKG_ERR_UNSUPPORTED, "%s: d above 2^40", name);
  if (x_row_stride < 2 * d || y_row_stride < d) return fail(AKG_ERR_INVALID_ARG, "%s: row stride too small", name);
  const int64_t es = (dtype == AKG_F32) ? 4 : 2;
  if (static_cast<long double>(rows) * x_row_stride * es > 9.0e18L ||
      static_cast<long double>(rows) * y_row_stride * es > 9.0e18L)
    return fail(AKG_ERR_INVALID_ARG, "%s: rows * stride overflows", name);
  // y may be x itself with the same row stride (the result then replaces the gate half: every
  // element is read before the same thread writes it); any other overlap is refused
  const uintptr_t x0 = reinterpret_cast<uintptr_t>(x), y0 = reinterpret_cast<uintptr_t>(y);
  const uintptr_t x1 = x0 + static_cast<uintptr_t>(((rows - 1) * x_row_stride + 2 * d) * es);
  const uintptr_t y1 = y0 + static_cast<uintptr_t>(((rows - 1) * y_row_stride + d) * es);
  if (x0 < y1 && y0 < x1 && !(x0 == y0 && (rows == 1 || x_row_stride == y_row_stride)))
    return fail(AKG_ERR_INVALID_ARG, "%s: x and y overlap without y being x", name);

  ActParams p;
  p.x = x; p.y = y; p.rows = rows; p.d = d; p.xs = x_row_stride; p.ys = y_row_stride;
  const int64_t epv = 16 / es;
  // (the vector kernel indexes a row's vectors with 32 bits)
  const bool vec = g_forced_variant.load() != V_STREAM && d % epv == 0 && aligned16(x) && aligned16(y) &&
                   d / epv <= (int64_t(1) << 29) &&
                   (rows == 1 || ((x_row_stride * es) % 16 == 0 && (y_row_stride * es) % 16 == 0));
  const int64_t lanes = vec ? d / epv : d;
  const int u = act_mul_unroll();
  int threads = 32;
  while (threads < 256 && static_cast<int64_t>(threads) * u < lanes) threads <<= 1;
  const int64_t chunks = (lanes + static_cast<int64_t>(threads) * u - 1) / (static_cast<int64_t>(threads) * u);
  const int cap = g_tune_grid_cap.load();
  const dim3 grid(static_cast<unsigned>(std::min<int64_t>(chunks, cap > 0 ? cap : (int64_t(1) << 30))),
                  static_cast<unsigned>(std::min<int64_t>(rows, 65535)));
  const cudaError_t err = launch_act_mul(static_cast<int>(act), static_cast<int>(dtype), vec, p, grid, threads,
                                         g_tune_pdl.load() == 2 ? 0 : 1, static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) return cuda_fail(name, err);
  std::snprintf(t_kernel, sizeof t_kernel, "act_mul<%s,%s,%s,t%d,grid%ux%u>",
                act == AKG_ACT_SILU ? "silu" : (act == AKG_ACT_GELU ? "gelu" : "gelu_tanh"),
                dtype_name(dtype), vec ? "vec" : "scalar", threads, grid.x, grid.y);
  return AKG_OK;
}

// ---- arg-max / arg-min and cumulative sum / product over the last axis -------------------------
extern "C" akg_status akg_argreduce(int want_min, const void* x, int64_t* index_out, int64_t rows, int64_t cols,
                                    int64_t x_row_stride, akg_dtype dtype, void* stream) {
  using namespace akg;
  const char* name = "akg_argreduce";
  t_error[0] = '\0';
  if (want_min != 0 && want_min != 1) return fail(AKG_ERR_INVALID_ARG, "%s: want_min must be 0 or 1", name);
  if (!valid_dtype(dtype)) return fail(AKG_ERR_INVALID_ARG, "%s: unknown dtype", name);
  if (rows < 0 || cols < 0) return fail(AKG_ERR_INVALID_ARG, "%s: negative rows or cols", name);
  if (rows == 0) return AKG_OK;
  if (cols == 0) return fail(AKG_ERR_INVALID_ARG, "%s: an empty row has no arg-max", name);
  if (x == nullptr || index_out == nullptr) return fail(AKG_ERR_INVALID_ARG, "%s: x and index_out must not be NULL", name);
  if (x_row_stride < cols) return fail(AKG_ERR_INVALID_ARG, "%s: row stride smaller than cols", name);
  if (cols > INT_MAX / 2) return fail(AKG_ERR_UNSUPPORTED, "%s: cols above 2^30 - 1", name);
  const int64_t es = (dtype == AKG_F32) ? 4 : 2;
  if (static_cast<long double>(rows) * x_row_stride * es > 9.0e18L)
    return fail(AKG_ERR_INVALID_ARG, "%s: rows * stride overflows", name);
  const bool vec = g_forced_variant.load() != V_STREAM && cols % (16 / es) == 0 && aligned16(x) &&
                   (rows == 1 || (x_row_stride * es) % 16 == 0);
  const int t_group = g_tune_reg_group.load();
  // a warp per row up to 8 KB rows (16 KB in the 16-bit types), measured: fp32 2048 columns 97 % of
  // the copy rate against 45 % with a CTA per row, bf16 4096 columns 93 % against 39 %, bf16 8192
  // columns 89 % against 82 %; from there on the CTA per row is ahead
  const int64_t warp_bytes = !vec ? 4096 : (es == 2 ? 16384 : 8192);
  const bool warp_rows = t_group == 32 || (t_group == 0 && cols * es <= warp_bytes);
  const int64_t ctas = warp_rows ? (rows + 7) / 8 : rows;
  int cap = g_tune_grid_cap.load();
  // a CTA per row runs grid-stride over four resident waves (five CTAs per SM), which lets it load
  // its next row early; rows of 64 KB and more measured a little better with a CTA each
  if (cap == 0 && !warp_rows && vec && cols * es < 65536) cap = sm_count() * 20;
  const unsigned grid = static_cast<unsigned>(std::min<int64_t>(ctas, cap > 0 ? cap : INT_MAX));
  // few, long rows (a batch of vocabulary-sized rows): cut every row into segments so that about
  // four CTAs per SM are busy, each with at least 4096 lanes of work
  const int64_t lanes = vec ? cols / (16 / es) : cols;
  int64_t segments = 1;
  if (!warp_rows && rows < 2 * static_cast<int64_t>(sm_count()) && g_tune_reg_general.load() == 0) {
    segments = std::min<int64_t>((4 * static_cast<int64_t>(sm_count()) + rows - 1) / rows, lanes / 4096);
    segments = std::max<int64_t>(1, std::min<int64_t>(segments, 1024));
  }
  const int64_t seg_vecs = (lanes + segments - 1) / segments;
  const cudaError_t err = launch_argreduce(want_min == 1, static_cast<int>(dtype), vec, warp_rows, x,
                                           reinterpret_cast<long long*>(index_out), rows, cols, x_row_stride, grid,
                                           static_cast<unsigned>(segments), seg_vecs,
                                           g_tune_pdl.load() == 2 ? 0 : 1, static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) return cuda_fail(name, err);
  if (segments > 1)
    std::snprintf(t_kernel, sizeof t_kernel, "arg_split<%s,%s,%s,t256,seg%u>", want_min ? "min" : "max",
                  dtype_name(dtype), vec ? "vec" : "scalar", static_cast<unsigned>(segments));
  else
    std::snprintf(t_kernel, sizeof t_kernel, "arg<%s,%s,%s,g%d,t256,grid%u>", want_min ? "min" : "max",
                  dtype_name(dtype), vec ? "vec" : "scalar", warp_rows ? 32 : 256, grid);
  return AKG_OK;
}

// Rows up to this many bytes take a warp each (measured against a CTA per row: fp32 512 columns 107 %
// of the copy rate against 61 %, 1024 - 2048 columns level, 8192 columns 98 % against 105 %; bf16
// 1024 columns 96 % against 60 %, 8192 columns 95 % against 80 %, 16384 columns 91 % against 87 %).
namespace akg { constexpr int64_t scan_warp_row_bytes(int64_t es) { return es == 2 ? 32768 : 2048; } }

extern "C" akg_status akg_cumulative(int want_prod, const void* x, void* y, int64_t rows, int64_t cols,
                                     int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype, void* stream) {
  using namespace akg;
  const char* name = "akg_cumulative";
  t_error[0] = '\0';
  if (want_prod != 0 && want_prod != 1) return fail(AKG_ERR_INVALID_ARG, "%s: want_prod must be 0 or 1", name);
  Call c;
  c.op = OP_SOFTMAX; c.x = x; c.y = y; c.rows = rows; c.cols = cols; c.xs = x_row_stride; c.ys = y_row_stride;
  c.dtype = static_cast<int>(dtype); c.mask = nullptr; c.gamma = nullptr; c.beta = nullptr; c.eps = 0.f; c.stream = stream;
  const akg_status st = validate(c, name);                  // shapes, strides, NULLs, overlap (in place allowed)
  if (st != AKG_OK) return st;
  if (rows == 0 || cols == 0) return AKG_OK;
  const int64_t es = (dtype == AKG_F32) ? 4 : 2;
  const bool vec = g_forced_variant.load() != V_STREAM && vector_ok(c);
  const int64_t nvec = vec ? cols / (16 / es) : cols;
  const int u = scan_unroll();
  int threads = 32;
  while (threads < 256 && static_cast<int64_t>(threads) * u < nvec) threads <<= 1;
  const int cap = g_tune_grid_cap.load();
  const int t_group = g_tune_reg_group.load();
  // short rows: a warp per row, eight rows per CTA (no CTA barrier, no one- or two-warp CTAs)
  const bool warp_rows = vec && (t_group == 32 || (t_group == 0 && cols * es <= scan_warp_row_bytes(es)));
  const int64_t ctas = warp_rows ? (rows + 7) / 8 : rows;
  const unsigned grid = static_cast<unsigned>(std::min<int64_t>(ctas, cap > 0 ? cap : INT_MAX));
  // Rows of at most 64 vectors (a kilobyte): 4, 8 or 16 lanes per row, several rows per warp (scan_short_kernel)
  if (vec && nvec <= 64 && t_group == 0 && g_tune_reg_general.load() == 0) {
    int lanes = 4;
    while (4 * lanes < nvec) lanes *= 2;
    const int64_t rows_per_cta = 8 * (32 / lanes);
    int64_t sctas = (rows + rows_per_cta - 1) / rows_per_cta;
    const int64_t scap = cap > 0 ? cap : static_cast<int64_t>(sm_count()) * 32;     // grid-stride beyond four waves
    if (sctas > scap) sctas = scap;
    const cudaError_t e1 = launch_cumulative_short(want_prod == 1, static_cast<int>(dtype), lanes, x, y, rows, cols,
                                                   x_row_stride, y_row_stride, static_cast<unsigned>(sctas),
                                                   g_tune_pdl.load() == 2 ? 0 : 1, static_cast<cudaStream_t>(stream));
    if (e1 != cudaSuccess) return cuda_fail(name, e1);
    std::snprintf(t_kernel, sizeof t_kernel, "scan_short<%s,%s,l%d,grid%u>", want_prod ? "prod" : "sum", dtype_name(dtype),
                  lanes, static_cast<unsigned>(sctas));
    return AKG_OK;
  }
  // Few, long rows (at least 8192 vectors each, fewer rows than SMs): a cluster per row, every CTA a slice of
  // about 4096 vectors, the carry of a slice from the cluster's totals (scan_split_kernel).  Measured against a
  // CTA per row, fraction of the copy rate: [64, 2^20] fp32 0.54 against 0.30, bf16 0.64 against 0.22;
  // [100, 262144] fp32 0.66 against 0.49, bf16 0.57 against 0.45; from one row per SM on a CTA per row is ahead
  // ([256, 262144] fp32 0.85 against 0.75; bf16, with its loads three chunks ahead, 0.80 against 0.74).
  const int t_cs = g_tune_cluster_size.load();
  if (vec && !warp_rows && g_tune_reg_general.load() == 0 &&
      (t_cs > 1 || (t_cs == 0 && rows < static_cast<int64_t>(sm_count()) && nvec >= 8192))) {
    int cs = t_cs;
    if (cs == 0) {
      cs = 2;
      while (cs < kMaxCluster && (nvec / (2 * cs) >= 3072 || rows * cs < 2 * static_cast<int64_t>(sm_count()))) cs *= 2;
    }
    if (cs >= 2 && cs <= kMaxCluster && (cs & (cs - 1)) == 0 && nvec / cs >= 256 && nvec <= INT_MAX / 2) {
      int64_t slice = (nvec + cs - 1) / cs;
      slice = (slice + 255) / 256 * 256;
      // rows in flight stay in L2 between the two phases: at most 64 MB of them
      int64_t clusters = (int64_t(64) << 20) / (cols * es);
      if (clusters < (160 + cs - 1) / cs) clusters = (160 + cs - 1) / cs;
      if (cap > 0) clusters = std::max(1, cap / cs);
      const cudaError_t e2 = launch_cumulative_split(want_prod == 1, static_cast<int>(dtype), x, y, rows, cols, x_row_stride,
                                                     y_row_stride, cs, static_cast<int>(slice), clusters, status_word_ptr(),
                                                     g_tune_test_wait_us.load() > 0 ? static_cast<unsigned>(g_tune_test_wait_us.load()) : 0u,
                                                     static_cast<cudaStream_t>(stream));
      if (e2 != cudaSuccess) return cuda_fail(name, e2);
      std::snprintf(t_kernel, sizeof t_kernel, "scan_split<%s,%s,t256,cs%d,slice%d>", want_prod ? "prod" : "sum",
                    dtype_name(dtype), cs, static_cast<int>(slice));
      return AKG_OK;
    }
  }
  // 16-bit rows, a CTA per row with fewer CTAs than two per SM and rows of several chunks: the loads run three
  // chunks ahead (bf16 [256, 262144] 0.67 -> 0.80 of the copy rate, [148, 131072] 0.48 -> 0.57; fp32 measured level
  // or a little slower with them, 0.85 / 0.85 and 0.82 / 0.84, and keeps one chunk)
  const int t_depth = g_tune_reg_vpt.load();                   // (tuning: reg_vpt 1 / 3 forces the depth)
  const int depth = (vec && !warp_rows && threads == 256 &&
                     (t_depth == 3 || (t_depth == 0 && es == 2 && ctas <= 2 * static_cast<int64_t>(sm_count()) &&
                                       nvec >= 4 * 1024)))
                        ? 3 : 1;
  const cudaError_t err = launch_cumulative(want_prod == 1, static_cast<int>(dtype), vec, x, y, rows, cols, x_row_stride,
                                            y_row_stride, grid, threads, warp_rows, g_tune_pdl.load() == 2 ? 0 : 1,
                                            static_cast<cudaStream_t>(stream), depth);
  if (err != cudaSuccess) return cuda_fail(name, err);
  std::snprintf(t_kernel, sizeof t_kernel, "scan<%s,%s,%s,%s%d,grid%u%s>", want_prod ? "prod" : "sum",
                dtype_name(dtype), vec ? "vec" : "scalar", warp_rows ? "g32,t" : "t", warp_rows ? 256 : threads, grid,
                depth > 1 ? ",ahead3" : "");
  return AKG_OK;
}

// ---- BatchNorm-style column normalisation ------------------------------------------------------
namespace akg {
constexpr int kColMaxBlocks = 256;
// row blocks that fill the GPU (up to eight CTAs per SM) when the strips are a full warp of 16-byte vectors wide
int64_t colnorm_blocks(int64_t cols, int64_t es) {
  const int64_t strips = (cols * es + 511) / 512;
  return std::max<int64_t>(1, std::min<int64_t>(kColMaxBlocks, (int64_t(sm_count()) * 8 + strips - 1) / strips));
}
}

extern "C" size_t akg_colnorm_workspace_bytes(int64_t rows, int64_t cols) {
  if (rows <= 0 || cols <= 0) return 0;
  return static_cast<size_t>(akg::colnorm_blocks(cols, 2)) * static_cast<size_t>(cols) * sizeof(float2);
}

extern "C" akg_status akg_colnorm(const void* x, void* y, int64_t rows, int64_t cols, int64_t x_row_stride,
                                  int64_t y_row_stride, akg_dtype dtype, const void* gamma, const void* beta,
                                  float eps, float* mean_out, float* var_out, void* workspace,
                                  size_t workspace_bytes, void* stream) {
  using namespace akg;
  const char* name = "akg_colnorm";
  t_error[0] = '\0';
  Call c;
  c.op = OP_LAYERNORM; c.x = x; c.y = y; c.rows = rows; c.cols = cols; c.xs = x_row_stride; c.ys = y_row_stride;
  c.dtype = static_cast<int>(dtype); c.mask = nullptr; c.gamma = gamma; c.beta = beta; c.eps = eps; c.stream = stream;
  const akg_status st = validate(c, name);
  if (st != AKG_OK) return st;
  if (rows == 0 || cols == 0) return AKG_OK;
  const int64_t es = (dtype == AKG_F32) ? 4 : 2;
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 7u) != 0 ||
      workspace_bytes < static_cast<size_t>(cols) * sizeof(float2))
    return fail(AKG_ERR_INVALID_ARG, "%s: workspace must be 8-byte aligned and hold at least cols * 8 bytes", name);
  const bool vec = g_forced_variant.load() != V_STREAM && cols % (16 / es) == 0 && aligned16(x) && aligned16(y) &&
                   (rows == 1 || ((x_row_stride * es) % 16 == 0 && (y_row_stride * es) % 16 == 0));
  const int64_t w = vec ? 16 / es : 1;
  // Row blocks the workspace and the matrix allow, then the lanes of a warp along the columns: 32
  // (512-byte row segments) unless narrower strips are needed to give every SM its CTAs.
  const int64_t ws_blocks = static_cast<int64_t>(workspace_bytes / (static_cast<size_t>(cols) * sizeof(float2)));
  int64_t max_rb = std::min<int64_t>(kColMaxBlocks, ws_blocks);
  const int t_rb = g_tune_grid_cap.load();
  if (t_rb > 0) max_rb = std::min<int64_t>(max_rb, t_rb);
  const int64_t want = static_cast<int64_t>(sm_count()) * 4;
  int lc_shift = 5;
  while (lc_shift > 3 && ((int64_t(1) << lc_shift) * w > cols ||
                          ((cols + (int64_t(1) << lc_shift) * w - 1) / ((int64_t(1) << lc_shift) * w)) * max_rb < want))
    --lc_shift;
  const int t_lc = g_tune_axis_lc.load();
  if (t_lc > 0) lc_shift = std::min(5, std::max(0, t_lc - 1));
  const int64_t cw = (int64_t(1) << lc_shift) * w;
  const int64_t strips = (cols + cw - 1) / cw;
  if (strips > INT_MAX) return fail(AKG_ERR_UNSUPPORTED, "%s: too many columns", name);
  const int64_t slots = colnorm_row_slots(lc_shift);
  // Four CTAs are resident per SM, so strips * blocks is aimed at one full wave of them, or at two
  // where that still leaves blocks of 512 rows or more; a partial second wave measured 10 - 20 %
  // slower than either (16384 x 8192: 64 x 10 blocks 76 %, 64 x 18 blocks 95 % of the three-stream rate).
  const int64_t one = std::max<int64_t>(1, want / strips), two = std::max<int64_t>(1, 2 * want / strips);
  int64_t rb = (two <= max_rb && rows / two >= 512) ? two : std::min<int64_t>(one, max_rb);
  rb = std::max<int64_t>(1, std::min<int64_t>(rb, (rows + slots - 1) / slots));
  int64_t rpb = (rows + rb - 1) / rb;
  rpb = (rpb + slots - 1) / slots * slots;
  rb = (rows + rpb - 1) / rpb;

  ColParams p;
  p.x = x; p.y = y; p.rows = rows; p.cols = cols; p.xs = x_row_stride; p.ys = y_row_stride;
  p.gamma = gamma; p.beta = beta; p.eps = eps; p.partial = static_cast<float2*>(workspace);
  p.mean_out = mean_out; p.var_out = var_out; p.rows_per_block = rpb; p.lc_shift = lc_shift;
  // L2 priorities ("keep" while the statistics are taken, "drop" when the rows are read again) while the
  // matrix is at most about twice the size of L2
  p.l2_keep = (static_cast<long double>(rows) * cols * es <= 288.0L * 1048576.0L) ? 1 : 0;
  const dim3 grid(static_cast<unsigned>(strips), static_cast<unsigned>(rb));
  const cudaError_t err = launch_colnorm(static_cast<int>(dtype), vec, p, grid, g_tune_pdl.load() == 2 ? 0 : 1,
                                         static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) return cuda_fail(name, err);
  std::snprintf(t_kernel, sizeof t_kernel, "colnorm<%s,%s,lc%d,grid%ux%u>", dtype_name(dtype), vec ? "vec" : "scalar",
                1 << lc_shift, grid.x, grid.y);
  return AKG_OK;
}

// ---- host buffers without any allocation ---------------------------------------------------
// akg_rowop_host needs a device staging area from its caller.  Some callers have no way to
// get one: a plug-in that is handed host buffers and a stream but no allocator, a service
// whose device memory is wholly owned by another component's pool, a control loop that may
// not allocate once it is running.  For them the staging area below is part of the library
// image: the driver reserves it on every GPU that loads the library and keeps it until the
// process exits.  It is shared by every call on that GPU and keeps whatever the last call
// left in it; nothing in it has to start at zero, because each chunk is fully overwritten
// by its upload before a kernel reads it.
namespace {

constexpr size_t kStaticStagingBytes = size_t(16) << 20;          // AKG_STATIC_STAGING_BYTES
static __device__ __align__(256) unsigned char g_static_staging[kStaticStagingBytes];

// In host code `g_static_staging` is only a handle for the runtime, not a device address.
// The address is asked for once per device, with that device current, and cached.
akg_status static_staging_address(const char* name, unsigned char** out) {
  static std::atomic<unsigned char*> cache[64];
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return akg::cuda_fail(name, err);
  if (dev < 0 || dev >= 64) return akg::fail(AKG_ERR_UNSUPPORTED, "%s: device index above 63", name);
  unsigned char* ptr = cache[dev].load();
  if (ptr == nullptr) {
    void* sym = nullptr;
    err = cudaGetSymbolAddress(&sym, g_static_staging);
    if (err != cudaSuccess || sym == nullptr) return akg::cuda_fail(name, err);
    ptr = static_cast<unsigned char*>(sym);
    cache[dev].store(ptr);
  }
  *out = ptr;
  return AKG_OK;
}

}  // namespace

extern "C" akg_status akg_rowop_host_static(akg_op op, const void* x_host, void* y_host, int64_t rows, int64_t cols,
                                            int64_t x_row_stride, int64_t y_row_stride, akg_dtype dtype,
                                            const void* gamma_host, const void* beta_host, float eps,
                                            const akg_mask* mask, void* stream) {
  const char* name = "akg_rowop_host_static";
  if (op < AKG_OP_SOFTMAX || op > AKG_OP_RMSNORM) return akg::fail(AKG_ERR_INVALID_ARG, "%s: unknown operator", name);
  const bool softmax_like = (op == AKG_OP_SOFTMAX || op == AKG_OP_LOG_SOFTMAX);
  akg::Call hc{static_cast<int>(op), x_host, y_host, rows, cols, x_row_stride, y_row_stride, static_cast<int>(dtype),
               softmax_like ? mask : nullptr, softmax_like ? nullptr : gamma_host,
               op == AKG_OP_LAYERNORM ? beta_host : nullptr, softmax_like ? 0.f : eps, stream};
  akg::t_error[0] = '\0';
  akg_status st = akg::validate(hc, name);
  if (st != AKG_OK) return st;
  if (hc.rows == 0 || hc.cols == 0) return AKG_OK;
  if (hc.mask != nullptr && hc.mask->additive != nullptr)
    return akg::fail(AKG_ERR_UNSUPPORTED, "%s: an additive mask is not supported with host buffers", name);
  const size_t es = (hc.dtype == AKG_F32) ? 4 : 2;
  const size_t row_bytes = static_cast<size_t>(hc.cols) * es;
  const size_t vec_bytes = akg::host_vector_bytes(hc.cols, hc.dtype, hc.gamma != nullptr, hc.beta != nullptr);
  if (vec_bytes + akg::round_up(row_bytes, 256) > kStaticStagingBytes) {
    std::snprintf(akg::t_error, sizeof akg::t_error,
                  "%s: a row of %lld columns (with its vectors) does not fit the built-in %zu-byte staging area; "
                  "use akg_rowop_host with a workspace of your own", name, static_cast<long long>(hc.cols),
                  kStaticStagingBytes);
    return AKG_ERR_UNSUPPORTED;
  }
  unsigned char* ws = nullptr;
  st = static_staging_address(name, &ws);
  if (st != AKG_OK) return st;

  // One slot, one stream: upload a chunk, run the operator on it in place, download it.
  cudaStream_t user = static_cast<cudaStream_t>(hc.stream);
  cudaError_t err;
  void* d_gamma = nullptr;
  void* d_beta = nullptr;
  size_t off = 0;
  if (hc.gamma != nullptr) {
    d_gamma = ws + off; off += akg::round_up(row_bytes, 256);
    if ((err = cudaMemcpyAsync(d_gamma, hc.gamma, row_bytes, cudaMemcpyHostToDevice, user)) != cudaSuccess)
      return akg::cuda_fail(name, err);
  }
  if (hc.beta != nullptr) {
    d_beta = ws + off; off += akg::round_up(row_bytes, 256);
    if ((err = cudaMemcpyAsync(d_beta, hc.beta, row_bytes, cudaMemcpyHostToDevice, user)) != cudaSuccess)
      return akg::cuda_fail(name, err);
  }
  unsigned char* slot = ws + vec_bytes;
  const int64_t chunk_rows = static_cast<int64_t>((kStaticStagingBytes - vec_bytes) / row_bytes);
  const unsigned char* hx = static_cast<const unsigned char*>(hc.x);
  unsigned char* hy = static_cast<unsigned char*>(hc.y);
  for (int64_t r0 = 0; r0 < hc.rows; r0 += chunk_rows) {
    const int64_t n = (hc.rows - r0 < chunk_rows) ? hc.rows - r0 : chunk_rows;
    err = cudaMemcpy2DAsync(slot, row_bytes, hx + static_cast<size_t>(r0) * hc.xs * es, static_cast<size_t>(hc.xs) * es,
                            row_bytes, static_cast<size_t>(n), cudaMemcpyHostToDevice, user);
    if (err != cudaSuccess) return akg::cuda_fail(name, err);
    akg::Call dc = hc;
    dc.x = slot; dc.y = slot; dc.rows = n; dc.xs = hc.cols; dc.ys = hc.cols;
    dc.gamma = d_gamma; dc.beta = d_beta; dc.row_base = r0;
    st = akg::run(dc, name);
    if (st != AKG_OK) return st;
    err = cudaMemcpy2DAsync(hy + static_cast<size_t>(r0) * hc.ys * es, static_cast<size_t>(hc.ys) * es, slot, row_bytes,
                            row_bytes, static_cast<size_t>(n), cudaMemcpyDeviceToHost, user);
    if (err != cudaSuccess) return akg::cuda_fail(name, err);
  }
  return AKG_OK;
}

static_assert(kStaticStagingBytes == AKG_STATIC_STAGING_BYTES, "the header states the size of the staging area");
