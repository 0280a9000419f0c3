// Internal declarations shared by the translation units of the library.
// Nothing here is part of the public C ABI (see include/abs.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "abs.h"

namespace absk {

constexpr int kSmCountFallback = 148;
constexpr size_t kDefaultWorkspace = 64ull << 20;
constexpr int kFlagWords = 64;                              // flag words at the head of abs_ctx::flags
constexpr int kTicketWords = 4096;                          // per-worker ticket counters that follow them
constexpr int kMaxFastRows = 4096;                          // largest b the tiled and cluster kernels cover
constexpr long long kDefaultTimeoutCycles = 4000000000ll;   // about two seconds of SM clock

struct Tuning {
  long long stats_stages = 0;
  long long stats_ctas_per_worker = 0;
  long long stats_force_generic = 0;
  long long stats_flush_every = 0;
  long long stats_stage_kb = 0;
  long long stats_ctas_per_sm = 0;
  long long stats_no_gram = 0;
  long long stats_no_cluster = 0;
  long long stats_no_secondary = 0;        // 1: the cluster kernel does not use the SMs its clusters cannot occupy
  long long stats_secondary_pct = 0;       // speed of an SM of the second launch, per cent of the first's (0: 95)
  long long mlp_no_tensor_cores = 0;       // 1: the MLP producer's products stay on the CUDA cores
  long long stats_no_recheck = 0;          // 1: keep a Gram kernel's record whatever its conditioning
  long long stats_cluster_rows = 0;
  long long stats_timeout_cycles = 0;      // 0: about two seconds of SM clock
  long long stats_fault_drop_loads = 0;    // test hook: the tiled kernel's loader issues no copies
};

// What the launchers remember per kernel function, so that a call does not repeat host-side runtime
// queries whose answers cannot change: the largest dynamic shared-memory size already granted
// (cudaFuncSetAttribute costs about a microsecond per call) and, for cluster kernels, how many
// clusters of a given size and shared-memory footprint can be resident at once
// (cudaOccupancyMaxActiveClusters costs tens of microseconds).
struct FnCache {
  static constexpr int kSlots = 128;
  const void* fn[kSlots] = {};
  size_t smem_granted[kSlots] = {};
  int cluster_size[kSlots] = {};
  size_t cluster_smem[kSlots] = {};
  int max_clusters[kSlots] = {};
  int n = 0;
  int slot(const void* f) {            // index of f's entry, created if there is room; -1 otherwise
    for (int i = 0; i < n; ++i)
      if (fn[i] == f) return i;
    if (n == kSlots) return -1;
    fn[n] = f;
    return n++;
  }
};

}  // namespace absk

// The context: device, workspace for per-CTA partial sums, a device staging area
// for the *_host entry points, tuning knobs and the last error message.
struct abs_ctx {
  int device = 0;
  int sm_count = absk::kSmCountFallback;
  size_t smem_optin = 0;
  void* workspace = nullptr;       // device
  size_t workspace_bytes = 0;
  unsigned* flags = nullptr;       // device, 64 words: [0] async-copy timeout flag; then ticket_slots
                                   // zeroed words, one per worker, for the split finalisation
  int ticket_slots = 0;
  void* staging = nullptr;         // device buffer for *_host calls, grown on demand
  size_t staging_bytes = 0;
  void* staging_out = nullptr;     // device buffer for stats / gbar of *_host calls
  size_t staging_out_bytes = 0;
  absk::Tuning tuning;
  absk::FnCache fn_cache;
  char err[512] = {0};
};

namespace absk {

int set_error(abs_ctx* ctx, int code, const char* fmt, ...);

// Grants `kernel` at least `smem` bytes of dynamic shared memory (once per context).  The limit is a
// property of the kernel in the process, not of the context, and setting it again lowers it: so what
// is asked for is always the device's opt-in maximum, the same from every context and from the
// context-free entry point, and nobody's later, smaller need can take away what another remembers
// to have been granted.
template <typename K>
inline cudaError_t ensure_dynamic_smem(abs_ctx* ctx, K kernel, size_t smem) {
  const void* f = reinterpret_cast<const void*>(kernel);
  const int i = ctx->fn_cache.slot(f);
  if (i >= 0 && ctx->fn_cache.smem_granted[i] >= smem) return cudaSuccess;
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, f);               // its static shared memory counts against the maximum
  if (e != cudaSuccess) return e;
  const size_t room = ctx->smem_optin > fa.sharedSizeBytes ? ctx->smem_optin - fa.sharedSizeBytes : 0;
  const size_t grant = room > smem ? room : smem;
  e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(grant));
  if (e == cudaSuccess && i >= 0) ctx->fn_cache.smem_granted[i] = grant;
  return e;
}

#define ABS_CUDA_TRY(ctx, expr)                                                          \
  do {                                                                                   \
    cudaError_t e__ = (expr);                                                            \
    if (e__ != cudaSuccess)                                                              \
      return absk::set_error((ctx), ABS_ERR_CUDA, "%s failed: %s", #expr,                \
                             cudaGetErrorString(e__));                                   \
  } while (0)

// ---- programmatic dependent launch ---------------------------------------------------------
// The small kernels that follow a statistics kernel in the stream (finalisation, batch-size
// update) are launched with the programmatic-serialisation attribute: their launch overlaps the
// tail of the kernel before them, and they call pdl_wait() before they touch anything it wrote
// (the wait returns when that kernel has completed and its writes are visible).  The kernels
// before them call pdl_launch_dependents() once they are resident.  Both are no-ops in a kernel
// launched the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                             Args... args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---- decisions shared by the kernels that turn sums into records and records into sizes -----
#ifdef __CUDACC__
__device__ __forceinline__ double safe_ratio(double num, double den) {
  if (num == 0.0) return 0.0;            // 0/x and 0/0 count as 0
  if (den == 0.0) return INFINITY;       // x/0 counts as +infinity
  return num / den;
}
__device__ __forceinline__ long long ceil_saturating(double x) {
  if (!(x < 4611686018427387904.0)) return 1ll << 62;   // also catches NaN
  return static_cast<long long>(ceil(x));
}

// T of one worker (Eq. norm_test, Eq. test_stat; the augmented inner-product test takes the
// larger of its two ceilings).  All arithmetic that decides the integer is fp64, in the order
// scale * (variance / (constant^2 * N [* N])).  A record that cannot be used gives 0.
__device__ __forceinline__ long long test_size_from_record(const abs_stats& s, const abs_test_cfg& cfg) {
  const bool usable = (s.status & (ABS_STATUS_NONFINITE | ABS_STATUS_TIMEOUT)) == 0u &&
                      (cfg.kind != ABS_TEST_AUG_INNER_PRODUCT || (s.status & ABS_STATUS_NORM_ONLY) == 0u);
  if (!usable) return 0;
  const double scale = cfg.row_weight / cfg.divisor;
  const double N = s.gbar_sq;
  if (cfg.kind != ABS_TEST_AUG_INNER_PRODUCT)      // the norm test, on per-sample rows or on workers' batch gradients
    return ceil_saturating(scale * safe_ratio(s.var_norm, cfg.eta * cfg.eta * N));
  const long long t_ip = ceil_saturating(scale * safe_ratio(s.var_ip, cfg.theta * cfg.theta * N * N));
  const long long t_orth = ceil_saturating(scale * safe_ratio(s.var_orth, cfg.nu * cfg.nu * N));
  return t_ip > t_orth ? t_ip : t_orth;
}

// The record of one worker from its four sums (Eq. def_var): V = sum_i ||g_i - gbar||^2,
// N = ||gbar||^2, s_e = sum_i e_i and s_ee = sum_i e_i^2 with e_i = <g_i - gbar, gbar>.
__device__ __forceinline__ abs_stats record_from_sums(double V, double N, double s_e, double s_ee, long long b,
                                                      bool timed_out) {
  const double bd = static_cast<double>(b);
  const double var_norm = V / (bd - 1.0);
  double ss = s_ee - s_e * s_e / bd;     // sum_i (e_i - mean e)^2; mean e is rounding noise only
  if (ss < 0.0) ss = 0.0;
  const double var_ip = ss / (bd - 1.0);
  double var_orth = var_norm;
  if (N > 0.0) {
    var_orth = var_norm - var_ip / N;
    if (var_orth < 0.0) var_orth = 0.0;
  }
  unsigned status = 0u;
  if (!(isfinite(V) && isfinite(N) && isfinite(s_ee))) status |= ABS_STATUS_NONFINITE;
  if (N == 0.0) status |= ABS_STATUS_ZERO_MEAN;
  if (timed_out) status |= ABS_STATUS_TIMEOUT;
  abs_stats s;
  s.gbar_sq = N;
  s.var_norm = var_norm;
  s.var_ip = var_ip;
  s.var_orth = var_orth;
  s.sum_sq = V + bd * N;
  s.rows = b;
  s.status = status;
  s.recomputed = 0u;
  return s;
}
#endif

// ---- statistics kernels (abs_stats_tiled.cu, abs_stats_generic.cu) ---------------------
// Layout of the partial-sum workspace written by both statistics kernels:
//   ws[(m * P + p) * (b + 2) + r]      r < b : sum over the CTA's columns of (g_rj - gbar_j) gbar_j
//   ws[(m * P + p) * (b + 2) + b]              sum over the CTA's columns of sum_r (g_rj - gbar_j)^2
//   ws[(m * P + p) * (b + 2) + b + 1]          sum over the CTA's columns of gbar_j^2
struct StatsLaunch {
  const void* G;
  abs_dtype dtype;
  int M;
  long long b, d, row_stride, worker_stride;
  float* gbar_out;
  abs_stats* stats_out;
  cudaStream_t stream;
  const unsigned* guard = nullptr;   // device word or NULL: the tiled kernel returns at once while it is zero
};

// How the finalisation treats the records of a tensor-core Gram kernel.  Those kernels only ever
// see uncentred products added in fp32, so sum_i ||g_i - gbar||^2 = tr K - 1'K1/b loses
// b N / ((b-1) var_norm) in relative accuracy (rows dominated by a common vector), and
// e_i = (K1)_i/b - N loses N / sqrt(var_ip).  A record beyond the limits raises *redo; the tiled
// kernel (centred accumulation) and a second finalisation then run guarded by that word, and
// return at once when it is zero.
struct Recheck {
  double max_kv = 0.0;       // 0: no check; else recompute when b N > max_kv (b-1) var_norm
  double max_kip = 0.0;      //                          or when N^2 > max_kip^2 var_ip
  unsigned* redo = nullptr;  // device word
  int second = 0;            // 1: the finalisation of the recomputation: a no-op unless *redo, which it clears
};

// Returns ABS_OK, or ABS_ERR_UNSUPPORTED when the tiled kernel cannot take the call
// (alignment, b too large); *P_out receives the number of partial records per worker.
int launch_stats_tiled(abs_ctx* ctx, const StatsLaunch& a, int* P_out);
int launch_stats_gram(abs_ctx* ctx, const StatsLaunch& a, int* P_out);      // bf16, b <= 32
int launch_stats_umma(abs_ctx* ctx, const StatsLaunch& a, int* P_out);      // bf16, 32 < b <= 256 (tcgen05)
int launch_stats_cluster(abs_ctx* ctx, const StatsLaunch& a, int* P_out);   // 256 < b <= 4096
int launch_stats_generic(abs_ctx* ctx, const StatsLaunch& a, int* P_out);
int launch_stats_finalize(abs_ctx* ctx, const StatsLaunch& a, int P, const Recheck& rk = Recheck());
// True when launch_stats_tiled would take the call (shape, alignment, workspace).
bool stats_tiled_feasible(abs_ctx* ctx, const StatsLaunch& a);

// Round end of Algorithm 2 (abs_rounds.cu), shared by the per-round drivers.
int worker_gradient_test(abs_ctx* ctx, const float* Gb, int M, long long d, long long b, const abs_test_cfg* cfg,
                         abs_stats* stats, long long* T_out, long long* b_dev, void* stream);

// Host-side planning shared by the launchers and abs_plan_stats; ABS_OK or ABS_ERR_UNSUPPORTED.
int plan_stats_gram(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, abs_stats_plan* out);
int plan_stats_umma(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, abs_stats_plan* out);
int plan_stats_cluster(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, int cluster_size,
                       abs_stats_plan* out);   // cluster_size 0: the preferred size
int plan_stats_tiled(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, abs_stats_plan* out);

}  // namespace absk
