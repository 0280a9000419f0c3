// Context management, argument validation and dispatch for the statistics entry points.
#include <stdarg.h>
#include <new>

#include "abs_internal.cuh"

namespace absk {

static thread_local char g_create_error[512] = {0};

int set_error(abs_ctx* ctx, int code, const char* fmt, ...) {
  char* dst = ctx != nullptr ? ctx->err : g_create_error;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 512, fmt, ap);
  va_end(ap);
  return code;
}

namespace {

struct DeviceScope {
  int prev = -1;
  bool ok = true;
  explicit DeviceScope(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceScope() { if (prev >= 0) cudaSetDevice(prev); }
};

int validate_stats(abs_ctx* ctx, const void* G, abs_dtype dtype, int M, long long b, long long d,
                   long long row_stride, long long worker_stride, const abs_stats* stats_out) {
  if (G == nullptr || stats_out == nullptr) return set_error(ctx, ABS_ERR_INVALID_ARG, "G or stats_out is null");
  if (dtype != ABS_F32 && dtype != ABS_BF16) return set_error(ctx, ABS_ERR_INVALID_ARG, "unknown dtype %d", (int)dtype);
  if (M < 1) return set_error(ctx, ABS_ERR_INVALID_ARG, "M must be >= 1, got %d", M);
  if (b < 2) return set_error(ctx, ABS_ERR_INVALID_ARG, "b must be >= 2 (the variance divides by b-1), got %lld", b);
  if (d < 1) return set_error(ctx, ABS_ERR_INVALID_ARG, "d must be >= 1, got %lld", d);
  if (b > (1ll << 24)) return set_error(ctx, ABS_ERR_UNSUPPORTED, "b = %lld exceeds 2^24 rows", b);
  if (row_stride < d) return set_error(ctx, ABS_ERR_INVALID_ARG, "row_stride %lld < d %lld", row_stride, d);
  if (M > 1 && worker_stride < (b - 1) * row_stride + d)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "worker_stride %lld overlaps the previous worker", worker_stride);
  return ABS_OK;
}

// Limits beyond which a Gram kernel's record is recomputed by the tiled kernel (see Recheck).
// Measured on bf16 rows = common vector + unit noise, d = 4 M: the relative error of var_norm is
// about 1e-5 (tcgen05, fp32 sums over 4096..8192 columns) resp. 1e-7 (mma.sync, 256 columns) times
// b N / ((b-1) var_norm); var_ip stays below 4e-4 up to N / sqrt(var_ip) = 5e5.  The limits keep
// both a factor of four inside the 1e-3 tolerance of bf16 inputs.
constexpr double kRedoKvUmma = 25.0, kRedoKvMma = 2500.0, kRedoKip = 2.0e5;

int run_stats(abs_ctx* ctx, const StatsLaunch& a) {
  // ctx->flags[0] (time-out flag) is zero here: abs_create clears it and the finalisation kernel
  // of the previous call cleared it again after reading it.
  int P = 0;
  int rc = ABS_ERR_UNSUPPORTED;
  bool gram = false, umma = false;
  if (!ctx->tuning.stats_force_generic && !ctx->tuning.stats_no_gram) {
    rc = launch_stats_gram(ctx, a, &P);
    if (rc == ABS_ERR_UNSUPPORTED) {
      rc = launch_stats_umma(ctx, a, &P);
      umma = rc == ABS_OK;
    }
    gram = rc == ABS_OK;
  }
  if (rc == ABS_ERR_UNSUPPORTED && !ctx->tuning.stats_force_generic && !ctx->tuning.stats_no_cluster)
    rc = launch_stats_cluster(ctx, a, &P);
  if (rc == ABS_ERR_UNSUPPORTED && !ctx->tuning.stats_force_generic) rc = launch_stats_tiled(ctx, a, &P);
  if (rc == ABS_ERR_UNSUPPORTED) rc = launch_stats_generic(ctx, a, &P);
  if (rc != ABS_OK) return rc;
  if (!gram || ctx->tuning.stats_no_recheck || !stats_tiled_feasible(ctx, a)) return launch_stats_finalize(ctx, a, P);
  // Tensor-core route: finalise with the conditioning check, then the centred kernel and its
  // finalisation, both guarded by the word the check may have raised (flags[3]).
  Recheck rk;
  rk.max_kv = umma ? kRedoKvUmma : kRedoKvMma;
  rk.max_kip = kRedoKip;
  rk.redo = ctx->flags + 3;
  rc = launch_stats_finalize(ctx, a, P, rk);
  if (rc != ABS_OK) return rc;
  StatsLaunch again = a;
  again.guard = rk.redo;
  rc = launch_stats_tiled(ctx, again, &P);
  if (rc != ABS_OK) return rc;
  rk.second = 1;
  return launch_stats_finalize(ctx, again, P, rk);
}

int grow(abs_ctx* ctx, void** buf, size_t* have, size_t need) {
  if (*have >= need) return ABS_OK;
  if (*buf != nullptr) {
    ABS_CUDA_TRY(ctx, cudaFree(*buf));
    *buf = nullptr;
    *have = 0;
  }
  ABS_CUDA_TRY(ctx, cudaMalloc(buf, need));
  *have = need;
  return ABS_OK;
}

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int abs_create(abs_ctx** out, int device, size_t workspace_bytes) {
  if (out == nullptr) return set_error(nullptr, ABS_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || count < 1) {
    cudaGetLastError();
    return set_error(nullptr, ABS_ERR_NO_DEVICE, "no CUDA device is visible; this library has no CPU fallback");
  }
  if (device < 0 || device >= count) return set_error(nullptr, ABS_ERR_INVALID_ARG, "device %d out of range", device);
  int major = 0, sms = 0, optin = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess)
    return set_error(nullptr, ABS_ERR_CUDA, "cannot query device %d", device);
  if (major != 10)
    return set_error(nullptr, ABS_ERR_NO_DEVICE, "device %d has compute capability %d.x; the kernels are built for 10.x only",
                     device, major);
  abs_ctx* ctx = new (std::nothrow) abs_ctx();
  if (ctx == nullptr) return set_error(nullptr, ABS_ERR_CUDA, "out of host memory");
  ctx->device = device;
  ctx->sm_count = sms;
  ctx->smem_optin = static_cast<size_t>(optin);
  ctx->workspace_bytes = workspace_bytes ? workspace_bytes : kDefaultWorkspace;
  DeviceScope scope(device);
  cudaError_t e = scope.ok ? cudaMalloc(&ctx->workspace, ctx->workspace_bytes) : cudaErrorInvalidDevice;
  const size_t flag_bytes = static_cast<size_t>(kFlagWords + kTicketWords) * sizeof(unsigned);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->flags), flag_bytes);
  if (e == cudaSuccess) e = cudaMemset(ctx->flags, 0, flag_bytes);
  if (e == cudaSuccess) ctx->ticket_slots = kTicketWords;
  if (e != cudaSuccess) {
    set_error(nullptr, ABS_ERR_CUDA, "allocating the context failed: %s", cudaGetErrorString(e));
    if (ctx->workspace) cudaFree(ctx->workspace);
    if (ctx->flags) cudaFree(ctx->flags);
    delete ctx;
    return ABS_ERR_CUDA;
  }
  *out = ctx;
  return ABS_OK;
}

extern "C" int abs_destroy(abs_ctx* ctx) {
  if (ctx == nullptr) return ABS_OK;
  DeviceScope scope(ctx->device);
  if (ctx->workspace) cudaFree(ctx->workspace);
  if (ctx->flags) cudaFree(ctx->flags);
  if (ctx->staging) cudaFree(ctx->staging);
  if (ctx->staging_out) cudaFree(ctx->staging_out);
  delete ctx;
  return ABS_OK;
}

extern "C" const char* abs_last_error(const abs_ctx* ctx) { return ctx != nullptr ? ctx->err : g_create_error; }

extern "C" int abs_set_tuning(abs_ctx* ctx, const char* key, long long value) {
  if (ctx == nullptr || key == nullptr) return ABS_ERR_INVALID_ARG;
  if (value < 0) return set_error(ctx, ABS_ERR_INVALID_ARG, "tuning values are >= 0");
  if (strcmp(key, "stats_stages") == 0) {
    if (value != 0 && (value < 2 || value > 8)) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_stages must be 0 or 2..8");
    ctx->tuning.stats_stages = value;
  } else if (strcmp(key, "stats_ctas_per_worker") == 0) {
    if (value > 65535) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_ctas_per_worker must be <= 65535");
    ctx->tuning.stats_ctas_per_worker = value;
  } else if (strcmp(key, "stats_force_generic") == 0) {
    ctx->tuning.stats_force_generic = value ? 1 : 0;
  } else if (strcmp(key, "stats_flush_every") == 0) {
    if (value > 4096) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_flush_every must be <= 4096");
    ctx->tuning.stats_flush_every = value;
  } else if (strcmp(key, "stats_stage_kb") == 0) {
    if (value != 0 && (value < 4 || value > 200)) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_stage_kb must be 0 or 4..200");
    ctx->tuning.stats_stage_kb = value;
  } else if (strcmp(key, "stats_timeout_cycles") == 0) {
    if (value != 0 && (value < 100000 || value > 4000000000ll))
      return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_timeout_cycles must be 0 or 1e5..4e9");
    ctx->tuning.stats_timeout_cycles = value;
  } else if (strcmp(key, "mlp_no_tensor_cores") == 0) {
    ctx->tuning.mlp_no_tensor_cores = value ? 1 : 0;
  } else if (strcmp(key, "stats_no_secondary") == 0) {
    ctx->tuning.stats_no_secondary = value ? 1 : 0;
  } else if (strcmp(key, "stats_secondary_pct") == 0) {
    if (value > 200) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_secondary_pct must be 0..200");
    ctx->tuning.stats_secondary_pct = value;
  } else if (strcmp(key, "stats_no_recheck") == 0) {
    ctx->tuning.stats_no_recheck = value ? 1 : 0;
  } else if (strcmp(key, "stats_fault_drop_loads") == 0) {
    ctx->tuning.stats_fault_drop_loads = value ? 1 : 0;
  } else if (strcmp(key, "stats_cluster_rows") == 0) {
    if (value != 0 && (value < 16 || value > 512)) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_cluster_rows must be 0 or 16..512");
    ctx->tuning.stats_cluster_rows = value;
  } else if (strcmp(key, "stats_no_cluster") == 0) {
    ctx->tuning.stats_no_cluster = value ? 1 : 0;
  } else if (strcmp(key, "stats_no_gram") == 0) {
    ctx->tuning.stats_no_gram = value ? 1 : 0;
  } else if (strcmp(key, "stats_ctas_per_sm") == 0) {
    if (value > 2) return set_error(ctx, ABS_ERR_INVALID_ARG, "stats_ctas_per_sm must be 0, 1 or 2");
    ctx->tuning.stats_ctas_per_sm = value;
  } else {
    return set_error(ctx, ABS_ERR_INVALID_ARG, "unknown tuning key '%s'", key);
  }
  return ABS_OK;
}

extern "C" int abs_plan_stats(abs_dtype dtype, long long b, int aligned, int sm_count, size_t smem_optin,
                              abs_stats_plan* out) {
  if (out == nullptr || b < 2 || (dtype != ABS_F32 && dtype != ABS_BF16) || sm_count < 1) return ABS_ERR_INVALID_ARG;
  const Tuning t;     // the automatic choices
  int rc = ABS_ERR_UNSUPPORTED;
  if (aligned) {
    rc = plan_stats_gram(t, smem_optin, dtype, b, out);
    if (rc == ABS_ERR_UNSUPPORTED) rc = plan_stats_umma(t, smem_optin, dtype, b, out);
    if (rc == ABS_ERR_UNSUPPORTED) rc = plan_stats_cluster(t, smem_optin, dtype, b, 0, out);
    if (rc == ABS_ERR_UNSUPPORTED) rc = plan_stats_tiled(t, smem_optin, dtype, b, out);
  }
  if (rc == ABS_ERR_UNSUPPORTED) {
    memset(out, 0, sizeof(*out));
    out->route = 3;
    out->cluster_size = 1;
    out->rows_per_cta = static_cast<int>(b > 0x7fffffff ? 0x7fffffff : b);
    rc = ABS_OK;
  }
  return rc;
}

extern "C" int abs_test_stats(abs_ctx* ctx, const void* G, abs_dtype dtype, int M, long long b, long long d,
                              long long row_stride, long long worker_stride, float* gbar_out, abs_stats* stats_out,
                              void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  int rc = validate_stats(ctx, G, dtype, M, b, d, row_stride, worker_stride, stats_out);
  if (rc != ABS_OK) return rc;
  DeviceScope scope(ctx->device);
  if (!scope.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  StatsLaunch a{G, dtype, M, b, d, row_stride, worker_stride, gbar_out, stats_out, static_cast<cudaStream_t>(stream)};
  return run_stats(ctx, a);
}

extern "C" int abs_test_stats_host(abs_ctx* ctx, const void* G_host, abs_dtype dtype, int M, long long b, long long d,
                                   float* gbar_host, abs_stats* stats_host, float* gbar_dev, abs_stats* stats_dev,
                                   void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  int rc = validate_stats(ctx, G_host, dtype, M, b, d, d, b * d, stats_host);
  if (rc != ABS_OK) return rc;
  DeviceScope scope(ctx->device);
  if (!scope.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t es = dtype == ABS_F32 ? 4 : 2;
  const size_t g_bytes = static_cast<size_t>(M) * b * d * es;
  const size_t stats_bytes = (static_cast<size_t>(M) * sizeof(abs_stats) + 255) / 256 * 256;
  const bool own_gbar = gbar_host != nullptr && gbar_dev == nullptr;
  const size_t gbar_bytes = static_cast<size_t>(M) * d * sizeof(float);
  rc = grow(ctx, &ctx->staging, &ctx->staging_bytes, g_bytes);
  if (rc != ABS_OK) return rc;
  rc = grow(ctx, &ctx->staging_out, &ctx->staging_out_bytes, stats_bytes + (own_gbar ? gbar_bytes : 0));
  if (rc != ABS_OK) return rc;
  abs_stats* d_stats = stats_dev != nullptr ? stats_dev : static_cast<abs_stats*>(ctx->staging_out);
  float* d_gbar = gbar_dev;
  if (own_gbar) d_gbar = reinterpret_cast<float*>(static_cast<char*>(ctx->staging_out) + stats_bytes);
  ABS_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->staging, G_host, g_bytes, cudaMemcpyHostToDevice, st));
  StatsLaunch a{ctx->staging, dtype, M, b, d, d, b * d, d_gbar, d_stats, st};
  rc = run_stats(ctx, a);
  if (rc != ABS_OK) return rc;
  ABS_CUDA_TRY(ctx, cudaMemcpyAsync(stats_host, d_stats, static_cast<size_t>(M) * sizeof(abs_stats),
                                    cudaMemcpyDeviceToHost, st));
  if (gbar_host != nullptr)
    ABS_CUDA_TRY(ctx, cudaMemcpyAsync(gbar_host, d_gbar, gbar_bytes, cudaMemcpyDeviceToHost, st));
  ABS_CUDA_TRY(ctx, cudaStreamSynchronize(st));
  return ABS_OK;
}
