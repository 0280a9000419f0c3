// abs_test_stats_noalloc: the batch-size-test statistics for callers that must not allocate.
//
// Who needs this: code that runs where device allocation is forbidden or would stall --
// a training loop whose memory is entirely handed out by a caching allocator that must
// not see foreign cudaMalloc calls, a library plugged into a host application with a
// fixed memory budget, a latency-critical section in which the implicit device
// synchronisation of cudaMalloc / cudaFree is not acceptable.  abs_create allocates a
// workspace; this entry point needs no context and takes its scratch (the per-CTA
// partial sums and the status word of the statistics kernels) from a fixed array that
// is part of the loaded library image on every GPU.
#include <mutex>

#include "abs_internal.cuh"

namespace {

constexpr size_t kScratchBytes = ABS_NOALLOC_SCRATCH_BYTES;   // partial sums
constexpr size_t kFlagBytes = 256;                            // status words, kept apart from the sums
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime; the
// device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes + kFlagBytes];

struct DeviceSlot {
  bool ready = false;
  void* scratch = nullptr;
  int sm_count = 0;
  size_t smem_optin = 0;
};
DeviceSlot g_slots[kMaxDevices];
std::mutex g_slots_mutex;

// First call on a device: resolves the device address of the scratch array and reads the
// device attributes the launch heuristics need.  Allocates nothing.
int prepare_device(int device, DeviceSlot* out, char* err, size_t err_len) {
  std::lock_guard<std::mutex> lock(g_slots_mutex);
  DeviceSlot& slot = g_slots[device];
  if (!slot.ready) {
    int major = 0, sms = 0, optin = 0;
    cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) {
      snprintf(err, err_len, "cannot query device %d: %s", device, cudaGetErrorString(e));
      return ABS_ERR_CUDA;
    }
    if (major != 10) {
      snprintf(err, err_len, "device %d has compute capability %d.x; the kernels are built for 10.x only", device, major);
      return ABS_ERR_NO_DEVICE;
    }
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);     // device `device` is current here
    if (e != cudaSuccess || ptr == nullptr) {
      snprintf(err, err_len, "cudaGetSymbolAddress on the scratch array failed: %s", cudaGetErrorString(e));
      return ABS_ERR_CUDA;
    }
    slot.scratch = ptr;
    slot.sm_count = sms;
    slot.smem_optin = static_cast<size_t>(optin);
    slot.ready = true;
  }
  *out = slot;
  return ABS_OK;
}

thread_local char g_noalloc_error[512] = {0};

}  // namespace

extern "C" const char* abs_noalloc_last_error(void) { return g_noalloc_error; }

extern "C" int abs_test_stats_noalloc(const void* G, abs_dtype dtype, int M, long long b, long long d,
                                      long long row_stride, long long worker_stride, float* gbar_out,
                                      abs_stats* stats_out, void* stream) {
  using namespace absk;
  char* err = g_noalloc_error;
  const size_t err_len = sizeof(g_noalloc_error);
  err[0] = 0;
  if (G == nullptr || stats_out == nullptr) { snprintf(err, err_len, "G or stats_out is null"); return ABS_ERR_INVALID_ARG; }
  if (dtype != ABS_F32 && dtype != ABS_BF16) { snprintf(err, err_len, "unknown dtype %d", (int)dtype); return ABS_ERR_INVALID_ARG; }
  if (M < 1 || b < 2 || d < 1 || row_stride < d || (M > 1 && worker_stride < (b - 1) * row_stride + d)) {
    snprintf(err, err_len, "need M >= 1, b >= 2, d >= 1, row_stride >= d and non-overlapping workers");
    return ABS_ERR_INVALID_ARG;
  }
  if (b > ABS_NOALLOC_MAX_ROWS || M > ABS_NOALLOC_MAX_WORKERS) {
    snprintf(err, err_len, "abs_test_stats_noalloc covers b <= %d rows and M <= %d workers (got b=%lld, M=%d): "
             "its scratch is a fixed %zu-byte array; use abs_test_stats with a context for larger problems",
             ABS_NOALLOC_MAX_ROWS, ABS_NOALLOC_MAX_WORKERS, b, M, kScratchBytes);
    return ABS_ERR_UNSUPPORTED;
  }
  int device = -1;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess || device < 0 || device >= kMaxDevices) {
    snprintf(err, err_len, "no usable current CUDA device (%s)", cudaGetErrorString(e));
    cudaGetLastError();
    return ABS_ERR_NO_DEVICE;
  }
  DeviceSlot slot;
  int rc = prepare_device(device, &slot, err, err_len);
  if (rc != ABS_OK) return rc;

  // A context on the stack that points at the static scratch: the launchers below only
  // read it.  Nothing here is allocated, and nothing outlives the call.
  abs_ctx ctx;
  ctx.device = device;
  ctx.sm_count = slot.sm_count;
  ctx.smem_optin = slot.smem_optin;
  ctx.workspace = slot.scratch;
  ctx.workspace_bytes = kScratchBytes;
  ctx.flags = reinterpret_cast<unsigned*>(static_cast<unsigned char*>(slot.scratch) + kScratchBytes);

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  StatsLaunch a{G, dtype, M, b, d, row_stride, worker_stride, gbar_out, stats_out, st};
  // The array keeps whatever the previous call left: the status word must start at zero
  // (the partial sums are fully overwritten by the statistics kernels before they are read).
  e = cudaMemsetAsync(ctx.flags, 0, sizeof(unsigned), st);
  if (e != cudaSuccess) { snprintf(err, err_len, "cudaMemsetAsync failed: %s", cudaGetErrorString(e)); return ABS_ERR_CUDA; }
  int P = 0;
  rc = launch_stats_tiled(&ctx, a, &P);
  if (rc == ABS_ERR_UNSUPPORTED) rc = launch_stats_generic(&ctx, a, &P);
  if (rc == ABS_OK) rc = launch_stats_finalize(&ctx, a, P);
  if (rc != ABS_OK) snprintf(err, err_len, "%s", ctx.err[0] ? ctx.err : "statistics launch failed");
  return rc;
}
