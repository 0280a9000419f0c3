// Producers of per-sample gradients for the two synthetic end-to-end problems (Algorithm 1,
// per-sample gradient step; Algorithm 2 for the round structure), and the round drivers
// that chain producer -> statistics -> local SGD step -> averaging -> batch-size update.
//
//   logistic regression   g_i = (sigmoid(a_i^T x) - y_i) a_i
//   ReLU MLP              softmax cross-entropy; per-sample gradients are outer products
//                         delta_l,i (x) h_{l-1},i, written out row by row when the test needs them
//
// These kernels feed the hot path.  The logistic producer is plain fp32 CUDA-core code; the MLP's
// matrix products run on the tensor cores with operands split so that the result keeps fp32
// accuracy (abs_gemm_tc.cu), which the parity bound on the parameters, 1e-6, needs.
#include "abs_internal.cuh"

namespace absk {
namespace {

struct DeviceScopeP {
  int prev = -1;
  bool ok = true;
  explicit DeviceScopeP(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceScopeP() { if (prev >= 0) cudaSetDevice(prev); }
};

// ---- logistic regression --------------------------------------------------------------------
// One warp per (worker, sample): dot product, sigmoid, scaled copy of the feature row.
__global__ void __launch_bounds__(256)
logreg_grads_kernel(const float* __restrict__ A, const float* __restrict__ y, long long n, long long d,
                    const int* __restrict__ idx, long long idx_stride, const float* __restrict__ X, int M,
                    long long b, float* __restrict__ G) {
  const long long w = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= static_cast<long long>(M) * b) return;
  const int m = static_cast<int>(w / b);
  const long long i = w % b;
  // indices outside the data are clamped, as in the fused rounds: never an out-of-range read
  const long long raw = idx[static_cast<long long>(m) * idx_stride + i];
  const long long row = raw < 0 ? 0 : (raw >= n ? n - 1 : raw);
  const float* a = A + row * d;
  const float* x = X + static_cast<long long>(m) * d;
  float z = 0.f;
  for (long long j = lane; j < d; j += 32) z = fmaf(a[j], x[j], z);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
  // sigmoid(z) - label; for the labels 1 and 0 nothing is subtracted (sigmoid(z) - 1 = -sigmoid(-z)),
  // so a well-fitted sample, whose residual is tiny, keeps its relative accuracy
  const float ez = expf(-fabsf(z));
  const float big = 1.f / (1.f + ez), small = ez * big;          // sigmoid(|z|), sigmoid(-|z|)
  const float p = z >= 0.f ? big : small, q = z >= 0.f ? small : big;
  const float label = y[row];
  const float r = label == 1.f ? -q : (label == 0.f ? p : p - label);
  float* g = G + (static_cast<long long>(m) * b + i) * d;
  for (long long j = lane; j < d; j += 32) g[j] = r * a[j];
}

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int abs_logreg_grads(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                const int* idx, long long idx_stride, const float* X, int M, long long b, float* G,
                                void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (A == nullptr || y == nullptr || idx == nullptr || X == nullptr || G == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (n < 1 || d < 1 || M < 1 || b < 1 || idx_stride < b)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need n, d, M, b >= 1 and idx_stride >= b");
  DeviceScopeP scope(ctx->device);
  if (!scope.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  const long long warps = static_cast<long long>(M) * b;
  const long long blocks = (warps * 32 + 255) / 256;
  logreg_grads_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      A, y, n, d, idx, idx_stride, X, M, b, G);
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  return ABS_OK;
}

// One communication round of local SGD on the logistic problem (Algorithm 2 structure with the
// per-sample statistic of Algorithm 1, evaluated once per round on the last local step).
extern "C" int abs_logreg_round(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                const int* idx, long long idx_stride, float* X, int M, int H, long long b, float lr,
                                const abs_test_cfg* cfg, float* G_scratch, float* Gb_scratch, abs_stats* stats,
                                long long* T_out, long long* b_dev, abs_round_ctl* ctl, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (cfg == nullptr || G_scratch == nullptr || Gb_scratch == nullptr || stats == nullptr || b_dev == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (H < 1 || b < 2) return set_error(ctx, ABS_ERR_INVALID_ARG, "need H >= 1 and b >= 2");
  for (int h = 0; h < H; ++h) {
    const int* idx_h = idx + static_cast<long long>(h) * M * idx_stride;
    int rc = abs_logreg_grads(ctx, A, y, n, d, idx_h, idx_stride, X, M, b, G_scratch, stream);
    if (rc != ABS_OK) return rc;
    // the statistics kernel also delivers the batch gradient (the column means) for the step
    rc = abs_test_stats(ctx, G_scratch, ABS_F32, M, b, d, d, b * d, Gb_scratch, stats, stream);
    if (rc != ABS_OK) return rc;
    rc = local_sgd_step(ctx, X, Gb_scratch, M, d, d, lr, h == H - 1 ? 1 : 0, stream);
    if (rc != ABS_OK) return rc;
  }
  if (ctl != nullptr) {      // Alg. 2: B <- B + H M b_k, k <- k + 1 (with the size the round ran with)
    const int rc = abs_round_count(ctx, ctl, b_dev, 1, static_cast<long long>(H) * M, 1, stream);
    if (rc != ABS_OK) return rc;
  }
  if (cfg->kind == ABS_TEST_NORM_WORKERS)
    return worker_gradient_test(ctx, Gb_scratch, M, d, b, cfg, stats, T_out, b_dev, stream);
  return abs_next_batch(ctx, stats, M, cfg, b_dev, T_out, b_dev, stream);
}
