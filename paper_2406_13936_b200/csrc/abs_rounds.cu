// Bookkeeping of the outer loops of Algorithm 1 and Algorithm 2 (the sample counter B, the round
// counter k, "while B < N"), and the round drivers with the per-step cadence of Algorithm 1: the
// test after every local step, b^m <- max{T^m, b^m}, per worker or with the maximum over workers.
//
// The per-step drivers launch ordinary kernels whose grids depend on the batch sizes, and the sizes
// of step h + 1 are decided on the device in step h.  So, unlike every other call of the library,
// they wait for the stream once per local step to read M integers back.  abs_logreg_rounds_fused_opts
// keeps everything on the device and is the fast way to run this cadence on the logistic problem.
#include "abs_internal.cuh"

namespace absk {
namespace {

// samples += times * sum_i sizes[i]; rounds += add_rounds.  One thread: M is small.
__global__ void round_count_kernel(abs_round_ctl* ctl, const long long* __restrict__ sizes, int n, long long times,
                                   long long add_rounds) {
  long long s = 0;
  for (int i = 0; i < n; ++i) s += sizes[i];
  ctl->samples += times * s;
  ctl->rounds += add_rounds;
}

// Every worker continues with the largest of the sizes (display below Eq. test_stat).
__global__ void share_max_kernel(long long* __restrict__ sizes, int M) {
  long long best = 0;
  for (int m = 0; m < M; ++m) best = sizes[m] > best ? sizes[m] : best;
  for (int m = 0; m < M; ++m) sizes[m] = best;
}

struct DeviceScopeR {
  int prev = -1;
  bool ok = true;
  explicit DeviceScopeR(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceScopeR() { if (prev >= 0) cudaSetDevice(prev); }
};

// The part both problems share.  `produce(m0, nm, b, h, rows_before)` enqueues, for the workers
// m0 .. m0 + nm - 1 that all have batch size b at step h, the batch gradients into Gb[m0..] and the
// records into stats[h][m0..]; rows_before = the rows the groups before this one used in this step.
template <typename Produce>
int round_per_step(abs_ctx* ctx, float* X, int M, int H, long long d, long long* b_host, float lr,
                   const abs_test_cfg* cfg, const abs_round_opts* opts, float* Gb, abs_stats* stats, long long* T_out,
                   long long* b_dev, cudaStream_t st, Produce produce) {
  if (H < 1 || M < 1) return set_error(ctx, ABS_ERR_INVALID_ARG, "need H >= 1 and M >= 1");
  if (cfg->kind == ABS_TEST_NORM_WORKERS)
    return set_error(ctx, ABS_ERR_UNSUPPORTED, "the test on the workers' batch gradients runs once per round (Algorithm 2)");
  const bool per_worker = opts != nullptr && opts->per_worker != 0;
  const double* eta_m = opts != nullptr ? opts->eta_m : nullptr;
  abs_round_ctl* ctl = opts != nullptr ? opts->ctl : nullptr;
  for (int m = 0; m < M; ++m) {
    if (b_host[m] > cfg->b_max) b_host[m] = cfg->b_max;
    if (b_host[m] < 2) return set_error(ctx, ABS_ERR_INVALID_ARG, "worker %d has batch size %lld < 2", m, b_host[m]);
  }
  ABS_CUDA_TRY(ctx, cudaMemcpyAsync(b_dev, b_host, sizeof(long long) * M, cudaMemcpyHostToDevice, st));
  for (int h = 0; h < H; ++h) {
    long long rows_before = 0;
    for (int m0 = 0; m0 < M;) {
      int nm = 1;
      while (m0 + nm < M && b_host[m0 + nm] == b_host[m0]) ++nm;     // neighbours of equal size share launches
      const int rc = produce(m0, nm, b_host[m0], h, rows_before);
      if (rc != ABS_OK) return rc;
      rows_before += static_cast<long long>(nm) * b_host[m0];
      m0 += nm;
    }
    abs_stats* stats_h = stats + static_cast<long long>(h) * M;
    if (ctl != nullptr) {
      round_count_kernel<<<1, 1, 0, st>>>(ctl, b_dev, M, 1, h == H - 1 ? 1 : 0);     // B += sum_m b^m_{k,h}
      ABS_CUDA_TRY(ctx, cudaGetLastError());
    }
    int rc = abs_next_batch_local(ctx, stats_h, M, cfg, eta_m, b_dev,
                                  T_out != nullptr ? T_out + static_cast<long long>(h) * M : nullptr, b_dev, st);
    if (rc != ABS_OK) return rc;
    if (!per_worker) {
      share_max_kernel<<<1, 1, 0, st>>>(b_dev, M);
      ABS_CUDA_TRY(ctx, cudaGetLastError());
    }
    rc = local_sgd_step(ctx, X, Gb, M, d, d, lr, h == H - 1 ? 1 : 0, st);
    if (rc != ABS_OK) return rc;
    ABS_CUDA_TRY(ctx, cudaMemcpyAsync(b_host, b_dev, sizeof(long long) * M, cudaMemcpyDeviceToHost, st));
    ABS_CUDA_TRY(ctx, cudaStreamSynchronize(st));                    // the next step's launches need the sizes
  }
  return ABS_OK;
}

}  // namespace
}  // namespace absk

using namespace absk;

// The end of a round under Algorithm 2 as printed: statistics of the M workers' batch gradients
// (rows of Gb [M][d]) into stats[0], T and the size update with row_weight = b and divisor = M.
int absk::worker_gradient_test(abs_ctx* ctx, const float* Gb, int M, long long d, long long b, const abs_test_cfg* cfg,
                               abs_stats* stats, long long* T_out, long long* b_dev, void* stream) {
  if (M < 2) return set_error(ctx, ABS_ERR_INVALID_ARG, "the variance over the workers needs M >= 2");
  int rc = abs_test_stats(ctx, Gb, ABS_F32, 1, M, d, d, static_cast<long long>(M) * d, nullptr, stats, stream);
  if (rc != ABS_OK) return rc;
  abs_test_cfg c = *cfg;
  c.kind = ABS_TEST_NORM;
  c.row_weight = static_cast<double>(b);     // a row is the mean of b samples (Section 4.3)
  c.divisor = static_cast<double>(M);        // Eq. test_stat_actual
  return abs_next_batch(ctx, stats, 1, &c, b_dev, T_out, b_dev, stream);
}

extern "C" int abs_round_count(abs_ctx* ctx, abs_round_ctl* ctl, const long long* sizes, int n, long long times,
                               long long add_rounds, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (ctl == nullptr || sizes == nullptr || n < 1 || times < 0 || add_rounds < 0)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need ctl, sizes, n >= 1, times >= 0, add_rounds >= 0");
  DeviceScopeR scope(ctx->device);
  if (!scope.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  round_count_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(ctl, sizes, n, times, add_rounds);
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  return ABS_OK;
}

extern "C" int abs_logreg_round_per_step(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                         const int* idx, long long idx_stride, float* X, int M, int H,
                                         long long* b_host, float lr, const abs_test_cfg* cfg,
                                         const abs_round_opts* opts, float* G_scratch, float* Gb_scratch,
                                         abs_stats* stats, long long* T_out, long long* b_dev, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (cfg == nullptr || b_host == nullptr || G_scratch == nullptr || Gb_scratch == nullptr || stats == nullptr ||
      b_dev == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  DeviceScopeR scope(ctx->device);
  if (!scope.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto produce = [&](int m0, int nm, long long b, int h, long long rows_before) -> int {
    const int* idx_h = idx + (static_cast<long long>(h) * M + m0) * idx_stride;
    float* G = G_scratch + rows_before * d;
    int rc = abs_logreg_grads(ctx, A, y, n, d, idx_h, idx_stride, X + static_cast<long long>(m0) * d, nm, b, G, st);
    if (rc != ABS_OK) return rc;
    return abs_test_stats(ctx, G, ABS_F32, nm, b, d, d, b * d, Gb_scratch + static_cast<long long>(m0) * d,
                          stats + static_cast<long long>(h) * M + m0, st);
  };
  return round_per_step(ctx, X, M, H, d, b_host, lr, cfg, opts, Gb_scratch, stats, T_out, b_dev, st, produce);
}

extern "C" int abs_mlp_round_per_step(abs_ctx* ctx, const float* inputs, const int* labels, long long n,
                                      const int* dims, const int* idx, long long idx_stride, float* X, int M, int H,
                                      long long* b_host, float lr, const abs_test_cfg* cfg, const abs_round_opts* opts,
                                      void* scratch, size_t scratch_bytes, float* Gb_scratch, abs_stats* stats,
                                      long long* T_out, long long* b_dev, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (cfg == nullptr || b_host == nullptr || dims == nullptr || Gb_scratch == nullptr || stats == nullptr ||
      b_dev == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  long long d = 0;
  int rc = abs_mlp_param_count(dims, &d);
  if (rc != ABS_OK) return set_error(ctx, rc, "invalid layer widths");
  DeviceScopeR scope(ctx->device);
  if (!scope.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto produce = [&](int m0, int nm, long long b, int h, long long) -> int {
    const int* idx_h = idx + (static_cast<long long>(h) * M + m0) * idx_stride;
    float* Gb = Gb_scratch + static_cast<long long>(m0) * d;
    int r = abs_mlp_grads(ctx, inputs, labels, n, dims, idx_h, idx_stride, X + static_cast<long long>(m0) * d, nm, b,
                          Gb, scratch, scratch_bytes, st);
    if (r != ABS_OK) return r;
    // the statistics straight from activations and deltas: no per-sample gradient matrix
    return abs_mlp_fused_stats(ctx, dims, b, nm, scratch, scratch_bytes, Gb, stats + static_cast<long long>(h) * M + m0,
                               st);
  };
  return round_per_step(ctx, X, M, H, d, b_host, lr, cfg, opts, Gb_scratch, stats, T_out, b_dev, st, produce);
}
