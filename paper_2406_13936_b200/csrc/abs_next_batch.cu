// Next local batch size from the per-worker statistics (Eq. norm_test, Eq. test_stat,
// Algorithm 1: b <- max{T, b}; maximum over workers; cap).  All arithmetic that decides
// the integer is fp64, in the order  scale * (variance / (constant^2 * N [* N])).
#include "abs_internal.cuh"

namespace absk {
namespace {

constexpr int kThreads = 1024;

__global__ void __launch_bounds__(kThreads)
abs_next_batch_kernel(const abs_stats* __restrict__ stats, int M, abs_test_cfg cfg,
                      const long long* __restrict__ b_cur, long long* __restrict__ T_out,
                      long long* __restrict__ b_next) {
  __shared__ long long red[kThreads / 32];
  const int tid = threadIdx.x;
  long long T = 0;
  pdl_wait();                    // the records (and b_cur) written by the kernels before
  pdl_launch_dependents();
  if (tid < M) {
    T = test_size_from_record(stats[tid], cfg);
    if (T_out != nullptr) T_out[tid] = T;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const long long o = __shfl_xor_sync(0xffffffffu, T, off);
    T = o > T ? o : T;
  }
  if ((tid & 31) == 0) red[tid >> 5] = T;
  __syncthreads();
  if (tid == 0) {
    long long best = b_cur[0];
    for (int w = 0; w < kThreads / 32; ++w) best = red[w] > best ? red[w] : best;
    b_next[0] = best < cfg.b_max ? best : cfg.b_max;
  }
}

}  // namespace
}  // namespace absk

extern "C" int abs_next_batch(abs_ctx* ctx, const abs_stats* stats, int M, const abs_test_cfg* cfg,
                              const long long* b_cur, long long* T_out, long long* b_next, void* stream) {
  using namespace absk;
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (stats == nullptr || cfg == nullptr || b_cur == nullptr || b_next == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (M < 1 || M > kThreads) return set_error(ctx, ABS_ERR_INVALID_ARG, "M must be in 1..%d, got %d", kThreads, M);
  if (cfg->kind != ABS_TEST_NORM && cfg->kind != ABS_TEST_AUG_INNER_PRODUCT && cfg->kind != ABS_TEST_NORM_WORKERS)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "unknown test kind %d", cfg->kind);
  if (cfg->b_max < 1 || !(cfg->row_weight > 0.0) || !(cfg->divisor > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need b_max >= 1, row_weight > 0, divisor > 0");
  if (cfg->kind != ABS_TEST_AUG_INNER_PRODUCT ? !(cfg->eta > 0.0) : !(cfg->theta > 0.0 && cfg->nu > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "test constants must be positive");
  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  const cudaError_t e = launch_dependent(abs_next_batch_kernel, dim3(1), dim3(kThreads), 0,
                                         static_cast<cudaStream_t>(stream), stats, M, *cfg, b_cur, T_out, b_next);
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) return set_error(ctx, ABS_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return ABS_OK;
}
