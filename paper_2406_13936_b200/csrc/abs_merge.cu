// Norm-test statistics of a batch that arrives as several sub-batches (gradient accumulation over
// micro-batches, Section 6), and per-worker batch sizes (Eq. test_stat without the maximum over
// workers, one eta_m per worker, Eq. approx_norm_local).
//
// Two disjoint sub-batches a, b with means and centred sums S = (n-1) Var (Eq. def_var) combine to
//   mean = (n_a mean_a + n_b mean_b) / n,   S = S_a + S_b + ||mean_a - mean_b||^2 n_a n_b / n,
// so a running (mean, record) pair can absorb one sub-batch after the other without ever holding
// all rows.  The inner-product and orthogonality variances need the final mean for every row and
// cannot be merged; merged records carry ABS_STATUS_NORM_ONLY.
#include "abs_internal.cuh"

namespace absk {
namespace {

constexpr int kMergeThreads = 256;

__global__ void __launch_bounds__(kMergeThreads)
merge_means_kernel(float* __restrict__ mean_a, const float* __restrict__ mean_b, long long d,
                   const abs_stats* __restrict__ ra, const abs_stats* __restrict__ rb, double* __restrict__ ws, int P) {
  __shared__ double red[2][kMergeThreads / 32];
  const int m = blockIdx.y, p = blockIdx.x, tid = threadIdx.x;
  const double na = static_cast<double>(ra[m].rows), nb = static_cast<double>(rb[m].rows);
  const float wa = static_cast<float>(na / (na + nb)), wb = static_cast<float>(nb / (na + nb));
  float* A = mean_a + static_cast<long long>(m) * d;
  const float* B = mean_b + static_cast<long long>(m) * d;
  double dsq = 0.0, msq = 0.0;
  for (long long j0 = static_cast<long long>(p) * kMergeThreads * 4; j0 < d;
       j0 += static_cast<long long>(P) * kMergeThreads * 4) {
    float dl = 0.f, ml = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long j = j0 + u * kMergeThreads + tid;
      if (j < d) {
        const float a = A[j], b = B[j];
        const float diff = a - b;
        const float mean = fmaf(wa, a, wb * b);
        A[j] = mean;
        dl = fmaf(diff, diff, dl);
        ml = fmaf(mean, mean, ml);
      }
    }
    dsq += static_cast<double>(dl);
    msq += static_cast<double>(ml);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    dsq += __shfl_xor_sync(0xffffffffu, dsq, off);
    msq += __shfl_xor_sync(0xffffffffu, msq, off);
  }
  if ((tid & 31) == 0) {
    red[0][tid >> 5] = dsq;
    red[1][tid >> 5] = msq;
  }
  __syncthreads();
  if (tid == 0) {
    double s0 = 0.0, s1 = 0.0;
    for (int w = 0; w < kMergeThreads / 32; ++w) {
      s0 += red[0][w];
      s1 += red[1][w];
    }
    ws[(static_cast<size_t>(m) * P + p) * 2] = s0;
    ws[(static_cast<size_t>(m) * P + p) * 2 + 1] = s1;
  }
}

__global__ void merge_records_kernel(abs_stats* __restrict__ ra, const abs_stats* __restrict__ rb,
                                     const double* __restrict__ ws, int P, int M) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= M) return;
  double dsq = 0.0, msq = 0.0;
  for (int p = 0; p < P; ++p) {
    dsq += ws[(static_cast<size_t>(m) * P + p) * 2];
    msq += ws[(static_cast<size_t>(m) * P + p) * 2 + 1];
  }
  const abs_stats a = ra[m], b = rb[m];
  const double na = static_cast<double>(a.rows), nb = static_cast<double>(b.rows), n = na + nb;
  const double S = (na - 1.0) * a.var_norm + (nb - 1.0) * b.var_norm + dsq * na * nb / n;
  abs_stats o;
  o.gbar_sq = msq;
  o.var_norm = S / (n - 1.0);
  o.var_ip = 0.0;
  o.var_orth = 0.0;
  o.sum_sq = S + n * msq;
  o.rows = a.rows + b.rows;
  o.status = ((a.status | b.status) & (ABS_STATUS_NONFINITE | ABS_STATUS_TIMEOUT)) | ABS_STATUS_NORM_ONLY;
  if (!(isfinite(S) && isfinite(msq))) o.status |= ABS_STATUS_NONFINITE;
  if (msq == 0.0) o.status |= ABS_STATUS_ZERO_MEAN;
  o.recomputed = 0u;
  ra[m] = o;
}

__device__ __forceinline__ double ratio_or_inf(double num, double den) {
  if (num == 0.0) return 0.0;
  if (den == 0.0) return INFINITY;
  return num / den;
}

__global__ void next_batch_local_kernel(const abs_stats* __restrict__ stats, int M, abs_test_cfg cfg,
                                        const double* __restrict__ eta_m, const long long* __restrict__ b_cur,
                                        long long* __restrict__ T_out, long long* __restrict__ b_next) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= M) return;
  const abs_stats s = stats[m];
  long long T = 0;
  const bool norm = cfg.kind == ABS_TEST_NORM;
  const bool usable = (s.status & (ABS_STATUS_NONFINITE | ABS_STATUS_TIMEOUT)) == 0u &&
                      (norm || (s.status & ABS_STATUS_NORM_ONLY) == 0u);
  if (usable) {
    const double scale = cfg.row_weight / cfg.divisor;
    const double N = s.gbar_sq;
    const double eta = eta_m != nullptr ? eta_m[m] : cfg.eta;
    double x;
    if (norm) {
      x = scale * ratio_or_inf(s.var_norm, eta * eta * N);
    } else {
      const double x_ip = scale * ratio_or_inf(s.var_ip, cfg.theta * cfg.theta * N * N);
      const double x_or = scale * ratio_or_inf(s.var_orth, cfg.nu * cfg.nu * N);
      x = x_ip > x_or ? x_ip : x_or;
    }
    T = !(x < 4611686018427387904.0) ? (1ll << 62) : static_cast<long long>(ceil(x));
  }
  if (T_out != nullptr) T_out[m] = T;
  const long long b = b_cur[m] > T ? b_cur[m] : T;
  b_next[m] = b < cfg.b_max ? b : cfg.b_max;
}

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int abs_stats_merge(abs_ctx* ctx, float* mean_a, const float* mean_b, int M, long long d, abs_stats* rec_a,
                               const abs_stats* rec_b, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (mean_a == nullptr || mean_b == nullptr || rec_a == nullptr || rec_b == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (M < 1 || M > 65535 || d < 1) return set_error(ctx, ABS_ERR_INVALID_ARG, "need 1 <= M <= 65535 and d >= 1");
  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  long long P = (d + kMergeThreads * 4 - 1) / (kMergeThreads * 4);
  const long long cap = static_cast<long long>(ctx->sm_count) * 8 / M;
  if (P > cap) P = cap < 1 ? 1 : cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double* ws = static_cast<double*>(ctx->workspace);
  cudaError_t e = cudaSuccess;
  if (static_cast<size_t>(M) * P * 2 * sizeof(double) > ctx->workspace_bytes) {
    if (prev != ctx->device) cudaSetDevice(prev);
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_stats_merge: workspace too small");
  }
  merge_means_kernel<<<dim3(static_cast<unsigned>(P), M), kMergeThreads, 0, st>>>(mean_a, mean_b, d, rec_a, rec_b, ws,
                                                                                  static_cast<int>(P));
  merge_records_kernel<<<(M + 127) / 128, 128, 0, st>>>(rec_a, rec_b, ws, static_cast<int>(P), M);
  e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) return set_error(ctx, ABS_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return ABS_OK;
}

extern "C" int abs_next_batch_local(abs_ctx* ctx, const abs_stats* stats, int M, const abs_test_cfg* cfg,
                                    const double* eta_m, const long long* b_cur, long long* T_out, long long* b_next,
                                    void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (stats == nullptr || cfg == nullptr || b_cur == nullptr || b_next == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (M < 1) return set_error(ctx, ABS_ERR_INVALID_ARG, "M must be >= 1");
  if (cfg->kind != ABS_TEST_NORM && cfg->kind != ABS_TEST_AUG_INNER_PRODUCT && cfg->kind != ABS_TEST_NORM_WORKERS)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "unknown test kind %d", cfg->kind);
  if (cfg->b_max < 1 || !(cfg->row_weight > 0.0) || !(cfg->divisor > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need b_max >= 1, row_weight > 0, divisor > 0");
  if (cfg->kind != ABS_TEST_AUG_INNER_PRODUCT ? (eta_m == nullptr && !(cfg->eta > 0.0)) : !(cfg->theta > 0.0 && cfg->nu > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "test constants must be positive");
  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  next_batch_local_kernel<<<(M + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(stats, M, *cfg, eta_m, b_cur,
                                                                                         T_out, b_next);
  const cudaError_t e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) return set_error(ctx, ABS_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return ABS_OK;
}
