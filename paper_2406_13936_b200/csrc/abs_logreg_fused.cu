// Whole communication rounds of local SGD on the logistic problem in ONE cooperative launch
// (Algorithm 2's structure with Algorithm 1's per-sample statistic once per round, Section 4.3).
//
// The round driver abs_logreg_round enqueues about four small kernels per local step; for a
// problem of a few hundred parameters every one of them is pure launch latency.  Here a grid of
// M x P resident CTAs (P CTAs per worker, all co-resident: cooperative launch) keeps the
// parameters of its worker in shared memory and walks through the steps with one grid-wide
// barrier per local step:
//
//   phase A   every warp takes samples of the step's batch: z = <a_i, x>, r_i = sigmoid(z) - y_i,
//             and adds r_i a_i to its partial batch gradient; one partial per CTA goes to global
//             memory
//   barrier
//   phase B   every CTA of the worker adds the P partials in a fixed order -> gbar (Eq. batch_grad)
//             and takes the step x <- x - lr gbar (Eq. local_sgd_alt); all CTAs of a worker do the
//             same arithmetic, so their copies of x stay bit-identical
//   last step of a round, between B and the update:
//   phase C   the CTA's samples again (from L1/L2): sum_i ||g_i - gbar||^2, e_i = <g_i - gbar, gbar>
//             (Eq. def_var, centred), partial sums per CTA in fp64
//   barrier
//   phase D   model averaging over the M workers (Eq. local_sgd_alt, second line), the records,
//             T per worker, b <- min(b_max, max(b, max_m T_m)) (Algorithm 1) - computed by every
//             CTA from the same numbers, so the next round's batch size needs no further barrier
//             and never leaves the device.
//
// The per-sample gradient matrix is never written.  Data written by one CTA and read by another
// inside the launch goes through L2 only (st.cg / ld.cg); buffers are reused no sooner than two
// barriers later.  Every CTA executes the same sequence of barriers: the trip counts depend only
// on (rounds, H) and on b, which all CTAs derive from the same values.
#include <cooperative_groups.h>

#include "abs_internal.cuh"

namespace cg = cooperative_groups;

namespace absk {
namespace {

constexpr int kFW = 8;                     // warps per CTA
constexpr int kFThreads = kFW * 32;
constexpr int kMaxWorkersFused = 64;
constexpr int kMaxDimFused = 1024;
constexpr int kMaxCtasPerWorker = 32;

struct FusedParams {
  const float* A;
  const float* y;
  long long n;
  int d;
  const int* idx;
  long long idx_stride;
  int rounds, M, H, P;
  float lr;
  abs_test_cfg cfg;
  float* X;
  abs_stats* stats;
  long long* T_out;
  long long* b_hist;
  long long* b_dev;
  float* partial;   // [2][M][P][d]   partial batch gradients, two buffers alternate by step
  double* S;        // [M][P][4]      V, sum e, sum e^2, N
  float* Xpre;      // [M][d]         parameters before the averaging
};

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}
__device__ __forceinline__ double warp_sum_dd(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}
__device__ __forceinline__ float dot4(const float4 a, const float4 b, float acc) {
  acc = fmaf(a.x, b.x, acc);
  acc = fmaf(a.y, b.y, acc);
  acc = fmaf(a.z, b.z, acc);
  return fmaf(a.w, b.w, acc);
}
// numerically stable logistic function minus the label
__device__ __forceinline__ float residual(float z, float label) {
  const float ez = expf(-fabsf(z));
  const float p = z >= 0.f ? 1.f / (1.f + ez) : ez / (1.f + ez);
  return p - label;
}

// KV: 16-byte column vectors per lane (slot k of a lane is vector k*32 + lane of the row).
template <int KV>
__global__ void __launch_bounds__(kFThreads, 1) logreg_rounds_kernel(const FusedParams prm) {
  cg::grid_group grid = cg::this_grid();
  extern __shared__ __align__(16) float smem_f[];
  const int d = prm.d, DV = d >> 2;
  float4* x4 = reinterpret_cast<float4*>(smem_f);              // [DV] parameters of this worker
  float4* g4 = x4 + DV;                                         // [DV] batch gradient of the step
  float4* wacc4 = g4 + DV;                                      // [kFW][DV] per-warp partial sums
  __shared__ double red[kFW][3];
  __shared__ double N_s;
  __shared__ long long T_s[kMaxWorkersFused];
  __shared__ long long b_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int M = prm.M, P = prm.P;
  const int m = blockIdx.x / P, p = blockIdx.x % P;
  const float4* A4 = reinterpret_cast<const float4*>(prm.A);
  float4* X4 = reinterpret_cast<float4*>(prm.X);
  float4* Xpre4 = reinterpret_cast<float4*>(prm.Xpre);
  const float lr = prm.lr;

  for (int j = tid; j < DV; j += kFThreads) x4[j] = X4[static_cast<long long>(m) * DV + j];
  long long b = prm.b_dev[0];
  if (b > prm.cfg.b_max) b = prm.cfg.b_max;
  if (b < 2) b = 2;                        // the variance needs two rows
  if (blockIdx.x == 0 && tid == 0 && prm.b_hist != nullptr) prm.b_hist[0] = b;
  __syncthreads();

  // Row index and label of the warp's t-th sample of the step are fetched by lane t % 32 ahead
  // of the loop over the samples, so that the loop's loads do not wait for an index first.
  const long long first = p + static_cast<long long>(P) * warp;     // this warp's first sample
  const long long hop = static_cast<long long>(P) * kFW;

  for (int r = 0; r < prm.rounds; ++r) {
    const int Pa = static_cast<int>(b < P ? b : P);                 // CTAs of a worker that have samples
    const long long n_mine = b > first ? (b - first + hop - 1) / hop : 0;
    const float inv_b = 1.0f / static_cast<float>(b);
    for (int h = 0; h < prm.H; ++h) {
      const long long gstep = static_cast<long long>(r) * prm.H + h;
      const bool last = h == prm.H - 1;
      const int* idx_m = prm.idx + (gstep * M + m) * prm.idx_stride;
      float4* part4 = reinterpret_cast<float4*>(prm.partial) + (gstep & 1) * static_cast<long long>(M) * P * DV;

      // ---- phase A: partial batch gradient of this CTA ------------------------------------
      float4 acc[KV];
#pragma unroll
      for (int k = 0; k < KV; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (long long t0 = 0; t0 < n_mine; t0 += 32) {
        const int cnt = static_cast<int>(n_mine - t0 < 32 ? n_mine - t0 : 32);
        long long my_row = 0;
        float my_label = 0.f;
        if (lane < cnt) {
          long long row = idx_m[first + (t0 + lane) * hop];
          row = row < 0 ? 0 : (row >= prm.n ? prm.n - 1 : row);     // indices outside the data are clamped
          my_row = row;
          my_label = prm.y[row];
        }
        for (int t = 0; t < cnt; t += 2) {
          const bool two = t + 1 < cnt;
          const long long row0 = __shfl_sync(0xffffffffu, my_row, t);
          const long long row1 = __shfl_sync(0xffffffffu, my_row, two ? t + 1 : t);
          const float lab0 = __shfl_sync(0xffffffffu, my_label, t);
          const float lab1 = __shfl_sync(0xffffffffu, my_label, two ? t + 1 : t);
          float4 a0[KV], a1[KV];
          float z0 = 0.f, z1 = 0.f;
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              a0[k] = __ldg(A4 + row0 * DV + j);
              a1[k] = __ldg(A4 + row1 * DV + j);
            } else {
              a0[k] = a1[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
          }
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              const float4 xv = x4[j];
              z0 = dot4(a0[k], xv, z0);
              z1 = dot4(a1[k], xv, z1);
            }
          }
          z0 = warp_sum_f(z0);
          z1 = warp_sum_f(z1);
          const float r0 = residual(z0, lab0);
          const float r1 = two ? residual(z1, lab1) : 0.f;
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            acc[k].x = fmaf(r0, a0[k].x, acc[k].x);
            acc[k].y = fmaf(r0, a0[k].y, acc[k].y);
            acc[k].z = fmaf(r0, a0[k].z, acc[k].z);
            acc[k].w = fmaf(r0, a0[k].w, acc[k].w);
            acc[k].x = fmaf(r1, a1[k].x, acc[k].x);
            acc[k].y = fmaf(r1, a1[k].y, acc[k].y);
            acc[k].z = fmaf(r1, a1[k].z, acc[k].z);
            acc[k].w = fmaf(r1, a1[k].w, acc[k].w);
          }
        }
      }
#pragma unroll
      for (int k = 0; k < KV; ++k) {
        const int j = k * 32 + lane;
        if (j < DV) wacc4[warp * DV + j] = acc[k];
      }
      __syncthreads();
      if (p < Pa) {
        for (int j = tid; j < DV; j += kFThreads) {
          float4 s = wacc4[j];
#pragma unroll
          for (int w = 1; w < kFW; ++w) {
            const float4 v = wacc4[w * DV + j];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          __stcg(part4 + (static_cast<long long>(m) * P + p) * DV + j, s);
        }
      }
      grid.sync();

      // ---- phase B: batch gradient of the worker; the step unless statistics come first -----
      // The P partials are split over thread groups (group q takes partials q, q + groups, ...),
      // then the groups' sums are added in group order.
      {
        const int groups = kFThreads / DV >= kFW ? kFW : (kFThreads / DV > 0 ? kFThreads / DV : 1);   // wacc4 has kFW rows
        const int grp = tid / DV, j = tid - grp * DV;
        if (grp < groups) {
          float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
          const float4* src = part4 + static_cast<long long>(m) * P * DV + j;
#pragma unroll 4
          for (int q = grp; q < Pa; q += groups) {
            const float4 v = __ldcg(src + static_cast<long long>(q) * DV);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          wacc4[grp * DV + j] = s;
        }
        __syncthreads();
        for (int jj = tid; jj < DV; jj += kFThreads) {
          float4 s = wacc4[jj];
          for (int q = 1; q < groups; ++q) {
            const float4 v = wacc4[q * DV + jj];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          s.x *= inv_b; s.y *= inv_b; s.z *= inv_b; s.w *= inv_b;
          g4[jj] = s;
          if (!last) {
            float4 xv = x4[jj];
            xv.x = fmaf(-lr, s.x, xv.x); xv.y = fmaf(-lr, s.y, xv.y);
            xv.z = fmaf(-lr, s.z, xv.z); xv.w = fmaf(-lr, s.w, xv.w);
            x4[jj] = xv;
          }
        }
        __syncthreads();
      }
      if (!last) continue;

      // ---- phase C: statistics of the last local step's per-sample gradients -----------------
      if (warp == 0) {
        const float* g = reinterpret_cast<const float*>(g4);
        double s = 0.0;
        for (int j = lane; j < d; j += 32) s += static_cast<double>(g[j]) * static_cast<double>(g[j]);
        s = warp_sum_dd(s);
        if (lane == 0) N_s = s;
      }
      double V = 0.0, se = 0.0, see = 0.0;
      for (long long t0 = 0; t0 < n_mine; t0 += 32) {
        const int cnt = static_cast<int>(n_mine - t0 < 32 ? n_mine - t0 : 32);
        long long my_row = 0;
        float my_label = 0.f;
        if (lane < cnt) {
          long long row = idx_m[first + (t0 + lane) * hop];
          row = row < 0 ? 0 : (row >= prm.n ? prm.n - 1 : row);
          my_row = row;
          my_label = prm.y[row];
        }
        for (int t = 0; t < cnt; ++t) {
          const long long row = __shfl_sync(0xffffffffu, my_row, t);
          const float lab = __shfl_sync(0xffffffffu, my_label, t);
          float4 a[KV];
          float z = 0.f;
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              a[k] = __ldg(A4 + row * DV + j);
              z = dot4(a[k], x4[j], z);
            }
          }
          z = warp_sum_f(z);
          const float rr = residual(z, lab);
          float s1 = 0.f, s2 = 0.f;
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              const float4 gv = g4[j];
              const float tx = fmaf(rr, a[k].x, -gv.x), ty = fmaf(rr, a[k].y, -gv.y);
              const float tz = fmaf(rr, a[k].z, -gv.z), tw = fmaf(rr, a[k].w, -gv.w);
              s1 = fmaf(tx, tx, s1); s1 = fmaf(ty, ty, s1); s1 = fmaf(tz, tz, s1); s1 = fmaf(tw, tw, s1);
              s2 = fmaf(tx, gv.x, s2); s2 = fmaf(ty, gv.y, s2); s2 = fmaf(tz, gv.z, s2); s2 = fmaf(tw, gv.w, s2);
            }
          }
          s1 = warp_sum_f(s1);
          s2 = warp_sum_f(s2);
          V += static_cast<double>(s1);
          se += static_cast<double>(s2);
          see += static_cast<double>(s2) * static_cast<double>(s2);
        }
      }
      if (lane == 0) {
        red[warp][0] = V;
        red[warp][1] = se;
        red[warp][2] = see;
      }
      __syncthreads();
      if (tid == 0 && p < Pa) {
        double a0 = 0.0, a1 = 0.0, a2 = 0.0;
        for (int w = 0; w < kFW; ++w) {
          a0 += red[w][0];
          a1 += red[w][1];
          a2 += red[w][2];
        }
        double* dst = prm.S + (static_cast<long long>(m) * P + p) * 4;
        __stcg(dst + 0, a0);
        __stcg(dst + 1, a1);
        __stcg(dst + 2, a2);
        __stcg(dst + 3, N_s);
      }
      // the step that was held back, and this worker's parameters for the averaging
      for (int j = tid; j < DV; j += kFThreads) {
        const float4 s = g4[j];
        float4 xv = x4[j];
        xv.x = fmaf(-lr, s.x, xv.x); xv.y = fmaf(-lr, s.y, xv.y);
        xv.z = fmaf(-lr, s.z, xv.z); xv.w = fmaf(-lr, s.w, xv.w);
        x4[j] = xv;
        if (p == 0) __stcg(Xpre4 + static_cast<long long>(m) * DV + j, xv);
      }
      grid.sync();

      // ---- phase D: averaging, records, next batch size ---------------------------------------
      const float inv_M = 1.0f / static_cast<float>(M);
      for (int j = tid; j < DV; j += kFThreads) {
        float4 s = __ldcg(Xpre4 + j);
        for (int w = 1; w < M; ++w) {
          const float4 v = __ldcg(Xpre4 + static_cast<long long>(w) * DV + j);
          s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        s.x *= inv_M; s.y *= inv_M; s.z *= inv_M; s.w *= inv_M;
        x4[j] = s;
        if (p == 0 && r == prm.rounds - 1) X4[static_cast<long long>(m) * DV + j] = s;
      }
      if (tid < M) {
        const double* src = prm.S + static_cast<long long>(tid) * P * 4;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0;
        for (int q = 0; q < Pa; ++q) {
          a0 += __ldcg(src + q * 4 + 0);
          a1 += __ldcg(src + q * 4 + 1);
          a2 += __ldcg(src + q * 4 + 2);
        }
        const abs_stats rec = record_from_sums(a0, __ldcg(src + 3), a1, a2, b, false);
        const long long T = test_size_from_record(rec, prm.cfg);
        T_s[tid] = T;
        if (blockIdx.x == 0) {
          prm.stats[static_cast<long long>(r) * M + tid] = rec;
          if (prm.T_out != nullptr) prm.T_out[static_cast<long long>(r) * M + tid] = T;
        }
      }
      __syncthreads();
      if (tid == 0) {
        long long best = b;
        for (int w = 0; w < M; ++w) best = T_s[w] > best ? T_s[w] : best;
        best = best < prm.cfg.b_max ? best : prm.cfg.b_max;
        b_s = best;
        if (blockIdx.x == 0 && prm.b_hist != nullptr) prm.b_hist[r + 1] = best;
      }
      __syncthreads();
      b = b_s;
    }
  }
  if (blockIdx.x == 0 && tid == 0) prm.b_dev[0] = b;
}

using KernelFn = void (*)(const FusedParams);
KernelFn pick_kernel(int DV) {
  if (DV <= 32) return logreg_rounds_kernel<1>;
  if (DV <= 64) return logreg_rounds_kernel<2>;
  if (DV <= 128) return logreg_rounds_kernel<4>;
  return logreg_rounds_kernel<8>;
}

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int abs_logreg_rounds_fused(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                       const int* idx, long long idx_stride, int rounds, float* X, int M, int H,
                                       float lr, const abs_test_cfg* cfg, abs_stats* stats, long long* T_out,
                                       long long* b_hist, long long* b_dev, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (A == nullptr || y == nullptr || idx == nullptr || X == nullptr || cfg == nullptr || stats == nullptr ||
      b_dev == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (n < 1 || d < 1 || M < 1 || H < 1 || rounds < 1)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need n, d, M, H, rounds >= 1");
  if (cfg->kind != ABS_TEST_NORM && cfg->kind != ABS_TEST_AUG_INNER_PRODUCT)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "unknown test kind %d", cfg->kind);
  if (cfg->b_max < 2 || !(cfg->row_weight > 0.0) || !(cfg->divisor > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need b_max >= 2, row_weight > 0, divisor > 0");
  if (cfg->kind == ABS_TEST_NORM ? !(cfg->eta > 0.0) : !(cfg->theta > 0.0 && cfg->nu > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "test constants must be positive");
  if (idx_stride < cfg->b_max)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "idx_stride (%lld) must cover b_max (%lld): the batch may grow to it",
                     idx_stride, cfg->b_max);
  if (d > kMaxDimFused || (d & 3) != 0 || M > kMaxWorkersFused)
    return set_error(ctx, ABS_ERR_UNSUPPORTED, "the fused rounds need d <= %d, d %% 4 == 0 and M <= %d (d=%lld, M=%d)",
                     kMaxDimFused, kMaxWorkersFused, d, M);
  if ((reinterpret_cast<uintptr_t>(A) & 15u) != 0 || (reinterpret_cast<uintptr_t>(X) & 15u) != 0)
    return set_error(ctx, ABS_ERR_UNSUPPORTED, "the fused rounds need 16-byte aligned A and X");

  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  struct Restore {
    int prev, dev;
    ~Restore() { if (prev != dev) cudaSetDevice(prev); }
  } restore{prev, ctx->device};

  const int DV = static_cast<int>(d / 4);
  KernelFn kernel = pick_kernel(DV);
  const size_t smem = static_cast<size_t>(2 + kFW) * d * sizeof(float);
  int per_sm = 0;
  ABS_CUDA_TRY(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kFThreads, smem));
  const long long resident = static_cast<long long>(per_sm) * ctx->sm_count;
  long long P = resident / M;
  if (P > kMaxCtasPerWorker) P = kMaxCtasPerWorker;
  if (P < 1) return set_error(ctx, ABS_ERR_UNSUPPORTED, "%d workers do not fit a co-resident grid (%lld CTAs)", M, resident);

  // scratch in the context's workspace: partial gradients, statistics partials, pre-average parameters
  const size_t partial_bytes = 2ull * M * P * d * sizeof(float);
  const size_t S_bytes = static_cast<size_t>(M) * P * 4 * sizeof(double);
  const size_t xpre_bytes = static_cast<size_t>(M) * d * sizeof(float);
  if (partial_bytes + S_bytes + xpre_bytes > ctx->workspace_bytes)
    return set_error(ctx, ABS_ERR_WORKSPACE, "workspace of %zu bytes is too small (%zu needed)", ctx->workspace_bytes,
                     partial_bytes + S_bytes + xpre_bytes);
  unsigned char* ws = static_cast<unsigned char*>(ctx->workspace);

  FusedParams prm;
  prm.A = A; prm.y = y; prm.n = n; prm.d = static_cast<int>(d);
  prm.idx = idx; prm.idx_stride = idx_stride;
  prm.rounds = rounds; prm.M = M; prm.H = H; prm.P = static_cast<int>(P);
  prm.lr = lr; prm.cfg = *cfg;
  prm.X = X; prm.stats = stats; prm.T_out = T_out; prm.b_hist = b_hist; prm.b_dev = b_dev;
  prm.partial = reinterpret_cast<float*>(ws);
  prm.S = reinterpret_cast<double*>(ws + partial_bytes);
  prm.Xpre = reinterpret_cast<float*>(ws + partial_bytes + S_bytes);
  void* args[] = {&prm};
  ABS_CUDA_TRY(ctx, cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(kernel), dim3(static_cast<unsigned>(M * P)),
                                                dim3(kFThreads), args, smem, static_cast<cudaStream_t>(stream)));
  return ABS_OK;
}
