// Fused local-optimiser steps for M parameter replicas held on one GPU, and the
// model averaging of Eq. local_sgd_alt.
//
// One thread owns a 16-byte column vector of ALL replicas: it streams x (and the
// optimiser state and the gradient) of replica m, updates them, and -- when the step
// is the last of a round -- keeps a running sum of the updated parameters so that the
// mean can be written to every replica without reading anything twice.  The averaging
// therefore costs no memory traffic beyond the step itself.  Replicas are processed
// four at a time with all loads issued before the arithmetic, which keeps
// 16 x 16 bytes in flight per thread.  Everything is fp32, as stored.
#include "abs_internal.cuh"

namespace absk {
namespace {

constexpr int kThreads = 256;
constexpr int kChunk = 4;      // replicas whose loads are issued together

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, const float4& v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(float* p, float v) { __stcs(p, v); }

__device__ __forceinline__ float4 add4(const float4& a, const float4& b) {
  return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
}
__device__ __forceinline__ float add4(float a, float b) { return a + b; }
__device__ __forceinline__ float4 scale4(const float4& a, float s) { return make_float4(a.x * s, a.y * s, a.z * s, a.w * s); }
__device__ __forceinline__ float scale4(float a, float s) { return a * s; }
template <typename V> __device__ __forceinline__ V zero4();
template <> __device__ __forceinline__ float4 zero4<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ float zero4<float>() { return 0.f; }

// ---- update rules ---------------------------------------------------------------------------
// Each rule names how many state tensors it carries besides X and whether it reads a
// gradient, and updates one scalar.  st[0], st[1] are the state values (in/out).
struct SgdRule {            // x <- x - lr g                          (Eq. local_sgd_alt)
  static constexpr int kStates = 0;
  static constexpr bool kGrad = true;
  float lr;
  __device__ __forceinline__ float apply(float x, float g, float*) const { return fmaf(-lr, g, x); }
};
struct AdamWRule {          // decoupled weight decay, bias-corrected moments
  static constexpr int kStates = 2;
  static constexpr bool kGrad = true;
  float beta1, one_m_beta1, beta2, one_m_beta2;
  float decay;              // 1 - lr * wd
  float step_size;          // lr / (1 - beta1^t)
  float inv_sqrt_bc2;       // 1 / sqrt(1 - beta2^t)
  float eps;
  __device__ __forceinline__ float apply(float x, float g, float* st) const {
    const float m = fmaf(beta1, st[0], one_m_beta1 * g);
    const float v = fmaf(beta2, st[1], one_m_beta2 * g * g);
    st[0] = m;
    st[1] = v;
    const float denom = fmaf(sqrtf(v), inv_sqrt_bc2, eps);
    return fmaf(-step_size, m / denom, x * decay);
  }
};
struct ShbRule {            // g <- g + wd x ; u <- mu u + g ; x <- x - lr u       (Section 6.1)
  static constexpr int kStates = 1;
  static constexpr bool kGrad = true;
  float lr, momentum, weight_decay;
  __device__ __forceinline__ float apply(float x, float g, float* st) const {
    const float u = fmaf(momentum, st[0], fmaf(weight_decay, x, g));
    st[0] = u;
    return fmaf(-lr, u, x);
  }
};
struct CopyRule {           // no update: plain model averaging
  static constexpr int kStates = 0;
  static constexpr bool kGrad = false;
  __device__ __forceinline__ float apply(float x, float, float*) const { return x; }
};

template <typename Rule>
__device__ __forceinline__ float4 apply4(const Rule& r, const float4& x, const float4& g, float4* st) {
  float s0[2], s1[2], s2[2], s3[2];
#pragma unroll
  for (int k = 0; k < Rule::kStates; ++k) {
    s0[k] = st[k].x; s1[k] = st[k].y; s2[k] = st[k].z; s3[k] = st[k].w;
  }
  float4 o;
  o.x = r.apply(x.x, g.x, s0);
  o.y = r.apply(x.y, g.y, s1);
  o.z = r.apply(x.z, g.z, s2);
  o.w = r.apply(x.w, g.w, s3);
#pragma unroll
  for (int k = 0; k < Rule::kStates; ++k) st[k] = make_float4(s0[k], s1[k], s2[k], s3[k]);
  return o;
}
template <typename Rule>
__device__ __forceinline__ float apply4(const Rule& r, float x, float g, float* st) { return r.apply(x, g, st); }

struct StepArgs {
  float* X;
  float* S0;
  float* S1;
  const float* Gb;
  int M;
  long long n;         // number of V-sized columns to process
  long long offset;    // first scalar column (tail launches start past the vector part)
  long long stride;    // replica stride in scalars
  int average;
  float inv_M;
};

// V = float4 (aligned fast path) or float (alignment-free path and the tail columns)
template <typename Rule, typename V>
__global__ void __launch_bounds__(kThreads)
local_step_kernel(const Rule rule, const StepArgs a) {
  const long long step = static_cast<long long>(gridDim.x) * kThreads;
  pdl_wait();      // launched as a programmatic dependent: the gradient of the kernels before is complete now
  for (long long j = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x; j < a.n; j += step) {
    V acc = zero4<V>();
    for (int m0 = 0; m0 < a.M; m0 += kChunk) {
      V x[kChunk], g[kChunk], st[kChunk][2];
#pragma unroll
      for (int c = 0; c < kChunk; ++c) {
        if (m0 + c < a.M) {
          const long long off = static_cast<long long>(m0 + c) * a.stride + a.offset;
          x[c] = ld_stream(reinterpret_cast<const V*>(a.X + off) + j);
          if (Rule::kGrad) g[c] = ld_stream(reinterpret_cast<const V*>(a.Gb + off) + j); else g[c] = zero4<V>();
          if (Rule::kStates > 0) st[c][0] = ld_stream(reinterpret_cast<const V*>(a.S0 + off) + j);
          if (Rule::kStates > 1) st[c][1] = ld_stream(reinterpret_cast<const V*>(a.S1 + off) + j);
        }
      }
#pragma unroll
      for (int c = 0; c < kChunk; ++c) {
        if (m0 + c < a.M) {
          const long long off = static_cast<long long>(m0 + c) * a.stride + a.offset;
          const V xn = apply4(rule, x[c], g[c], st[c]);
          if (Rule::kStates > 0) st_stream(reinterpret_cast<V*>(a.S0 + off) + j, st[c][0]);
          if (Rule::kStates > 1) st_stream(reinterpret_cast<V*>(a.S1 + off) + j, st[c][1]);
          if (a.average) acc = add4(acc, xn);
          else st_stream(reinterpret_cast<V*>(a.X + off) + j, xn);
        }
      }
    }
    if (a.average) {
      const V mean = scale4(acc, a.inv_M);
      for (int m = 0; m < a.M; ++m)
        st_stream(reinterpret_cast<V*>(a.X + static_cast<long long>(m) * a.stride + a.offset) + j, mean);
    }
  }
}

template <typename Rule>
int launch_step(abs_ctx* ctx, const Rule& rule, float* X, float* S0, float* S1, const float* Gb, int M, long long d,
                long long stride, int average, cudaStream_t stream) {
  if (X == nullptr || (Rule::kGrad && Gb == nullptr) || (Rule::kStates > 0 && S0 == nullptr) ||
      (Rule::kStates > 1 && S1 == nullptr))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null tensor pointer");
  if (M < 1 || d < 1 || (M > 1 && stride < d))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need M >= 1, d >= 1, replica_stride >= d (M=%d d=%lld stride=%lld)", M,
                     d, stride);
  StepArgs a;
  a.X = X; a.S0 = S0; a.S1 = S1; a.Gb = Gb; a.M = M; a.stride = stride; a.average = average ? 1 : 0;
  a.inv_M = 1.0f / static_cast<float>(M);
  uintptr_t bits = reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(Gb) |
                   reinterpret_cast<uintptr_t>(S0) | reinterpret_cast<uintptr_t>(S1);
  const bool vec = (bits & 15u) == 0 && (M == 1 || (stride & 3) == 0);
  const long long nvec = vec ? d / 4 : 0;
  // One CTA per 256 column vectors, no grid-stride loop unless the grid limit is hit: a finished
  // CTA is replaced by one that starts with its loads at once (M = 8, d = 124 M AdamW: 6.1 TB/s with
  // 8 CTAs per SM walking the columns, 6.45 with 24, 6.8 with one CTA per 256 vectors).
  const long long max_blocks = 0x7fffffffll;
  const long long small_blocks = static_cast<long long>(ctx->sm_count) * 8;
  if (nvec > 0) {
    a.n = nvec; a.offset = 0;
    long long blocks = (nvec + kThreads - 1) / kThreads;
    if (blocks > max_blocks) blocks = max_blocks;
    // small steps are bound by launch latency: let the launch overlap the kernel before (the kernel
    // waits for it before it reads); large steps gain nothing from that and are launched the plain way
    if (blocks < small_blocks)
      ABS_CUDA_TRY(ctx, launch_dependent(local_step_kernel<Rule, float4>, dim3(static_cast<unsigned>(blocks)),
                                         dim3(kThreads), 0, stream, rule, a));
    else
      local_step_kernel<Rule, float4><<<static_cast<unsigned>(blocks), kThreads, 0, stream>>>(rule, a);
    ABS_CUDA_TRY(ctx, cudaGetLastError());
  }
  const long long tail = d - nvec * 4;
  if (tail > 0) {
    a.n = tail; a.offset = nvec * 4;
    long long blocks = (tail + kThreads - 1) / kThreads;
    if (blocks > max_blocks) blocks = max_blocks;
    ABS_CUDA_TRY(ctx, launch_dependent(local_step_kernel<Rule, float>, dim3(static_cast<unsigned>(blocks)),
                                       dim3(kThreads), 0, stream, rule, a));
  }
  return ABS_OK;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int local_sgd_step(abs_ctx* ctx, float* X, const float* Gb, int M, long long d, long long replica_stride,
                              float lr, int average_after, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  SgdRule r;
  r.lr = lr;
  return launch_step(ctx, r, X, nullptr, nullptr, Gb, M, d, replica_stride, average_after,
                     static_cast<cudaStream_t>(stream));
}

extern "C" int local_adamw_step(abs_ctx* ctx, float* X, float* Mom1, float* Mom2, const float* Gb, int M, long long d,
                                long long replica_stride, const abs_adamw_cfg* cfg, int average_after, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (cfg == nullptr) return set_error(ctx, ABS_ERR_INVALID_ARG, "cfg is null");
  if (cfg->step < 1 || !(cfg->beta1 >= 0.f && cfg->beta1 < 1.f) || !(cfg->beta2 >= 0.f && cfg->beta2 < 1.f))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need step >= 1 and betas in [0, 1)");
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  const double b1 = cfg->beta1, b2 = cfg->beta2, t = static_cast<double>(cfg->step);
  const double bc1 = 1.0 - pow(b1, t), bc2 = 1.0 - pow(b2, t);
  AdamWRule r;
  r.beta1 = cfg->beta1;
  r.one_m_beta1 = static_cast<float>(1.0 - b1);
  r.beta2 = cfg->beta2;
  r.one_m_beta2 = static_cast<float>(1.0 - b2);
  r.decay = static_cast<float>(1.0 - static_cast<double>(cfg->lr) * cfg->weight_decay);
  r.step_size = static_cast<float>(static_cast<double>(cfg->lr) / bc1);
  r.inv_sqrt_bc2 = static_cast<float>(1.0 / sqrt(bc2));
  r.eps = cfg->eps;
  return launch_step(ctx, r, X, Mom1, Mom2, Gb, M, d, replica_stride, average_after,
                     static_cast<cudaStream_t>(stream));
}

extern "C" int local_shb_step(abs_ctx* ctx, float* X, float* Buf, const float* Gb, int M, long long d,
                              long long replica_stride, float lr, float momentum, float weight_decay,
                              int average_after, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  ShbRule r;
  r.lr = lr;
  r.momentum = momentum;
  r.weight_decay = weight_decay;
  return launch_step(ctx, r, X, Buf, nullptr, Gb, M, d, replica_stride, average_after,
                     static_cast<cudaStream_t>(stream));
}

extern "C" int replica_average(abs_ctx* ctx, float* X, int M, long long d, long long replica_stride, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return set_error(ctx, ABS_ERR_CUDA, "cannot select device %d", ctx->device);
  CopyRule r;
  return launch_step(ctx, r, X, nullptr, nullptr, nullptr, M, d, replica_stride, 1,
                     static_cast<cudaStream_t>(stream));
}
