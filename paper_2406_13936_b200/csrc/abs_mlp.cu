// Producer for the MLP end-to-end problem: forward and backward pass of a three-layer ReLU
// classifier with softmax cross-entropy for M workers at once, the batch gradients, and -- for
// the batch-size test -- the per-sample gradients written out as rows (Algorithm 1, per-sample
// gradient step; they are outer products delta_l,i (x) h_{l-1},i).
//
// Parameter layout of one replica (flat, fp32): W1 [n1][n0], b1 [n1], W2 [n2][n1], b2 [n2],
// W3 [n3][n2], b3 [n3], each W row-major [out][in].
// Scratch layout per worker (floats): Xin [b][n0], H1 [b][n1], H2 [b][n2], D3 [b][n3], D2 [b][n2],
// D1 [b][n1], then work space of the fused statistics.
//
// Fused statistics (abs_mlp_fused_stats): the per-sample gradient of a layer is the outer product
// delta_i (x) h_i (plus delta_i for the bias), so the two per-sample quantities the batch-size
// test needs follow from activations and deltas without writing the b x d gradient matrix:
//   ||g_i||^2    = sum_l ||delta_l,i||^2 (||h_{l-1},i||^2 + 1)
//   <g_i, gbar>  = sum_l delta_l,i^T (dW_l h_{l-1},i + db_l)          (dW_l, db_l: the batch gradient)
// and with N = ||gbar||^2:  sum_i ||g_i - gbar||^2 = sum_i ||g_i||^2 - b N  (Eq. def_var expanded),
// Var_i <g_i, gbar> directly.  The expansions cancel only when the variance is far below b N,
// i.e. when the test is satisfied by a wide margin anyway.
#include "abs_gemm.cuh"

namespace absk {
namespace {

constexpr int kNormParts = 64;    // blocks per worker that sum ||gbar||^2

struct MlpShape {
  int n0, n1, n2, n3;
  long long oW1, ob1, oW2, ob2, oW3, ob3, d;      // offsets into the flat parameter vector
  long long sX, sH1, sH2, sD3, sD2, sD1, sU, sCQ, per_worker;   // offsets into a worker's scratch
};

MlpShape make_shape(const int* dims, long long b) {
  MlpShape s;
  s.n0 = dims[0]; s.n1 = dims[1]; s.n2 = dims[2]; s.n3 = dims[3];
  s.oW1 = 0;
  s.ob1 = s.oW1 + static_cast<long long>(s.n1) * s.n0;
  s.oW2 = s.ob1 + s.n1;
  s.ob2 = s.oW2 + static_cast<long long>(s.n2) * s.n1;
  s.oW3 = s.ob2 + s.n2;
  s.ob3 = s.oW3 + static_cast<long long>(s.n3) * s.n2;
  s.d = s.ob3 + s.n3;
  s.sX = 0;
  s.sH1 = s.sX + b * s.n0;
  s.sH2 = s.sH1 + b * s.n1;
  s.sD3 = s.sH2 + b * s.n2;
  s.sD2 = s.sD3 + b * s.n3;
  s.sD1 = s.sD2 + b * s.n2;
  // used by the fused statistics only: U [b][max width] products, then c_i, q_i [2][b] and 64 partial
  // sums of ||gbar||^2 as doubles
  const long long widest = s.n1 > s.n2 ? (s.n1 > s.n3 ? s.n1 : s.n3) : (s.n2 > s.n3 ? s.n2 : s.n3);
  s.sU = (s.sD1 + b * s.n1 + 3) / 4 * 4;
  s.sCQ = (s.sU + b * widest + 3) / 4 * 4;
  s.per_worker = (s.sCQ + 2 * (2 * b + kNormParts) + 3) / 4 * 4;
  return s;
}

// ---- batched fp32 GEMM with strided operands and a small epilogue (GemmArgs: abs_gemm.cuh) ----
constexpr int kTile = 64, kTileK = 16;

__global__ void __launch_bounds__(256)
sgemm_kernel(const GemmArgs g) {
  __shared__ float As[kTileK][kTile + 4];
  __shared__ float Bs[kTileK][kTile + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int z = blockIdx.z;
  const long long r0 = static_cast<long long>(blockIdx.y) * kTile, c0 = static_cast<long long>(blockIdx.x) * kTile;
  const float* A = g.A + z * g.a_bs;
  const float* B = g.B + z * g.b_bs;
  // fp32 products are summed in fp32 over one 16-deep slice and the slices in fp64: the rounding
  // error of a long dot product then stays near one fp32 ulp, which the 1e-6 parity bound on the
  // parameters needs
  double dacc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) dacc[i][j] = 0.0;

  for (int k0 = 0; k0 < g.K; k0 += kTileK) {
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int e = tid + t * 256;
      int r, k;
      if (g.a_cs == 1) { r = e / kTileK; k = e % kTileK; } else { r = e % kTile; k = e / kTile; }
      const long long rr = r0 + r;
      const int kk = k0 + k;
      As[k][r] = (rr < g.rows && kk < g.K) ? A[rr * g.a_rs + kk * g.a_cs] : 0.f;
      int c;
      if (g.b_cs == 1) { k = e / kTile; c = e % kTile; } else { c = e / kTileK; k = e % kTileK; }
      const long long cc = c0 + c;
      const int kb = k0 + k;
      Bs[k][c] = (cc < g.cols && kb < g.K) ? B[kb * g.b_rs + cc * g.b_cs] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTileK; ++k) {
      float a[4], bb[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bb[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) dacc[i][j] += static_cast<double>(acc[i][j]);
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long r = r0 + ty * 4 + i;
    if (r >= g.rows) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const long long c = c0 + tx * 4 + j;
      if (c >= g.cols) continue;
      float v = static_cast<float>(g.mode == 0 ? dacc[i][j] * static_cast<double>(g.alpha) : dacc[i][j]);
      if (g.mode == 0) {}
      else if (g.mode == 1) v = fmaxf(static_cast<float>(dacc[i][j] + g.bias[z * g.bias_bs + c]), 0.f);
      else if (g.mode == 2) v = static_cast<float>(dacc[i][j] + g.bias[z * g.bias_bs + c]);
      else v = g.mask[z * g.mask_bs + r * g.mask_rs + c] > 0.f ? v : 0.f;
      g.C[z * g.c_bs + r * g.c_rs + c] = v;
    }
  }
}

// ---- the same GEMM for large operands: 128 x 128 tiles, 8 x 8 outputs per thread -------------
// Operand tiles are fetched 16 bytes at a time along whichever index is contiguous in memory
// (rows or k for A, k or columns for B), one 16-deep slice ahead of the arithmetic (registers ->
// the other shared-memory buffer), so a slice costs one barrier.  Slices are summed in fp32 and
// folded into fp64 as in sgemm_kernel; the results are bit-identical to it (same products, same
// order of additions per output).
constexpr int kBig = 128;

// Four consecutive elements along the contiguous index starting at p; elements at or past `left`
// (counted from p) read as zero.  `vec` says that p is 16-byte aligned.
__device__ __forceinline__ float4 load4_guarded(const float* p, long long left, bool vec) {
  if (left >= 4 && vec) return __ldg(reinterpret_cast<const float4*>(p));
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (left > 0) v.x = __ldg(p);
  if (left > 1) v.y = __ldg(p + 1);
  if (left > 2) v.z = __ldg(p + 2);
  if (left > 3) v.w = __ldg(p + 3);
  return v;
}

// A_KCONT: k is the contiguous index of A (a_cs == 1), else the row index is (a_rs == 1).
// B_KCONT: k is the contiguous index of B (b_rs == 1), else the column index is (b_cs == 1).
template <bool A_KCONT, bool B_KCONT>
__global__ void __launch_bounds__(256, 1)
sgemm_big_kernel(const GemmArgs g) {
  __shared__ __align__(16) float As[2][kTileK][kBig + 4];
  __shared__ __align__(16) float Bs[2][kTileK][kBig + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int z = blockIdx.z;
  const long long r0 = static_cast<long long>(blockIdx.y) * kBig, c0 = static_cast<long long>(blockIdx.x) * kBig;
  const float* A = g.A + z * g.a_bs;
  const float* B = g.B + z * g.b_bs;
  // 16-byte loads need an aligned base and a stride of the other index that keeps the alignment
  const bool a_vec = (reinterpret_cast<uintptr_t>(A) & 15u) == 0 && ((A_KCONT ? g.a_rs : g.a_cs) & 3) == 0;
  const bool b_vec = (reinterpret_cast<uintptr_t>(B) & 15u) == 0 && ((B_KCONT ? g.b_cs : g.b_rs) & 3) == 0;

  // this thread's two 16-byte pieces of each operand tile (piece e = tid, tid + 256)
  //   k contiguous:  e -> (index e / 4 of the tile, k quad e % 4)
  //   else:          e -> (k = e / 32, quad e % 32 of the 128 rows / columns)
  float4 ra[2], rb[2];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int e = tid + 256 * t;
      if (A_KCONT) {
        const long long r = r0 + (e >> 2);
        const int k = k0 + 4 * (e & 3);
        ra[t] = load4_guarded(A + r * g.a_rs + k, r < g.rows ? g.K - k : 0, a_vec);
      } else {
        const int k = k0 + (e >> 5);
        const long long r = r0 + 4 * (e & 31);
        ra[t] = load4_guarded(A + k * g.a_cs + r, k < g.K ? g.rows - r : 0, a_vec);
      }
      if (B_KCONT) {
        const long long c = c0 + (e >> 2);
        const int k = k0 + 4 * (e & 3);
        rb[t] = load4_guarded(B + c * g.b_cs + k, c < g.cols ? g.K - k : 0, b_vec);
      } else {
        const int k = k0 + (e >> 5);
        const long long c = c0 + 4 * (e & 31);
        rb[t] = load4_guarded(B + k * g.b_rs + c, k < g.K ? g.cols - c : 0, b_vec);
      }
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int e = tid + 256 * t;
      if (A_KCONT) {
        const int r = e >> 2, k = 4 * (e & 3);
        As[buf][k][r] = ra[t].x; As[buf][k + 1][r] = ra[t].y; As[buf][k + 2][r] = ra[t].z; As[buf][k + 3][r] = ra[t].w;
      } else {
        *reinterpret_cast<float4*>(&As[buf][e >> 5][4 * (e & 31)]) = ra[t];
      }
      if (B_KCONT) {
        const int c = e >> 2, k = 4 * (e & 3);
        Bs[buf][k][c] = rb[t].x; Bs[buf][k + 1][c] = rb[t].y; Bs[buf][k + 2][c] = rb[t].z; Bs[buf][k + 3][c] = rb[t].w;
      } else {
        *reinterpret_cast<float4*>(&Bs[buf][e >> 5][4 * (e & 31)]) = rb[t];
      }
    }
  };

  double dacc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) dacc[i][j] = 0.0;

  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < g.K; k0 += kTileK) {
    const bool more = k0 + kTileK < g.K;
    if (more) fetch(k0 + kTileK);
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
#pragma unroll
    for (int k = 0; k < kTileK; ++k) {
      // rows ty*4 .. +3 and 64 + ty*4 .. +3; columns tx*4 .. +3 and 64 + tx*4 .. +3
      const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) dacc[i][j] += static_cast<double>(acc[i][j]);
    if (more) stash(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const long long r = r0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + i - 4);
    if (r >= g.rows) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long c = c0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + j - 4);
      if (c >= g.cols) continue;
      float v = static_cast<float>(g.mode == 0 ? dacc[i][j] * static_cast<double>(g.alpha) : dacc[i][j]);
      if (g.mode == 0) {}
      else if (g.mode == 1) v = fmaxf(static_cast<float>(dacc[i][j] + g.bias[z * g.bias_bs + c]), 0.f);
      else if (g.mode == 2) v = static_cast<float>(dacc[i][j] + g.bias[z * g.bias_bs + c]);
      else v = g.mask[z * g.mask_bs + r * g.mask_rs + c] > 0.f ? v : 0.f;
      g.C[z * g.c_bs + r * g.c_rs + c] = v;
    }
  }
}

void launch_gemm(abs_ctx* ctx, const GemmArgs& g, int batch, cudaStream_t st) {
  // large products go to the tensor cores (3 x TF32 split, abs_gemm_tc.cu); a wait that runs out there
  // raises the context's time-out word, which the statistics that follow report
  if (!ctx->tuning.mlp_no_tensor_cores &&
      launch_gemm_tc(g, batch, ctx->flags,
                     ctx->tuning.stats_timeout_cycles > 0 ? ctx->tuning.stats_timeout_cycles : kDefaultTimeoutCycles,
                     ctx->tuning.stats_fault_drop_loads != 0, st))
    return;
  // the large-tile kernel where a 128 x 128 tile is mostly used and both operands have a contiguous index
  const bool a_ok = g.a_cs == 1 || g.a_rs == 1, b_ok = g.b_rs == 1 || g.b_cs == 1;
  if (a_ok && b_ok && g.rows >= 96 && g.cols >= 96) {
    const dim3 big((g.cols + kBig - 1) / kBig, (g.rows + kBig - 1) / kBig, batch);
    const bool ak = g.a_cs == 1, bk = g.b_rs == 1;
    if (ak && bk) sgemm_big_kernel<true, true><<<big, 256, 0, st>>>(g);
    else if (ak) sgemm_big_kernel<true, false><<<big, 256, 0, st>>>(g);
    else if (bk) sgemm_big_kernel<false, true><<<big, 256, 0, st>>>(g);
    else sgemm_big_kernel<false, false><<<big, 256, 0, st>>>(g);
    return;
  }
  const dim3 grid((g.cols + kTile - 1) / kTile, (g.rows + kTile - 1) / kTile, batch);
  sgemm_kernel<<<grid, 256, 0, st>>>(g);
}

// Sample indices outside [0, n) are clamped: a bad index never becomes an out-of-range read.
__device__ __forceinline__ long long clamp_sample(int raw, long long n) {
  return raw < 0 ? 0 : (raw >= n ? n - 1 : static_cast<long long>(raw));
}

// Xin[m][i][:] = inputs[idx[m][i]][:]
__global__ void gather_rows_kernel(const float* __restrict__ inputs, long long n, const int* __restrict__ idx,
                                   long long idx_stride, long long b, int n0, float* __restrict__ scratch,
                                   long long per_worker) {
  const int m = blockIdx.y;
  const long long i = blockIdx.x;
  const float* src = inputs + clamp_sample(idx[m * idx_stride + i], n) * n0;
  float* dst = scratch + m * per_worker + i * n0;
  for (int j = threadIdx.x; j < n0; j += blockDim.x) dst[j] = src[j];
}

// In place on the logits: D3[i][:] = softmax(logits_i) - onehot(label_i); one thread per sample.
__global__ void softmax_delta_kernel(float* __restrict__ scratch, long long per_worker, long long off, long long b,
                                     int n3, const int* __restrict__ labels, long long n,
                                     const int* __restrict__ idx, long long idx_stride) {
  const int m = blockIdx.y;
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= b) return;
  float* z = scratch + m * per_worker + off + i * n3;
  float mx = z[0];
  for (int c = 1; c < n3; ++c) mx = fmaxf(mx, z[c]);
  float sum = 0.f;
  for (int c = 0; c < n3; ++c) {
    const float e = expf(z[c] - mx);
    z[c] = e;
    sum += e;
  }
  // the label's own entry is softmax - 1 = -(sum of the other classes) / sum: nothing is subtracted from
  // a probability near 1, so a well-fitted sample keeps the relative accuracy of its (tiny) delta
  const int label = labels[clamp_sample(idx[m * idx_stride + i], n)];
  float others = 0.f;
  for (int c = 0; c < n3; ++c) others += c == label ? 0.f : z[c];
  for (int c = 0; c < n3; ++c) z[c] = c == label ? -others / sum : z[c] / sum;
}

// db[o] = (1/b) sum_i D[i][o].  A CTA covers 32 output units of one worker: warp w sums the rows
// w, w + 32, ... of its 32 columns (128 contiguous bytes per row) in fp64, then the 32 partial sums
// of a column are added in warp order, so the result does not depend on the launch.
__global__ void __launch_bounds__(1024)
bias_grad_kernel(const float* __restrict__ scratch, long long per_worker, long long off, long long b, int n,
                 float* __restrict__ Gb, long long d, long long ob) {
  __shared__ double part[32][33];
  const int m = blockIdx.y, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int o = blockIdx.x * 32 + lane;
  const float* D = scratch + m * per_worker + off;
  double acc = 0.0;
  if (o < n)
    for (long long i = w; i < b; i += 32) acc += static_cast<double>(D[i * n + o]);
  part[w][lane] = acc;
  __syncthreads();
  if (w == 0 && o < n) {
    double tot = 0.0;
    for (int k = 0; k < 32; ++k) tot += part[k][lane];
    Gb[m * d + ob + o] = static_cast<float>(tot / static_cast<double>(b));
  }
}

// Row i of G: the flat gradient of sample i of one worker.  The weight segment of a layer is the
// outer product delta_i (x) h_i: a thread writes 16 bytes (four consecutive inputs of one output
// unit), so the kernel runs at the speed of the stores.  Needs n_in % 4 == 0 and 16-byte aligned
// segment starts and rows; per_sample_rows_scalar_kernel covers everything else.
__global__ void __launch_bounds__(256)
per_sample_layer_kernel(const float* __restrict__ delta, const float* __restrict__ h, unsigned n_out, unsigned n_in,
                        float* __restrict__ G, long long row_stride, long long seg_off) {
  const long long i = blockIdx.y;
  const unsigned quads = n_out * (n_in / 4u);
  const float* di = delta + i * n_out;
  const float4* hi = reinterpret_cast<const float4*>(h + i * n_in);
  float4* out = reinterpret_cast<float4*>(G + i * row_stride + seg_off);
  const unsigned q_in = n_in / 4u;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const unsigned f = (blockIdx.x * 4u + u) * 256u + threadIdx.x;
    if (f < quads) {
      const unsigned o = f / q_in, k4 = f - o * q_in;
      const float dv = __ldg(di + o);
      const float4 hv = __ldg(hi + k4);
      __stcs(out + f, make_float4(dv * hv.x, dv * hv.y, dv * hv.z, dv * hv.w));
    }
  }
}

// bias segments: G[i][seg_off + o] = delta[i][o]
__global__ void per_sample_bias_kernel(const float* __restrict__ delta, unsigned n_out, float* __restrict__ G,
                                       long long row_stride, long long seg_off) {
  const long long i = blockIdx.y;
  const unsigned o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o < n_out) G[i * row_stride + seg_off + o] = delta[i * n_out + o];
}

// Alignment-free variant: one thread per parameter.
__global__ void __launch_bounds__(256)
per_sample_rows_scalar_kernel(const float* __restrict__ ws, const MlpShape s, float* __restrict__ G,
                              long long row_stride) {
  const long long i = blockIdx.y;
  const long long j = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (j >= s.d) return;
  float v;
  if (j < s.ob1) {
    const long long o = j / s.n0, k = j % s.n0;
    v = ws[s.sD1 + i * s.n1 + o] * ws[s.sX + i * s.n0 + k];
  } else if (j < s.oW2) {
    v = ws[s.sD1 + i * s.n1 + (j - s.ob1)];
  } else if (j < s.ob2) {
    const long long o = (j - s.oW2) / s.n1, k = (j - s.oW2) % s.n1;
    v = ws[s.sD2 + i * s.n2 + o] * ws[s.sH1 + i * s.n1 + k];
  } else if (j < s.oW3) {
    v = ws[s.sD2 + i * s.n2 + (j - s.ob2)];
  } else if (j < s.ob3) {
    const long long o = (j - s.oW3) / s.n2, k = (j - s.oW3) % s.n2;
    v = ws[s.sD3 + i * s.n3 + o] * ws[s.sH2 + i * s.n2 + k];
  } else {
    v = ws[s.sD3 + i * s.n3 + (j - s.ob3)];
  }
  G[i * row_stride + j] = v;
}

// ---- fused statistics ------------------------------------------------------------------------
// One warp per sample: q_i += ||delta_i||^2 (||h_i||^2 + 1).
__global__ void __launch_bounds__(256)
fused_rownorm_kernel(float* __restrict__ scratch, long long per_worker, long long sD, long long sH, long long sCQ,
                     long long b, int n_out, int n_in) {
  const int m = blockIdx.y;
  const long long i = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (i >= b) return;
  const float* ws = scratch + m * per_worker;
  const float* dl = ws + sD + i * n_out;
  const float* hl = ws + sH + i * n_in;
  float dn = 0.f, hn = 0.f;
  for (int o = lane; o < n_out; o += 32) dn = fmaf(dl[o], dl[o], dn);
  for (int k = lane; k < n_in; k += 32) hn = fmaf(hl[k], hl[k], hn);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    dn += __shfl_xor_sync(0xffffffffu, dn, off);
    hn += __shfl_xor_sync(0xffffffffu, hn, off);
  }
  if (lane == 0) {
    double* q = reinterpret_cast<double*>(scratch + m * per_worker + sCQ) + b;
    q[i] += static_cast<double>(dn) * (static_cast<double>(hn) + 1.0);
  }
}

// One warp per sample: c_i += sum_o delta_i[o] (U_i[o] + db[o]), U = h dW^T.
__global__ void __launch_bounds__(256)
fused_rowdot_kernel(float* __restrict__ scratch, long long per_worker, long long sD, long long sU, long long sCQ,
                    long long b, int n_out, const float* __restrict__ Gb, long long d, long long ob) {
  const int m = blockIdx.y;
  const long long i = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (i >= b) return;
  const float* ws = scratch + m * per_worker;
  const float* dl = ws + sD + i * n_out;
  const float* ul = ws + sU + i * n_out;
  const float* db = Gb + m * d + ob;
  float acc = 0.f;
  for (int o = lane; o < n_out; o += 32) acc = fmaf(dl[o], ul[o] + db[o], acc);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (lane == 0) reinterpret_cast<double*>(scratch + m * per_worker + sCQ)[i] += static_cast<double>(acc);
}

// ||gbar||^2 of every worker in kNormParts partial sums, and c_i = q_i = 0.
__global__ void __launch_bounds__(256)
fused_norm_kernel(const float* __restrict__ Gb, long long d, float* __restrict__ scratch, long long per_worker,
                  long long sCQ, long long b) {
  __shared__ double red[8];
  const int m = blockIdx.y, p = blockIdx.x, tid = threadIdx.x;
  double* cq = reinterpret_cast<double*>(scratch + m * per_worker + sCQ);
  for (long long i = static_cast<long long>(p) * 256 + tid; i < 2 * b; i += static_cast<long long>(kNormParts) * 256)
    cq[i] = 0.0;
  const float* g = Gb + m * d;
  double acc = 0.0;
  for (long long j0 = static_cast<long long>(p) * 1024; j0 < d; j0 += static_cast<long long>(kNormParts) * 1024) {
    float a = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long j = j0 + u * 256 + tid;
      if (j < d) a = fmaf(g[j], g[j], a);
    }
    acc += static_cast<double>(a);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if ((tid & 31) == 0) red[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += red[w];
    cq[2 * b + p] = t;
  }
}

// One block per worker: abs_stats from c_i, q_i and N.
__global__ void __launch_bounds__(1024)
fused_finalize_kernel(const float* __restrict__ scratch, long long per_worker, long long sCQ, long long b,
                      abs_stats* __restrict__ stats, unsigned* __restrict__ flags) {
  __shared__ double red[3][32];
  const int m = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned timeout_word = 0u;      // raised by a tensor-core product whose wait ran out
  if (tid == 0) timeout_word = *reinterpret_cast<volatile unsigned*>(flags);
  const double* cq = reinterpret_cast<const double*>(scratch + m * per_worker + sCQ);
  const double bd = static_cast<double>(b);
  auto block_sum = [&](double v, int slot) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    if (lane == 0) red[slot][warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < 32; ++w) t += red[slot][w];
    __syncthreads();
    return t;
  };
  double sc = 0.0, sq = 0.0;
  for (long long i = tid; i < b; i += 1024) {
    sc += cq[i];
    sq += cq[b + i];
  }
  const double csum = block_sum(sc, 0);
  const double qsum = block_sum(sq, 1);
  const double cbar = csum / bd;
  double sv = 0.0;
  for (long long i = tid; i < b; i += 1024) {
    const double e = cq[i] - cbar;
    sv += e * e;
  }
  const double ss = block_sum(sv, 2);
  if (tid == 0) {
    double N = 0.0;
    for (int p = 0; p < kNormParts; ++p) N += cq[2 * b + p];
    double S = qsum - bd * N;                 // sum_i ||g_i - gbar||^2
    if (S < 0.0) S = 0.0;
    abs_stats o;
    o.gbar_sq = N;
    o.var_norm = S / (bd - 1.0);
    o.var_ip = ss / (bd - 1.0);
    o.var_orth = o.var_norm;
    if (N > 0.0) {
      o.var_orth = o.var_norm - o.var_ip / N;
      if (o.var_orth < 0.0) o.var_orth = 0.0;
    }
    o.sum_sq = qsum;
    o.rows = b;
    o.status = 0u;
    if (!(isfinite(qsum) && isfinite(N) && isfinite(ss))) o.status |= ABS_STATUS_NONFINITE;
    if (N == 0.0) o.status |= ABS_STATUS_ZERO_MEAN;
    if (timeout_word != 0u) o.status |= ABS_STATUS_TIMEOUT;
    o.recomputed = 0u;
    // the last worker to get here clears the time-out word and the arrival counter for the next call
    __threadfence();
    if (atomicAdd(flags + 1, 1u) == gridDim.x - 1) {
      flags[0] = 0u;
      flags[1] = 0u;
    }
    stats[m] = o;
  }
}

int check_dims(abs_ctx* ctx, const int* dims) {
  if (dims == nullptr) return set_error(ctx, ABS_ERR_INVALID_ARG, "dims is null");
  for (int l = 0; l < 4; ++l)
    if (dims[l] < 1) return set_error(ctx, ABS_ERR_INVALID_ARG, "layer widths must be >= 1");
  return ABS_OK;
}

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int abs_mlp_param_count(const int* dims, long long* out) {
  if (dims == nullptr || out == nullptr) return ABS_ERR_INVALID_ARG;
  *out = make_shape(dims, 1).d;
  return ABS_OK;
}

extern "C" int abs_mlp_scratch_bytes(int M, long long b, const int* dims, size_t* out) {
  if (dims == nullptr || out == nullptr || M < 1 || b < 1) return ABS_ERR_INVALID_ARG;
  *out = static_cast<size_t>(M) * make_shape(dims, b).per_worker * sizeof(float);
  return ABS_OK;
}

extern "C" int abs_mlp_grads(abs_ctx* ctx, const float* inputs, const int* labels, long long n, const int* dims,
                             const int* idx, long long idx_stride, const float* X, int M, long long b, float* Gb,
                             void* scratch, size_t scratch_bytes, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  int rc = check_dims(ctx, dims);
  if (rc != ABS_OK) return rc;
  if (inputs == nullptr || labels == nullptr || idx == nullptr || X == nullptr || Gb == nullptr || scratch == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (n < 1 || M < 1 || M > 65535 || b < 1 || idx_stride < b)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need n, b >= 1, 1 <= M <= 65535 and idx_stride >= b");
  const MlpShape s = make_shape(dims, b);
  if (scratch_bytes < static_cast<size_t>(M) * s.per_worker * sizeof(float))
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_mlp_grads needs %zu scratch bytes, got %zu",
                     static_cast<size_t>(M) * s.per_worker * sizeof(float), scratch_bytes);
  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* ws = static_cast<float*>(scratch);
  const long long pw = s.per_worker, d = s.d;
  const float inv_b = 1.0f / static_cast<float>(b);

  gather_rows_kernel<<<dim3(static_cast<unsigned>(b), M), 128, 0, st>>>(inputs, n, idx, idx_stride, b, s.n0, ws, pw);

  GemmArgs g;
  // forward: H1 = relu(Xin W1^T + b1), H2 = relu(H1 W2^T + b2), logits = H2 W3^T + b3
  g = GemmArgs{ws + s.sX, s.n0, 1, pw, X + s.oW1, 1, s.n0, d, ws + s.sH1, s.n1, pw, X + s.ob1, d, nullptr, 0, 0,
               static_cast<int>(b), s.n1, s.n0, 1.f, 1};
  launch_gemm(ctx, g, M, st);
  g = GemmArgs{ws + s.sH1, s.n1, 1, pw, X + s.oW2, 1, s.n1, d, ws + s.sH2, s.n2, pw, X + s.ob2, d, nullptr, 0, 0,
               static_cast<int>(b), s.n2, s.n1, 1.f, 1};
  launch_gemm(ctx, g, M, st);
  g = GemmArgs{ws + s.sH2, s.n2, 1, pw, X + s.oW3, 1, s.n2, d, ws + s.sD3, s.n3, pw, X + s.ob3, d, nullptr, 0, 0,
               static_cast<int>(b), s.n3, s.n2, 1.f, 2};
  launch_gemm(ctx, g, M, st);
  softmax_delta_kernel<<<dim3(static_cast<unsigned>((b + 127) / 128), M), 128, 0, st>>>(ws, pw, s.sD3, b, s.n3, labels,
                                                                                       n, idx, idx_stride);
  // backward: D2 = (D3 W3) .* (H2 > 0), D1 = (D2 W2) .* (H1 > 0)
  g = GemmArgs{ws + s.sD3, s.n3, 1, pw, X + s.oW3, s.n2, 1, d, ws + s.sD2, s.n2, pw, nullptr, 0, ws + s.sH2, s.n2, pw,
               static_cast<int>(b), s.n2, s.n3, 1.f, 3};
  launch_gemm(ctx, g, M, st);
  g = GemmArgs{ws + s.sD2, s.n2, 1, pw, X + s.oW2, s.n1, 1, d, ws + s.sD1, s.n1, pw, nullptr, 0, ws + s.sH1, s.n1, pw,
               static_cast<int>(b), s.n1, s.n2, 1.f, 3};
  launch_gemm(ctx, g, M, st);
  // batch gradients: dW_l = (1/b) D_l^T H_{l-1}, db_l = (1/b) sum_i D_l[i]
  g = GemmArgs{ws + s.sD3, 1, s.n3, pw, ws + s.sH2, s.n2, 1, pw, Gb + s.oW3, s.n2, d, nullptr, 0, nullptr, 0, 0,
               s.n3, s.n2, static_cast<int>(b), inv_b, 0};
  launch_gemm(ctx, g, M, st);
  g = GemmArgs{ws + s.sD2, 1, s.n2, pw, ws + s.sH1, s.n1, 1, pw, Gb + s.oW2, s.n1, d, nullptr, 0, nullptr, 0, 0,
               s.n2, s.n1, static_cast<int>(b), inv_b, 0};
  launch_gemm(ctx, g, M, st);
  g = GemmArgs{ws + s.sD1, 1, s.n1, pw, ws + s.sX, s.n0, 1, pw, Gb + s.oW1, s.n0, d, nullptr, 0, nullptr, 0, 0,
               s.n1, s.n0, static_cast<int>(b), inv_b, 0};
  launch_gemm(ctx, g, M, st);
  bias_grad_kernel<<<dim3((s.n3 + 31) / 32, M), 1024, 0, st>>>(ws, pw, s.sD3, b, s.n3, Gb, d, s.ob3);
  bias_grad_kernel<<<dim3((s.n2 + 31) / 32, M), 1024, 0, st>>>(ws, pw, s.sD2, b, s.n2, Gb, d, s.ob2);
  bias_grad_kernel<<<dim3((s.n1 + 31) / 32, M), 1024, 0, st>>>(ws, pw, s.sD1, b, s.n1, Gb, d, s.ob1);
  const cudaError_t e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) return set_error(ctx, ABS_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return ABS_OK;
}

extern "C" int abs_mlp_per_sample(abs_ctx* ctx, const int* dims, long long b, int worker, const void* scratch, float* G,
                                  long long row_stride, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  int rc = check_dims(ctx, dims);
  if (rc != ABS_OK) return rc;
  const MlpShape s = make_shape(dims, b);
  if (scratch == nullptr || G == nullptr || b < 1 || b > 65535 || worker < 0 || row_stride < s.d)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need scratch, G, 1 <= b <= 65535, worker >= 0, row_stride >= d");
  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  const float* ws = static_cast<const float*>(scratch) + static_cast<long long>(worker) * s.per_worker;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool vec = (s.n0 % 4 == 0) && (s.n1 % 4 == 0) && (s.n2 % 4 == 0) && (row_stride % 4 == 0) &&
                   (s.oW2 % 4 == 0) && (s.oW3 % 4 == 0) && (s.per_worker % 4 == 0) && ((b * s.n0) % 4 == 0) &&
                   ((b * s.n1) % 4 == 0) && ((b * s.n2) % 4 == 0) && ((b * s.n3) % 4 == 0) &&
                   (reinterpret_cast<uintptr_t>(G) % 16 == 0) && (reinterpret_cast<uintptr_t>(ws) % 16 == 0);
  if (vec) {
    const unsigned rows = static_cast<unsigned>(b);
    auto layer = [&](long long sD, long long sH, int n_out, int n_in, long long oW, long long ob) {
      const unsigned quads = static_cast<unsigned>(n_out) * static_cast<unsigned>(n_in / 4);
      per_sample_layer_kernel<<<dim3((quads + 1023) / 1024, rows), 256, 0, st>>>(
          ws + sD, ws + sH, static_cast<unsigned>(n_out), static_cast<unsigned>(n_in), G, row_stride, oW);
      per_sample_bias_kernel<<<dim3((n_out + 127) / 128, rows), 128, 0, st>>>(ws + sD, static_cast<unsigned>(n_out), G,
                                                                             row_stride, ob);
    };
    layer(s.sD1, s.sX, s.n1, s.n0, s.oW1, s.ob1);
    layer(s.sD2, s.sH1, s.n2, s.n1, s.oW2, s.ob2);
    layer(s.sD3, s.sH2, s.n3, s.n2, s.oW3, s.ob3);
  } else {
    const dim3 grid(static_cast<unsigned>((s.d + 255) / 256), static_cast<unsigned>(b));
    per_sample_rows_scalar_kernel<<<grid, 256, 0, st>>>(ws, s, G, row_stride);
  }
  const cudaError_t e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) return set_error(ctx, ABS_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return ABS_OK;
}


// Statistics of all M workers straight from the activations and deltas that abs_mlp_grads left in
// `scratch` and from the batch gradients Gb it wrote: no per-sample gradient matrix is formed.
extern "C" int abs_mlp_fused_stats(abs_ctx* ctx, const int* dims, long long b, int M, void* scratch,
                                   size_t scratch_bytes, const float* Gb, abs_stats* stats, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  int rc = check_dims(ctx, dims);
  if (rc != ABS_OK) return rc;
  if (scratch == nullptr || Gb == nullptr || stats == nullptr || b < 2 || M < 1 || M > 65535)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need scratch, Gb, stats, b >= 2 and 1 <= M <= 65535");
  const MlpShape s = make_shape(dims, b);
  if (scratch_bytes < static_cast<size_t>(M) * s.per_worker * sizeof(float))
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_mlp_fused_stats needs %zu scratch bytes, got %zu",
                     static_cast<size_t>(M) * s.per_worker * sizeof(float), scratch_bytes);
  int prev = -1;
  ABS_CUDA_TRY(ctx, cudaGetDevice(&prev));
  if (prev != ctx->device) ABS_CUDA_TRY(ctx, cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* ws = static_cast<float*>(scratch);
  const long long pw = s.per_worker, d = s.d;
  const unsigned warp_blocks = static_cast<unsigned>((b * 32 + 255) / 256);
  fused_norm_kernel<<<dim3(kNormParts, M), 256, 0, st>>>(Gb, d, ws, pw, s.sCQ, b);
  auto layer = [&](long long sD, long long sH, int n_out, int n_in, long long oW, long long ob) {
    fused_rownorm_kernel<<<dim3(warp_blocks, M), 256, 0, st>>>(ws, pw, sD, sH, s.sCQ, b, n_out, n_in);
    // U[i][o] = sum_k h[i][k] dW[o][k]
    GemmArgs g{ws + sH, n_in, 1, pw, Gb + oW, 1, n_in, d, ws + s.sU, n_out, pw, nullptr, 0, nullptr, 0, 0,
               static_cast<int>(b), n_out, n_in, 1.f, 0};
    launch_gemm(ctx, g, M, st);
    fused_rowdot_kernel<<<dim3(warp_blocks, M), 256, 0, st>>>(ws, pw, sD, s.sU, s.sCQ, b, n_out, Gb, d, ob);
  };
  layer(s.sD1, s.sX, s.n1, s.n0, s.oW1, s.ob1);
  layer(s.sD2, s.sH1, s.n2, s.n1, s.oW2, s.ob2);
  layer(s.sD3, s.sH2, s.n3, s.n2, s.oW3, s.ob3);
  fused_finalize_kernel<<<M, 1024, 0, st>>>(ws, pw, s.sCQ, b, stats, ctx->flags);
  const cudaError_t e = cudaGetLastError();
  if (prev != ctx->device) cudaSetDevice(prev);
  if (e != cudaSuccess) return set_error(ctx, ABS_ERR_CUDA, "launch failed: %s", cudaGetErrorString(e));
  return ABS_OK;
}

// One communication round of local SGD on the MLP problem (Algorithm 2's structure, the
// per-sample statistic of Algorithm 1 once per round on the last local step, one worker's
// per-sample gradients materialised at a time).
extern "C" int abs_mlp_round(abs_ctx* ctx, const float* inputs, const int* labels, long long n, const int* dims,
                             const int* idx, long long idx_stride, float* X, int M, int H, long long b, float lr,
                             const abs_test_cfg* cfg, void* scratch, size_t scratch_bytes, float* G_scratch,
                             long long g_row_stride, float* Gb_scratch, abs_stats* stats, long long* T_out,
                             long long* b_dev, abs_round_ctl* ctl, void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (cfg == nullptr || Gb_scratch == nullptr || stats == nullptr || b_dev == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (H < 1 || b < 2) return set_error(ctx, ABS_ERR_INVALID_ARG, "need H >= 1 and b >= 2");
  int rc = check_dims(ctx, dims);
  if (rc != ABS_OK) return rc;
  const long long d = make_shape(dims, b).d;
  for (int h = 0; h < H; ++h) {
    const int* idx_h = idx + static_cast<long long>(h) * M * idx_stride;
    rc = abs_mlp_grads(ctx, inputs, labels, n, dims, idx_h, idx_stride, X, M, b, Gb_scratch, scratch, scratch_bytes,
                       stream);
    if (rc != ABS_OK) return rc;
    if (h == H - 1 && cfg->kind == ABS_TEST_NORM_WORKERS) {
      // Algorithm 2: no per-sample statistics at all; the batch gradients are tested after the step
    } else if (h == H - 1 && G_scratch == nullptr) {
      rc = abs_mlp_fused_stats(ctx, dims, b, M, scratch, scratch_bytes, Gb_scratch, stats, stream);
      if (rc != ABS_OK) return rc;
    } else if (h == H - 1) {
      for (int m = 0; m < M; ++m) {
        rc = abs_mlp_per_sample(ctx, dims, b, m, scratch, G_scratch, g_row_stride, stream);
        if (rc != ABS_OK) return rc;
        rc = abs_test_stats(ctx, G_scratch, ABS_F32, 1, b, d, g_row_stride, b * g_row_stride, nullptr, stats + m,
                            stream);
        if (rc != ABS_OK) return rc;
      }
    }
    rc = local_sgd_step(ctx, X, Gb_scratch, M, d, d, lr, h == H - 1 ? 1 : 0, stream);
    if (rc != ABS_OK) return rc;
  }
  if (ctl != nullptr) {      // Alg. 2: B <- B + H M b_k, k <- k + 1 (with the size the round ran with)
    rc = abs_round_count(ctx, ctl, b_dev, 1, static_cast<long long>(H) * M, 1, stream);
    if (rc != ABS_OK) return rc;
  }
  if (cfg->kind == ABS_TEST_NORM_WORKERS)
    return worker_gradient_test(ctx, Gb_scratch, M, d, b, cfg, stats, T_out, b_dev, stream);
  return abs_next_batch(ctx, stats, M, cfg, b_dev, T_out, b_dev, stream);
}
