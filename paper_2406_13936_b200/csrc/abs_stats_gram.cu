// Gram-matrix statistics kernel for bf16 rows and small batches (b <= 32), sm_100a.
//
// For few rows the b x b Gram matrix K = G G^T carries everything the batch-size test needs:
//   N = 1^T K 1 / b^2,  c_i = (K 1)_i / b,  sum_i ||g_i - gbar||^2 = tr K - 1^T K 1 / b
// (Eq. batch_grad and Eq. def_var expanded).  Products of two bf16 values are exact in fp32,
// so the tensor cores (mma.sync m16n8k16, bf16 in, fp32 out) form exact products and add them
// in fp32; the fp32 partial sums cover one tile (256 columns) and are then folded into fp64,
// which is where the cancellation in c_i - N happens.  The CUDA-core kernel needs about six
// instructions per element for bf16 input, which caps it below the HBM rate; here a warp issues
// one 16-byte shared-memory load per 8 elements and one MMA per 64.
//
// Pipeline: as in the tiled kernel, one producer warp issues TMA box loads [b rows] x [512 B]
// into a ring of stages; each of the 8 consumer warps owns one box of a stage, so the main loop
// has no cross-warp synchronisation.  The k index of the MMA only has to mean the same column
// in both operands, so each thread takes its fragments straight from a 16-byte load of its row
// (columns 8t..8t+7 of a 32-column chunk) instead of a transposing load.
#include <cuda_bf16.h>

#include "abs_pipeline.cuh"

namespace absk {
namespace {

constexpr int kWarpsC = 8;                    // consumer warps
// A warp spends about 1300 clocks of MMA issue on a box of 256 columns however few rows it has, so
// below 7 rows the tiled kernel (a few instructions per element) is faster: 6.2 against 3.5 TB/s at b = 4.
constexpr int kMinRows = 7;
constexpr int kThreadsG = kWarpsC * 32 + 32;
// box width in columns: 512-byte rows for one 16-row block, 256-byte rows for two
__host__ __device__ constexpr int box_cols_for(int nb) { return nb == 1 ? 256 : 128; }

struct GramParams {
  long long b, d;
  int stages;
  unsigned box_bytes;     // 16 * NB * 512
  unsigned stage_bytes;   // 8 boxes
  long long n_iters;
  int P;
  double* ws;
  float* gbar_out;
  unsigned* flags;
  long long timeout_cycles;
  // b < 8 and d a multiple of 256: one copy per stage through the segment map; a tile row then holds
  // the 8 boxes side by side (row_pitch = 8 * 512 bytes, box q starts q * 512 bytes into the row)
  int segment_map;
  unsigned row_pitch, box_stride;
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NB: 16-row blocks (b_pad = 16 NB).  Lower-triangular block pairs (I, J <= I) are accumulated.
template <int NB, bool WANT_GBAR>
__global__ void __launch_bounds__(kThreadsG, 1)
abs_stats_gram_kernel(const __grid_constant__ CUtensorMap tmap, const GramParams prm) {
  constexpr int NPAIR = NB * (NB + 1) / 2;
  constexpr int BP = 16 * NB;                 // padded rows
  constexpr int kBoxCols = box_cols_for(NB);
  constexpr unsigned kRowBytes = kBoxCols * 2;
  extern __shared__ __align__(128) unsigned char smem_raw[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = blockIdx.y, p = blockIdx.x;
  const int b = static_cast<int>(prm.b);
  const int S = prm.stages;

  unsigned char* stage_mem = smem_raw;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(stage_mem + static_cast<size_t>(S) * prm.stage_bytes);
  volatile unsigned* abort_flag = reinterpret_cast<volatile unsigned*>(bars + 2 * S);
  const uint32_t stage_u32 = smem_u32(stage_mem);
  const uint32_t full_u32 = smem_u32(bars);
  const uint32_t empty_u32 = smem_u32(bars + S);

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_u32 + 8u * s, 1);
      mbar_init(empty_u32 + 8u * s, kWarpsC);
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Rows b..BP-1 of every box are never written by the loads (the box has b rows): zero them once.
  if (b < BP && prm.segment_map) {
    const int pad_words = (BP - b) * static_cast<int>(prm.row_pitch / 4);        // rows b.. of every stage
    for (int st = 0; st < S; ++st) {
      unsigned* dst = reinterpret_cast<unsigned*>(stage_mem + static_cast<size_t>(st) * prm.stage_bytes + b * prm.row_pitch);
      for (int i = tid; i < pad_words; i += kThreadsG) dst[i] = 0u;
    }
  } else if (b < BP) {
    const int pad_words = (BP - b) * (kRowBytes / 4);
    for (int box = 0; box < S * kWarpsC; ++box) {
      unsigned* dst = reinterpret_cast<unsigned*>(stage_mem + static_cast<size_t>(box) * prm.box_bytes + b * kRowBytes);
      for (int i = tid; i < pad_words; i += kThreadsG) dst[i] = 0u;
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  pdl_launch_dependents();      // the finalisation kernel may be scheduled; it waits for this grid to complete

  const long long n_mine = (prm.n_iters > p) ? (prm.n_iters - p + prm.P - 1) / prm.P : 0;

  double dacc[NPAIR][2][4];
#pragma unroll
  for (int q = 0; q < NPAIR; ++q)
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int k = 0; k < 4; ++k) dacc[q][h][k] = 0.0;

  if (warp == kWarpsC) {
    if (lane == 0) {
      // s = i % S and the pass number i / S are carried along instead of divided out per tile
      int s = 0;
      uint32_t pass = 0;
      long long x0 = static_cast<long long>(p) * kWarpsC * kBoxCols;
      const long long x_step = static_cast<long long>(prm.P) * kWarpsC * kBoxCols;
      for (long long i = 0; i < n_mine; ++i, x0 += x_step) {
        if (pass > 0) mbar_wait(empty_u32 + 8u * s, (pass - 1) & 1u, abort_flag, prm.timeout_cycles);
        const uint32_t full = full_u32 + 8u * s;
        mbar_expect_tx(full, static_cast<uint32_t>(kWarpsC) * static_cast<uint32_t>(b) * kRowBytes);
        if (prm.segment_map) {        // a copy costs about 100 clocks plus 8 per row: one for the whole stage
          tma_load_4d(stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes, &tmap, 0, static_cast<int>(x0 / kSegElems), 0, m,
                      full);
        } else {
          for (int q = 0; q < kWarpsC; ++q)
            tma_load_3d(stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + static_cast<uint32_t>(q) * prm.box_bytes,
                        &tmap, static_cast<int>(x0 + q * kBoxCols), 0, m, full);
        }
        if (++s == S) {
          s = 0;
          ++pass;
        }
      }
      for (int s = 0; s < S && s < n_mine; ++s) {    // leave no copy in flight
        const long long last_use = (n_mine - 1 - s) / S;
        volatile unsigned ignore = 0u;
        mbar_wait(full_u32 + 8u * s, static_cast<uint32_t>(last_use & 1), &ignore, prm.timeout_cycles);
      }
    }
  } else {
    const int r = lane >> 2, t = lane & 3;
    const uint32_t pitch = prm.row_pitch;
    const uint32_t lane_off = static_cast<uint32_t>(r) * pitch + static_cast<uint32_t>(t) * 16u;
    const float inv_b = 1.0f / static_cast<float>(b);
    int s = -1;
    uint32_t parity = 1u;
    for (long long i = 0; i < n_mine; ++i) {
      if (++s == S) s = 0;                        // s = i % S, parity = (i / S) & 1 without dividing
      if (s == 0) parity ^= 1u;
      mbar_wait(full_u32 + 8u * s, parity, abort_flag, prm.timeout_cycles);
      const uint32_t base = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes +
                            static_cast<uint32_t>(warp) * prm.box_stride;
      float acc[NPAIR][2][4];
#pragma unroll
      for (int q = 0; q < NPAIR; ++q)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[q][h][k] = 0.f;

#pragma unroll
      for (int ch = 0; ch < kBoxCols / 32; ++ch) {
        uint4 lo[NB], hi[NB];
#pragma unroll
        for (int I = 0; I < NB; ++I) {
          lo[I] = lds128(base + lane_off + static_cast<uint32_t>(I * 16) * pitch + ch * 64);
          hi[I] = lds128(base + lane_off + static_cast<uint32_t>(I * 16 + 8) * pitch + ch * 64);
        }
#pragma unroll
        for (int I = 0; I < NB; ++I) {
#pragma unroll
          for (int J = 0; J <= I; ++J) {
            const int q = I * (I + 1) / 2 + J;
            // first k-step: columns 8t..8t+3 of the chunk; second: 8t+4..8t+7
            mma_bf16(acc[q][0], lo[I].x, hi[I].x, lo[I].y, hi[I].y, lo[J].x, lo[J].y);
            mma_bf16(acc[q][1], lo[I].x, hi[I].x, lo[I].y, hi[I].y, hi[J].x, hi[J].y);
            mma_bf16(acc[q][0], lo[I].z, hi[I].z, lo[I].w, hi[I].w, lo[J].z, lo[J].w);
            mma_bf16(acc[q][1], lo[I].z, hi[I].z, lo[I].w, hi[I].w, hi[J].z, hi[J].w);
          }
        }
      }
      if (WANT_GBAR) {
        // column means on the CUDA cores: lane owns 8 consecutive columns of the box
        const long long it = p + i * prm.P;
        const long long col = (it * kWarpsC + warp) * kBoxCols + lane * 8;
        if (lane * 8 < kBoxCols) {
        float cs[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = 0.f;
        for (int row = 0; row < b; ++row) {
          const uint4 u = lds128(base + static_cast<uint32_t>(row) * pitch + lane * 16);
          cs[0] += __uint_as_float(u.x << 16);
          cs[1] += __uint_as_float(u.x & 0xffff0000u);
          cs[2] += __uint_as_float(u.y << 16);
          cs[3] += __uint_as_float(u.y & 0xffff0000u);
          cs[4] += __uint_as_float(u.z << 16);
          cs[5] += __uint_as_float(u.z & 0xffff0000u);
          cs[6] += __uint_as_float(u.w << 16);
          cs[7] += __uint_as_float(u.w & 0xffff0000u);
        }
        float* dst = prm.gbar_out + static_cast<long long>(m) * prm.d + col;
        if (col + 8 <= prm.d && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
          *reinterpret_cast<float4*>(dst) = make_float4(cs[0] * inv_b, cs[1] * inv_b, cs[2] * inv_b, cs[3] * inv_b);
          *reinterpret_cast<float4*>(dst + 4) = make_float4(cs[4] * inv_b, cs[5] * inv_b, cs[6] * inv_b, cs[7] * inv_b);
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (col + j < prm.d) dst[j] = cs[j] * inv_b;
        }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_u32 + 8u * s);
#pragma unroll
      for (int q = 0; q < NPAIR; ++q)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int k = 0; k < 4; ++k) dacc[q][h][k] += static_cast<double>(acc[q][h][k]);
    }
  }

  // ---- CTA epilogue: fold the 8 warps' Gram matrices, convert to (e_r, V, N) ----
  __syncthreads();                              // all tiles consumed: the stage memory is free
  double* Kw = reinterpret_cast<double*>(stage_mem);        // [8 warps][BP][BP]
  if (warp < kWarpsC) {
    const int r = lane >> 2, t = lane & 3;
    double* mine = Kw + static_cast<size_t>(warp) * BP * BP;
#pragma unroll
    for (int I = 0; I < NB; ++I)
#pragma unroll
      for (int J = 0; J <= I; ++J) {
        const int q = I * (I + 1) / 2 + J;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int col = J * 16 + h * 8 + 2 * t;
          const int row = I * 16 + r;
          mine[row * BP + col] = dacc[q][h][0];
          mine[row * BP + col + 1] = dacc[q][h][1];
          mine[(row + 8) * BP + col] = dacc[q][h][2];
          mine[(row + 8) * BP + col + 1] = dacc[q][h][3];
        }
      }
  }
  __syncthreads();
  double* Kc = Kw + static_cast<size_t>(kWarpsC) * BP * BP;   // [BP][BP] CTA total (lower blocks)
  for (int idx = tid; idx < BP * BP; idx += kThreadsG) {
    double acc = 0.0;
    for (int w = 0; w < kWarpsC; ++w) acc += Kw[static_cast<size_t>(w) * BP * BP + idx];
    Kc[idx] = acc;
  }
  __syncthreads();
  double* rowsum = Kc + BP * BP;                              // [BP], then total and trace
  if (tid < BP) {
    const int i = tid;
    double acc = 0.0;
    for (int j = 0; j < BP; ++j) {
      // blocks above the diagonal were not accumulated: K is symmetric
      const bool lower = (j / 16) <= (i / 16);
      acc += lower ? Kc[i * BP + j] : Kc[j * BP + i];
    }
    rowsum[i] = acc;
  }
  __syncthreads();
  if (tid == 0) {
    double total = 0.0, trace = 0.0;
    for (int i = 0; i < BP; ++i) {
      total += rowsum[i];
      trace += Kc[i * BP + i];
    }
    rowsum[BP] = total;
    rowsum[BP + 1] = trace;
  }
  __syncthreads();
  {
    const double bd = static_cast<double>(b);
    const double total = rowsum[BP], trace = rowsum[BP + 1];
    const double Ncta = total / (bd * bd);
    double* out = prm.ws + (static_cast<size_t>(m) * prm.P + p) * (static_cast<size_t>(b) + 2);
    for (int i = tid; i < b; i += kThreadsG) out[i] = rowsum[i] / bd - Ncta;   // sum_j (g_ij - gbar_j) gbar_j
    if (tid == 0) {
      out[b] = trace - total / bd;                                             // sum_ij (g_ij - gbar_j)^2
      out[b + 1] = Ncta;
      if (*abort_flag) atomicOr(prm.flags, 1u);
    }
  }
}

template <int NB, bool WANT_GBAR>
int launch_gram_variant(abs_ctx* ctx, const CUtensorMap& tmap, const GramParams& prm, dim3 grid, size_t smem,
                        cudaStream_t stream) {
  auto kern = abs_stats_gram_kernel<NB, WANT_GBAR>;
  ABS_CUDA_TRY(ctx, ensure_dynamic_smem(ctx, kern, smem));
  kern<<<grid, kThreadsG, smem, stream>>>(tmap, prm);
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  return ABS_OK;
}

}  // namespace

int plan_stats_gram(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, abs_stats_plan* out) {
  if (dtype != ABS_BF16 || b < kMinRows || b > 32) return ABS_ERR_UNSUPPORTED;
  const int NB = b <= 16 ? 1 : 2;
  const unsigned box_bytes = static_cast<unsigned>(16 * NB) * static_cast<unsigned>(box_cols_for(NB)) * 2u;
  int stages = static_cast<int>(t.stats_stages > 0 ? t.stats_stages : 3);
  while (stages > 2 && static_cast<size_t>(stages) * box_bytes * kWarpsC + 1024 > smem_optin) --stages;
  memset(out, 0, sizeof(*out));
  out->route = 0;
  out->lanes_per_row = box_cols_for(NB) / 8;
  out->warps_per_box = 1;
  out->boxes_per_stage = kWarpsC;
  out->stages = stages;
  out->box_rows = static_cast<int>(b);
  out->row_boxes = 1;
  out->rows_per_thread = 0;
  out->cluster_size = 1;
  out->rows_per_cta = static_cast<int>(b);
  out->stage_bytes = box_bytes * kWarpsC;
  out->smem_bytes = static_cast<size_t>(stages) * box_bytes * kWarpsC + 1024;
  return ABS_OK;
}

int launch_stats_gram(abs_ctx* ctx, const StatsLaunch& a, int* P_out) {
  if (a.dtype != ABS_BF16 || a.b < kMinRows || a.b > 32 || !tma_addressable(a)) return ABS_ERR_UNSUPPORTED;
  const int NB = a.b <= 16 ? 1 : 2;
  const int BP = 16 * NB;
  const int kBoxCols = box_cols_for(NB);
  const unsigned kRowBytes = static_cast<unsigned>(kBoxCols) * 2u;
  const unsigned box_bytes = static_cast<unsigned>(BP) * kRowBytes;
  const unsigned stage_bytes = box_bytes * kWarpsC;
  int stages = static_cast<int>(ctx->tuning.stats_stages > 0 ? ctx->tuning.stats_stages : 3);
  const size_t epilogue = (static_cast<size_t>(kWarpsC + 1) * BP * BP + BP + 2) * sizeof(double);
  auto smem_for = [&](int s) {
    const size_t ring = static_cast<size_t>(s) * stage_bytes;
    return (ring > epilogue ? ring : epilogue) + static_cast<size_t>(2 * s) * 8 + 16 + 128;
  };
  while (stages > 2 && smem_for(stages) > ctx->smem_optin) --stages;
  if (smem_for(stages) > ctx->smem_optin) return ABS_ERR_UNSUPPORTED;
  // the epilogue reuses the ring: make sure the ring alone is large enough to be carved as laid out
  if (static_cast<size_t>(stages) * stage_bytes < epilogue) return ABS_ERR_UNSUPPORTED;

  const long long n_boxes = (a.d + kBoxCols - 1) / kBoxCols;
  const long long n_iters = (n_boxes + kWarpsC - 1) / kWarpsC;
  long long P = ctx->tuning.stats_ctas_per_worker > 0 ? ctx->tuning.stats_ctas_per_worker
                                                      : static_cast<long long>(ctx->sm_count) / a.M;
  if (P < 1) P = 1;
  if (P > n_iters) P = n_iters;
  if (P > 65535) P = 65535;
  const size_t need = static_cast<size_t>(a.M) * P * (a.b + 2) * sizeof(double);
  if (need > ctx->workspace_bytes)
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_test_stats needs %zu workspace bytes, context has %zu", need,
                     ctx->workspace_bytes);
  // fewer than 8 rows: the copy engine's cost per copy (about 100 clocks) shows; the segment map
  // brings a whole stage in one copy, if the rows can be cut into segments of 256 elements
  const bool segment_map = NB == 1 && a.b < 8 && a.d % kSegElems == 0 && kBoxCols == kSegElems;
  CUtensorMap tmap;
  int rc = segment_map ? encode_g_segment_map(ctx, a, kWarpsC, static_cast<int>(a.b), &tmap)
                       : encode_g_tensor_map(ctx, a, kBoxCols, static_cast<int>(a.b), &tmap);
  if (rc != ABS_OK) return rc;

  GramParams prm;
  prm.b = a.b;
  prm.d = a.d;
  prm.stages = stages;
  prm.box_bytes = box_bytes;
  prm.stage_bytes = stage_bytes;
  prm.n_iters = n_iters;
  prm.P = static_cast<int>(P);
  prm.ws = static_cast<double*>(ctx->workspace);
  prm.gbar_out = a.gbar_out;
  prm.flags = ctx->flags;
  prm.timeout_cycles = ctx->tuning.stats_timeout_cycles > 0 ? ctx->tuning.stats_timeout_cycles : kDefaultTimeoutCycles;
  prm.segment_map = segment_map ? 1 : 0;
  prm.row_pitch = segment_map ? kWarpsC * kRowBytes : kRowBytes;
  prm.box_stride = segment_map ? kRowBytes : box_bytes;
  const dim3 grid(static_cast<unsigned>(P), static_cast<unsigned>(a.M));
  const size_t smem = smem_for(stages);
  const bool gb = a.gbar_out != nullptr;
  if (NB == 1)
    rc = gb ? launch_gram_variant<1, true>(ctx, tmap, prm, grid, smem, a.stream)
            : launch_gram_variant<1, false>(ctx, tmap, prm, grid, smem, a.stream);
  else
    rc = gb ? launch_gram_variant<2, true>(ctx, tmap, prm, grid, smem, a.stream)
            : launch_gram_variant<2, false>(ctx, tmap, prm, grid, smem, a.stream);
  if (rc != ABS_OK) return rc;
  *P_out = static_cast<int>(P);
  return ABS_OK;
}

}  // namespace absk
