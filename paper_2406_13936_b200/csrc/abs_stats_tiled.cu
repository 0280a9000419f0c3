// Tiled single-pass statistics kernel for the batch-size test (sm_100a).
//
// What it computes, per worker m with rows g_1..g_b (Eq. batch_grad, Eq. def_var):
//   gbar_j = (1/b) sum_i g_ij           column means
//   V      = sum_j sum_i (g_ij - gbar_j)^2
//   N      = sum_j gbar_j^2
//   e_i    = sum_j (g_ij - gbar_j) gbar_j      (= <g_i, gbar> - N, formed centred)
// Every quantity is a sum over columns of something that needs only that column's
// b entries, so a CTA that holds all b rows of a column strip in shared memory can
// finish the strip without a second trip to HBM.  G is therefore read exactly once.
//
// Structure: one producer warp issues TMA tile loads (cp.async.bulk.tensor) into a ring
// of `stages` buffers guarded by full/empty mbarriers; 8 consumer warps take the strip
// apart.  A stage holds `bx` boxes of [b rows] x [lpr * 16 bytes]; `rs` warps share a
// box.  Inside a warp, lane = (sub-row-group, 16-byte column vector).  Each thread
// keeps its (at most 16) row vectors in registers between the column-sum sweep and
// the centred sweep; with more rows per thread the second sweep re-reads shared memory.
// Per-row sums e_i live in fp32 registers for `flush_every` tiles, then are folded into
// fp64 accumulators in shared memory that have a single owner thread each; V and N are
// folded into per-thread fp64 every tile.  All reductions have a fixed order.
#include <cuda_bf16.h>

#include "abs_internal.cuh"

namespace absk {
namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;

struct TiledParams {
  long long b, d;
  int lpr_log2;          // lanes per row
  int rs_log2;           // warps per box
  int bx;                // boxes per stage (= 8 >> rs_log2)
  int stages;
  int box_rows;          // rows per TMA box
  int n_row_boxes;       // TMA boxes stacked to cover b rows
  unsigned box_bytes;    // rows_pad * lpr * 16
  unsigned stage_bytes;  // bx * box_bytes
  long long n_iters;     // stage iterations per worker
  int P;                 // CTAs per worker
  int flush_every;
  double* ws;
  float* gbar_out;
  unsigned* flags;
  long long timeout_cycles;
};

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `limit` clock cycles (or as soon as another thread of the
// CTA gave up), raises the CTA's abort flag and returns false.  The caller carries on
// with whatever is in shared memory; the record is flagged ABS_STATUS_TIMEOUT.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile unsigned* abort_flag,
                                          long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*abort_flag) return false;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag || clock64() - t0 > limit) {
      *abort_flag = 1u;
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// ---- element traits ------------------------------------------------------------------------
template <typename T>
struct Vec;
template <>
struct Vec<float> {
  static constexpr int VE = 4;  // elements per 16-byte vector
  static __device__ __forceinline__ void unpack(const uint4& v, float (&x)[4]) {
    x[0] = __uint_as_float(v.x);
    x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z);
    x[3] = __uint_as_float(v.w);
  }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int VE = 8;
  // a bfloat16 is the upper half of a binary32: widening is a shift / a mask
  static __device__ __forceinline__ void unpack(const uint4& v, float (&x)[8]) {
    x[0] = __uint_as_float(v.x << 16);
    x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16);
    x[3] = __uint_as_float(v.y & 0xffff0000u);
    x[4] = __uint_as_float(v.z << 16);
    x[5] = __uint_as_float(v.z & 0xffff0000u);
    x[6] = __uint_as_float(v.w << 16);
    x[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// ---- the kernel ----------------------------------------------------------------------------
template <typename T, int RMAX, bool KEEP>
__global__ void __launch_bounds__(kThreads, 1)
abs_stats_tiled_kernel(const __grid_constant__ CUtensorMap tmap, const TiledParams prm) {
  constexpr int VE = Vec<T>::VE;
  extern __shared__ __align__(128) unsigned char smem_raw[];

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int m = blockIdx.y;
  const int p = blockIdx.x;
  const int b = static_cast<int>(prm.b);
  const int S = prm.stages;
  const int lpr = 1 << prm.lpr_log2;
  const int rs = 1 << prm.rs_log2;
  const unsigned row_bytes = static_cast<unsigned>(lpr) * 16u;

  // shared-memory carve-up
  unsigned char* stage_mem = smem_raw;
  float* part = reinterpret_cast<float*>(stage_mem + static_cast<size_t>(S) * prm.stage_bytes);   // [2][8][lpr*VE]
  double* e_acc = reinterpret_cast<double*>(part + 2 * kConsumerWarps * lpr * VE);                // [bx][b]
  double* red = e_acc + static_cast<size_t>(prm.bx) * b;                                          // [2][8]
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(red + 2 * kConsumerWarps);      // full[S], empty[S]
  volatile unsigned* abort_flag = reinterpret_cast<volatile unsigned*>(bars + 2 * S);

  const uint32_t stage_u32 = smem_u32(stage_mem);
  const uint32_t full_u32 = smem_u32(bars);
  const uint32_t empty_u32 = smem_u32(bars + S);

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_u32 + 8u * s, 1);
      mbar_init(empty_u32 + 8u * s, kConsumerWarps);
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i < prm.bx * b; i += kThreads) e_acc[i] = 0.0;
  __syncthreads();

  // iterations of this CTA: it = p, p + P, ... < n_iters
  const long long n_mine = (prm.n_iters > p) ? (prm.n_iters - p + prm.P - 1) / prm.P : 0;

  double vacc = 0.0, nacc = 0.0;

  if (warp == kConsumerWarps) {
    // ------------------------------ producer ------------------------------
    if (lane == 0) {
      const int box_cols = lpr * VE;
      for (long long i = 0; i < n_mine; ++i) {
        const int s = static_cast<int>(i % S);
        const long long use = i / S;
        if (use > 0)
          mbar_wait(empty_u32 + 8u * s, static_cast<uint32_t>((use - 1) & 1), abort_flag, prm.timeout_cycles);
        const uint32_t full = full_u32 + 8u * s;
        mbar_expect_tx(full, prm.stage_bytes);
        const long long it = p + i * prm.P;
        for (int q = 0; q < prm.bx; ++q) {
          const long long x = (it * prm.bx + q) * box_cols;
          const uint32_t dst0 =
              stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + static_cast<uint32_t>(q) * prm.box_bytes;
          for (int rb = 0; rb < prm.n_row_boxes; ++rb)
            tma_load_3d(dst0 + static_cast<uint32_t>(rb * prm.box_rows) * row_bytes, &tmap, static_cast<int>(x),
                        rb * prm.box_rows, m, full);
        }
      }
      // Leave no copy in flight: every armed phase of every buffer must have completed
      // before the CTA may exit (a bounded wait; normally already true).
      for (int s = 0; s < S && s < n_mine; ++s) {
        const long long last_use = (n_mine - 1 - s) / S;
        volatile unsigned ignore = 0u;
        mbar_wait(full_u32 + 8u * s, static_cast<uint32_t>(last_use & 1), &ignore, prm.timeout_cycles);
      }
    }
  } else {
    // ------------------------------ consumers ------------------------------
    const int q = warp >> prm.rs_log2;            // box of this warp within the stage
    const int wr = warp & (rs - 1);               // warp index within the box's group
    const int sub = lane >> prm.lpr_log2;         // sub-row-group within the warp
    const int cv = lane & (lpr - 1);              // 16-byte column vector within the box row
    const int subs = 32 >> prm.lpr_log2;
    const int RG = rs * subs;                     // row groups per box
    const int rg = wr * subs + sub;
    const int n_rows_mine = (b > rg) ? (b - rg + RG - 1) / RG : 0;   // rows rg, rg+RG, ...
    const unsigned row_step = static_cast<unsigned>(RG) * row_bytes;
    const uint32_t my_off = static_cast<uint32_t>(q) * prm.box_bytes + static_cast<uint32_t>(rg) * row_bytes +
                            static_cast<uint32_t>(cv) * 16u;
    const float inv_b = 1.0f / static_cast<float>(b);
    const bool first_rg = (rg == 0);
    double* e_mine = e_acc + static_cast<size_t>(q) * b;

    float e[RMAX];
#pragma unroll
    for (int k = 0; k < RMAX; ++k) e[k] = 0.f;
    int since_flush = 0;

    for (long long i = 0; i < n_mine; ++i) {
      const int s = static_cast<int>(i % S);
      const uint32_t parity = static_cast<uint32_t>((i / S) & 1);
      mbar_wait(full_u32 + 8u * s, parity, abort_flag, prm.timeout_cycles);
      const uint32_t base = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + my_off;

      // sweep 1: column sums over this thread's rows
      uint4 v[KEEP ? RMAX : 1];
      float cs[VE];
#pragma unroll
      for (int j = 0; j < VE; ++j) cs[j] = 0.f;
#pragma unroll
      for (int k = 0; k < RMAX; ++k) {
        if (k < n_rows_mine) {
          const uint4 u = lds128(base + static_cast<uint32_t>(k) * row_step);
          if (KEEP) v[k] = u;
          float x[VE];
          Vec<T>::unpack(u, x);
#pragma unroll
          for (int j = 0; j < VE; ++j) cs[j] += x[j];
        }
      }
      if (KEEP) {   // the tile now lives in registers: hand the buffer back
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_u32 + 8u * s);
      }
      for (int off = lpr; off < 32; off <<= 1) {
#pragma unroll
        for (int j = 0; j < VE; ++j) cs[j] += __shfl_xor_sync(0xffffffffu, cs[j], off);
      }
      if (rs > 1) {
        float* buf = part + static_cast<size_t>(i & 1) * (kConsumerWarps * lpr * VE);
        if (sub == 0) {
#pragma unroll
          for (int j = 0; j < VE; ++j) buf[(warp * lpr + cv) * VE + j] = cs[j];
        }
        named_bar_sync(1 + q, rs * 32);
#pragma unroll
        for (int j = 0; j < VE; ++j) cs[j] = 0.f;
        const int w0 = q << prm.rs_log2;
        for (int w = 0; w < rs; ++w) {
          const float* src = buf + ((w0 + w) * lpr + cv) * VE;
#pragma unroll
          for (int j = 0; j < VE; ++j) cs[j] += src[j];
        }
      }
      float g[VE];
#pragma unroll
      for (int j = 0; j < VE; ++j) g[j] = cs[j] * inv_b;

      if (first_rg) {
        float nl = 0.f;
#pragma unroll
        for (int j = 0; j < VE; ++j) nl = fmaf(g[j], g[j], nl);
        nacc += static_cast<double>(nl);
        if (prm.gbar_out != nullptr) {
          const long long it = p + i * prm.P;
          const long long col = ((it * prm.bx + q) * lpr + cv) * VE;
          float* dst = prm.gbar_out + static_cast<long long>(m) * prm.d + col;
          if (col + VE <= prm.d && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
#pragma unroll
            for (int j = 0; j < VE; j += 4)
              *reinterpret_cast<float4*>(dst + j) = make_float4(g[j], g[j + 1], g[j + 2], g[j + 3]);
          } else {
#pragma unroll
            for (int j = 0; j < VE; ++j)
              if (col + j < prm.d) dst[j] = g[j];
          }
        }
      }

      // sweep 2: centred sums
      float vl = 0.f;
#pragma unroll
      for (int k = 0; k < RMAX; ++k) {
        if (k < n_rows_mine) {
          const uint4 u = KEEP ? v[k] : lds128(base + static_cast<uint32_t>(k) * row_step);
          float x[VE];
          Vec<T>::unpack(u, x);
          float ek = e[k];
#pragma unroll
          for (int j = 0; j < VE; ++j) {
            const float dlt = x[j] - g[j];
            vl = fmaf(dlt, dlt, vl);
            ek = fmaf(dlt, g[j], ek);
          }
          e[k] = ek;
        }
      }
      vacc += static_cast<double>(vl);
      if (!KEEP) {
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_u32 + 8u * s);
      }

      if (++since_flush >= prm.flush_every || i + 1 == n_mine) {
        since_flush = 0;
#pragma unroll
        for (int k = 0; k < RMAX; ++k) {
          float ek = e[k];
          for (int off = 1; off < lpr; off <<= 1) ek += __shfl_xor_sync(0xffffffffu, ek, off);
          if (cv == 0 && k < n_rows_mine) e_mine[rg + k * RG] += static_cast<double>(ek);
          e[k] = 0.f;
        }
      }
    }
  }

  // ------------------------------ CTA epilogue ------------------------------
  vacc = warp_sum(vacc);
  nacc = warp_sum(nacc);
  if (lane == 0 && warp < kConsumerWarps) {
    red[warp] = vacc;
    red[kConsumerWarps + warp] = nacc;
  }
  __syncthreads();
  double* out = prm.ws + (static_cast<size_t>(m) * prm.P + p) * (static_cast<size_t>(b) + 2);
  for (int r = tid; r < b; r += kThreads) {
    double acc = 0.0;
    for (int q = 0; q < prm.bx; ++q) acc += e_acc[static_cast<size_t>(q) * b + r];
    out[r] = acc;
  }
  if (tid == 0) {
    double vs = 0.0, ns = 0.0;
    for (int w = 0; w < kConsumerWarps; ++w) {
      vs += red[w];
      ns += red[kConsumerWarps + w];
    }
    out[b] = vs;
    out[b + 1] = ns;
    if (*abort_flag) atomicOr(prm.flags, 1u);
  }
}

// ---- host side -----------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

struct TileChoice {
  int lpr_log2, rs_log2, bx, stages, box_rows, n_row_boxes, rmax;
  bool keep;
  unsigned box_bytes, stage_bytes;
  size_t smem_bytes;
};

size_t extras_bytes(int lpr, int ve, int bx, long long b, int stages) {
  return static_cast<size_t>(2 * kConsumerWarps * lpr * ve) * 4 + static_cast<size_t>(bx) * b * 8 +
         2 * kConsumerWarps * 8 + static_cast<size_t>(2 * stages) * 8 + 16;
}

// Picks the widest box rows that leave every thread at most 16 rows (so the tile can stay in
// registers between the sweeps) and whose stage fits the per-stage budget.
bool choose_tile(long long b, int ve, size_t smem_optin, long long want_stages, size_t stage_max, TileChoice* c) {
  const int n_row_boxes = static_cast<int>((b + 255) / 256);
  for (int pass = 0; pass < 2; ++pass) {            // pass 0: tile kept in registers; pass 1: re-read
    const int rows_per_thread = pass == 0 ? 16 : 32;
    for (int lpr_log2 = 5; lpr_log2 >= 0; --lpr_log2) {
      const int lpr = 1 << lpr_log2;
      const int subs = 32 / lpr;
      // every TMA destination must start on a 128-byte boundary: round the rows of a box up
      // so that box_rows * lpr * 16 is a multiple of 128 (only matters for rows under 128 bytes)
      const int row_align = lpr >= 8 ? 1 : 8 / lpr;
      int box_rows = static_cast<int>((b + n_row_boxes - 1) / n_row_boxes);
      box_rows = (box_rows + row_align - 1) / row_align * row_align;
      const long long rows_pad = static_cast<long long>(box_rows) * n_row_boxes;
      const long long need_rg = (b + rows_per_thread - 1) / rows_per_thread;
      int rs_log2 = 0;
      while (rs_log2 < 3 && (static_cast<long long>(subs) << rs_log2) < need_rg) ++rs_log2;
      if ((static_cast<long long>(subs) << rs_log2) < need_rg) continue;
      // more warps per box if the stage would be too large
      while (rs_log2 < 3 && static_cast<size_t>(kConsumerWarps >> rs_log2) * rows_pad * lpr * 16 > stage_max) ++rs_log2;
      const int bx = kConsumerWarps >> rs_log2;
      const size_t stage = static_cast<size_t>(bx) * rows_pad * lpr * 16;
      if (stage > stage_max) continue;
      int stages = static_cast<int>(want_stages > 0 ? want_stages : 3);
      while (stages > 2 && stages * stage + extras_bytes(lpr, ve, bx, b, stages) + 128 > smem_optin) --stages;
      if (stages * stage + extras_bytes(lpr, ve, bx, b, stages) + 128 > smem_optin) continue;
      const long long RG = static_cast<long long>(subs) << rs_log2;
      const long long R = (b + RG - 1) / RG;
      c->lpr_log2 = lpr_log2;
      c->rs_log2 = rs_log2;
      c->bx = bx;
      c->stages = stages;
      c->box_rows = box_rows;
      c->n_row_boxes = n_row_boxes;
      c->keep = (pass == 0);
      c->rmax = pass == 0 ? (R <= 4 ? 4 : (R <= 8 ? 8 : 16)) : 32;
      c->box_bytes = static_cast<unsigned>(rows_pad * lpr * 16);
      c->stage_bytes = static_cast<unsigned>(stage);
      c->smem_bytes = stages * stage + extras_bytes(lpr, ve, bx, b, stages) + 128;
      return true;
    }
  }
  return false;
}

template <typename T, int RMAX, bool KEEP>
int launch_variant(abs_ctx* ctx, const CUtensorMap& tmap, const TiledParams& prm, dim3 grid, size_t smem,
                   cudaStream_t stream) {
  auto kern = abs_stats_tiled_kernel<T, RMAX, KEEP>;
  ABS_CUDA_TRY(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  kern<<<grid, kThreads, smem, stream>>>(tmap, prm);
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  return ABS_OK;
}

template <typename T>
int launch_typed(abs_ctx* ctx, const TileChoice& c, const CUtensorMap& tmap, const TiledParams& prm, dim3 grid,
                 cudaStream_t stream) {
  if (!c.keep) return launch_variant<T, 32, false>(ctx, tmap, prm, grid, c.smem_bytes, stream);
  switch (c.rmax) {
    case 4: return launch_variant<T, 4, true>(ctx, tmap, prm, grid, c.smem_bytes, stream);
    case 8: return launch_variant<T, 8, true>(ctx, tmap, prm, grid, c.smem_bytes, stream);
    default: return launch_variant<T, 16, true>(ctx, tmap, prm, grid, c.smem_bytes, stream);
  }
}

}  // namespace

int launch_stats_tiled(abs_ctx* ctx, const StatsLaunch& a, int* P_out) {
  const int es = a.dtype == ABS_F32 ? 4 : 2;
  const int ve = 16 / es;
  const unsigned long long row_b = static_cast<unsigned long long>(a.row_stride) * es;
  const unsigned long long wrk_b = static_cast<unsigned long long>(a.M > 1 ? a.worker_stride : a.b * a.row_stride) * es;
  if ((reinterpret_cast<uintptr_t>(a.G) & 15u) || (row_b & 15u) || (wrk_b & 15u)) return ABS_ERR_UNSUPPORTED;
  if (a.b > kMaxFastRows || a.d > 0x7fff0000ll || a.M > 65535) return ABS_ERR_UNSUPPORTED;
  if (row_b >= (1ull << 40) || wrk_b >= (1ull << 40)) return ABS_ERR_UNSUPPORTED;
  EncodeTiledFn encode = encode_tiled_fn();
  if (encode == nullptr) return ABS_ERR_UNSUPPORTED;

  TileChoice c;
  const size_t stage_max = ctx->tuning.stats_stage_kb > 0 ? static_cast<size_t>(ctx->tuning.stats_stage_kb) << 10
                                                          : (64u << 10);
  if (!choose_tile(a.b, ve, ctx->smem_optin, ctx->tuning.stats_stages, stage_max, &c)) return ABS_ERR_UNSUPPORTED;

  const int lpr = 1 << c.lpr_log2;
  const long long box_cols = static_cast<long long>(lpr) * ve;
  const long long n_boxes = (a.d + box_cols - 1) / box_cols;
  const long long n_iters = (n_boxes + c.bx - 1) / c.bx;

  int ctas_per_sm = static_cast<int>(ctx->smem_optin / (c.smem_bytes + 1024));
  if (ctas_per_sm < 1) ctas_per_sm = 1;
  if (ctas_per_sm > 2) ctas_per_sm = 2;
  long long P = ctx->tuning.stats_ctas_per_worker > 0
                    ? ctx->tuning.stats_ctas_per_worker
                    : (static_cast<long long>(ctx->sm_count) * ctas_per_sm) / a.M;
  if (P < 1) P = 1;
  if (P > n_iters) P = n_iters;
  if (P > 65535) P = 65535;
  const size_t need = static_cast<size_t>(a.M) * P * (a.b + 2) * sizeof(double);
  if (need > ctx->workspace_bytes)
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_test_stats needs %zu workspace bytes, context has %zu", need,
                     ctx->workspace_bytes);

  CUtensorMap tmap;
  const cuuint64_t gdim[3] = {static_cast<cuuint64_t>(a.d), static_cast<cuuint64_t>(a.b), static_cast<cuuint64_t>(a.M)};
  const cuuint64_t gstr[2] = {row_b, wrk_b};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(c.box_rows), 1u};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  const CUresult r = encode(&tmap, a.dtype == ABS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                            3, const_cast<void*>(a.G), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return set_error(ctx, ABS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r));

  TiledParams prm;
  prm.b = a.b;
  prm.d = a.d;
  prm.lpr_log2 = c.lpr_log2;
  prm.rs_log2 = c.rs_log2;
  prm.bx = c.bx;
  prm.stages = c.stages;
  prm.box_rows = c.box_rows;
  prm.n_row_boxes = c.n_row_boxes;
  prm.box_bytes = c.box_bytes;
  prm.stage_bytes = c.stage_bytes;
  prm.n_iters = n_iters;
  prm.P = static_cast<int>(P);
  prm.flush_every = static_cast<int>(ctx->tuning.stats_flush_every > 0 ? ctx->tuning.stats_flush_every : 8);
  prm.ws = static_cast<double*>(ctx->workspace);
  prm.gbar_out = a.gbar_out;
  prm.flags = ctx->flags;
  prm.timeout_cycles = 4000000000ll;   // about two seconds of SM clock

  const dim3 grid(static_cast<unsigned>(P), static_cast<unsigned>(a.M));
  int rc;
  if (a.dtype == ABS_F32)
    rc = launch_typed<float>(ctx, c, tmap, prm, grid, a.stream);
  else
    rc = launch_typed<__nv_bfloat16>(ctx, c, tmap, prm, grid, a.stream);
  if (rc != ABS_OK) return rc;
  *P_out = static_cast<int>(P);
  return ABS_OK;
}

}  // namespace absk
