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

#include "abs_pipeline.cuh"

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
  int drop_loads;        // fault injection for the bounded waits: the loader issues nothing
  int boxes_per_copy;    // neighbouring boxes that one copy brings in as one tile row: 1; 2, 4 or 8 for very small batches
  int segment_map;       // the tensor map is the 4-D segment map (x counted in segments of 256 elements)
  const unsigned* guard; // NULL, or a device word: while it is zero the kernel has nothing to do
};

// ---- the kernel ----------------------------------------------------------------------------
// RMAX: rows a thread owns (exactly ceil(b / row groups) when KEEP, an upper bound otherwise);
// KEEP: the rows stay in registers between the sweeps; FULL: every thread owns exactly RMAX
// rows (no predicates at all).  Variants with
// at most 8 rows per thread are compiled for two CTAs per SM.
template <typename T, int RMAX, bool KEEP, bool FULL>
__global__ void __launch_bounds__(kThreads, (RMAX <= 8 ? 2 : 1))
abs_stats_tiled_kernel(const __grid_constant__ CUtensorMap tmap, const TiledParams prm) {
  constexpr int VE = Vec<T>::VE;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  // a recomputation that the finalisation before this launch did not ask for
  if (prm.guard != nullptr && *reinterpret_cast<const volatile unsigned*>(prm.guard) == 0u) return;

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
  pdl_launch_dependents();      // the finalisation kernel may be scheduled; it waits for this grid to complete

  // iterations of this CTA: it = p, p + P, ... < n_iters
  const long long n_mine = (prm.n_iters > p) ? (prm.n_iters - p + prm.P - 1) / prm.P : 0;

  double vacc = 0.0, nacc = 0.0;

  if (warp == kConsumerWarps) {
    // ------------------------------ producer ------------------------------
    if (lane == 0) {
      const int box_cols = lpr * VE;
      // s = i % S and the pass number i / S are carried along: a 64-bit division per tile is most
      // of the work when a tile is a few KiB (very small batches)
      int s = 0;
      uint32_t pass = 0;
      long long x0 = static_cast<long long>(p) * prm.bx * box_cols;           // first column of the stage
      const long long x_step = static_cast<long long>(prm.P) * prm.bx * box_cols;
      for (long long i = 0; i < n_mine; ++i, x0 += x_step) {
        const int s_now = s;
        const uint32_t pass_now = pass;
        if (++s == S) {
          s = 0;
          ++pass;
        }
        if (pass_now > 0)
          mbar_wait(empty_u32 + 8u * s_now, (pass_now - 1) & 1u, abort_flag, prm.timeout_cycles);
        if (prm.drop_loads) continue;     // test hook: the consumers' waits must run out, not hang
        const uint32_t full = full_u32 + 8u * s_now;
        mbar_expect_tx(full, prm.stage_bytes);
        // a copy costs the copy engine about 100 clocks plus 8 per row, so boxes of a few rows are
        // brought in several at a time: one copy whose rows are boxes_per_copy boxes long, which
        // as many consumer warps share side by side
        const int q_step = prm.boxes_per_copy;
        for (int q = 0; q < prm.bx; q += q_step) {
          const long long x = x0 + static_cast<long long>(q) * box_cols;
          const uint32_t dst0 =
              stage_u32 + static_cast<uint32_t>(s_now) * prm.stage_bytes + static_cast<uint32_t>(q) * prm.box_bytes;
          if (prm.segment_map) {
            tma_load_4d(dst0, &tmap, 0, static_cast<int>(x / kSegElems), 0, m, full);
          } else {
            for (int rb = 0; rb < prm.n_row_boxes; ++rb)
              tma_load_3d(dst0 + static_cast<uint32_t>(rb * prm.box_rows) * row_bytes * q_step, &tmap, static_cast<int>(x),
                          rb * prm.box_rows, m, full);
          }
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
    // In the register-resident variants RMAX is exactly ceil(b / RG): every thread owns rows
    // 0..RMAX-2 of its group and only the last one can fall past the batch.
    const bool last_ok = n_rows_mine >= RMAX;
    // boxes_per_copy > 1: box q is one of the boxes that lie side by side in a longer tile row
    const int bpc = prm.boxes_per_copy;
    const unsigned row_pitch = static_cast<unsigned>(bpc) * row_bytes;
    const uint32_t box_off = static_cast<uint32_t>(q / bpc) * static_cast<uint32_t>(bpc) * prm.box_bytes +
                             static_cast<uint32_t>(q % bpc) * row_bytes;
    const unsigned row_step = static_cast<unsigned>(RG) * row_pitch;
    const uint32_t my_off = box_off + static_cast<uint32_t>(rg) * row_pitch + static_cast<uint32_t>(cv) * 16u;
    const float inv_b = 1.0f / static_cast<float>(b);
    const bool first_rg = (rg == 0);
    double* e_mine = e_acc + static_cast<size_t>(q) * b;

    float e[RMAX];
#pragma unroll
    for (int k = 0; k < RMAX; ++k) e[k] = 0.f;
    int since_flush = 0;

    int s = -1;
    uint32_t parity = 1u;
    for (long long i = 0; i < n_mine; ++i) {
      if (++s == S) s = 0;                        // s = i % S, parity = (i / S) & 1 without dividing
      if (s == 0) parity ^= 1u;
      mbar_wait(full_u32 + 8u * s, parity, abort_flag, prm.timeout_cycles);
      const uint32_t base = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + my_off;
      const uint32_t base0 = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + box_off +
                             static_cast<uint32_t>(cv) * 16u;   // row 0

      // sweep 1: column sums over this thread's rows
      uint4 v[KEEP ? RMAX : 1];
      float cs[VE];
#pragma unroll
      for (int j = 0; j < VE; ++j) cs[j] = 0.f;
#pragma unroll
      for (int k = 0; k < RMAX; ++k) {
        // Rows past the batch are loaded from a safe address and zeroed by a select: no branch,
        // so the loads of a sweep are issued back to back.
        const bool ok = FULL || (KEEP ? (k < RMAX - 1 || last_ok) : k < n_rows_mine);
        uint4 u = lds128(ok ? base + static_cast<uint32_t>(k) * row_step : base0);
        if (!ok) u = make_uint4(0u, 0u, 0u, 0u);
        if (KEEP) v[k] = u;
        float x[VE];
        Vec<T>::unpack(u, x);
#pragma unroll
        for (int j = 0; j < VE; ++j) cs[j] += x[j];
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
          smem_store_vec<VE>(buf + (warp * lpr + cv) * VE, cs);
        }
        named_bar_sync(1 + q, rs * 32);
#pragma unroll
        for (int j = 0; j < VE; ++j) cs[j] = 0.f;
        const int w0 = q << prm.rs_log2;
        for (int w = 0; w < rs; ++w) {
          const float* src = buf + ((w0 + w) * lpr + cv) * VE;
          smem_add_vec<VE>(src, cs);
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
      float vl[VE];     // one accumulator per column: VE independent dependency chains
#pragma unroll
      for (int j = 0; j < VE; ++j) vl[j] = 0.f;
#pragma unroll
      for (int k = 0; k < RMAX; ++k) {
        const bool ok = FULL || (KEEP ? (k < RMAX - 1 || last_ok) : k < n_rows_mine);
        const uint4 u = KEEP ? v[k] : lds128(ok ? base + static_cast<uint32_t>(k) * row_step : base0);
        float x[VE];
        Vec<T>::unpack(u, x);
        float ea = 0.f, eb = 0.f;
#pragma unroll
        for (int j = 0; j < VE; j += 2) {
          const float d0 = ok ? x[j] - g[j] : 0.f;
          const float d1 = ok ? x[j + 1] - g[j + 1] : 0.f;
          vl[j] = fmaf(d0, d0, vl[j]);
          vl[j + 1] = fmaf(d1, d1, vl[j + 1]);
          ea = fmaf(d0, g[j], ea);
          eb = fmaf(d1, g[j + 1], eb);
        }
        e[k] += ea + eb;
      }
      {
        float vs = 0.f;
#pragma unroll
        for (int j = 0; j < VE; ++j) vs += vl[j];
        vacc += static_cast<double>(vs);
      }
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
          if (cv == 0 && (FULL || (KEEP ? (k < RMAX - 1 || last_ok) : k < n_rows_mine))) e_mine[rg + k * RG] += static_cast<double>(ek);
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
struct TileChoice {
  int lpr_log2, rs_log2, bx, stages, box_rows, n_row_boxes, rmax;
  bool keep, full, small_rows;
  unsigned box_bytes, stage_bytes;
  size_t smem_bytes;
};

size_t extras_bytes(int lpr, int ve, int bx, long long b, int stages) {
  return static_cast<size_t>(2 * kConsumerWarps * lpr * ve) * 4 + static_cast<size_t>(bx) * b * 8 +
         2 * kConsumerWarps * 8 + static_cast<size_t>(2 * stages) * 8 + 16;
}

// Picks the widest box rows that leave every thread at most 16 rows (so the tile can stay in
// registers between the sweeps) and whose stage fits the per-stage budget.
bool choose_tile(long long b, int ve, size_t smem_optin, long long want_stages, size_t stage_max, int keep_rows,
                 TileChoice* c) {
  const int n_row_boxes = static_cast<int>((b + 255) / 256);
  // with at most 8 rows per thread the kernel is compiled for two CTAs per SM: leave room for both
  const size_t smem_budget = keep_rows <= 8 ? (smem_optin - 2048) / 2 : smem_optin;
  for (int pass = 0; pass < 2; ++pass) {            // pass 0: tile kept in registers; pass 1: re-read
    const int rows_per_thread = pass == 0 ? keep_rows : 32;
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
      while (stages > 2 && stages * stage + extras_bytes(lpr, ve, bx, b, stages) + 128 > smem_budget) --stages;
      if (stages * stage + extras_bytes(lpr, ve, bx, b, stages) + 128 > smem_budget) continue;
      const long long RG = static_cast<long long>(subs) << rs_log2;
      const long long R = (b + RG - 1) / RG;
      c->lpr_log2 = lpr_log2;
      c->rs_log2 = rs_log2;
      c->bx = bx;
      c->stages = stages;
      c->box_rows = box_rows;
      c->n_row_boxes = n_row_boxes;
      c->keep = (pass == 0);
      c->rmax = pass == 0 ? static_cast<int>(R) : 32;
      c->full = (b % RG == 0) && (pass == 0 ? (R == 2 || R == 4 || R == 8 || R == 16) : R == 32);
      // boxes of fewer than 8 rows, one per consumer warp: candidates for sharing a copy
      c->small_rows = (b < 8 && lpr == 32 && rs_log2 == 0 && n_row_boxes == 1);
      c->box_bytes = static_cast<unsigned>(rows_pad * lpr * 16);
      c->stage_bytes = static_cast<unsigned>(stage);
      c->smem_bytes = stages * stage + extras_bytes(lpr, ve, bx, b, stages) + 128;
      return true;
    }
  }
  return false;
}

// The tile shape for b rows: two resident CTAs per SM with 32 KiB tile buffers and 8 rows per
// thread, or (default) one CTA with 64 KiB buffers and 16 rows per thread.
bool tiled_choice(const Tuning& t, size_t smem_optin, int ve, long long b, TileChoice* c) {
  const int per_sm = t.stats_ctas_per_sm > 0 ? static_cast<int>(t.stats_ctas_per_sm) : 1;
  const size_t stage_max = t.stats_stage_kb > 0 ? static_cast<size_t>(t.stats_stage_kb) << 10
                                                : (per_sm == 2 ? (32u << 10) : (64u << 10));
  return choose_tile(b, ve, smem_optin, t.stats_stages, stage_max, per_sm == 2 ? 8 : 16, c) ||
         choose_tile(b, ve, smem_optin, t.stats_stages, 64u << 10, 16, c);
}

template <typename T, int RMAX, bool KEEP, bool FULL>
int launch_variant(abs_ctx* ctx, const CUtensorMap& tmap, const TiledParams& prm, dim3 grid, size_t smem,
                   cudaStream_t stream) {
  auto kern = abs_stats_tiled_kernel<T, RMAX, KEEP, FULL>;
  ABS_CUDA_TRY(ctx, ensure_dynamic_smem(ctx, kern, smem));
  kern<<<grid, kThreads, smem, stream>>>(tmap, prm);
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  return ABS_OK;
}

template <typename T>
int launch_typed(abs_ctx* ctx, const TileChoice& c, const CUtensorMap& tmap, const TiledParams& prm, dim3 grid,
                 cudaStream_t stream) {
  const size_t smem = c.smem_bytes;
  if (!c.keep)
    return c.full ? launch_variant<T, 32, false, true>(ctx, tmap, prm, grid, smem, stream)
                  : launch_variant<T, 32, false, false>(ctx, tmap, prm, grid, smem, stream);
  if (c.full) {
    switch (c.rmax) {
      case 2: return launch_variant<T, 2, true, true>(ctx, tmap, prm, grid, smem, stream);
      case 4: return launch_variant<T, 4, true, true>(ctx, tmap, prm, grid, smem, stream);
      case 8: return launch_variant<T, 8, true, true>(ctx, tmap, prm, grid, smem, stream);
      default: return launch_variant<T, 16, true, true>(ctx, tmap, prm, grid, smem, stream);
    }
  }
  switch (c.rmax) {
#define ABS_TILED_CASE(R) \
  case R: return launch_variant<T, R, true, false>(ctx, tmap, prm, grid, smem, stream);
    ABS_TILED_CASE(1) ABS_TILED_CASE(2) ABS_TILED_CASE(3) ABS_TILED_CASE(4) ABS_TILED_CASE(5) ABS_TILED_CASE(6)
    ABS_TILED_CASE(7) ABS_TILED_CASE(8) ABS_TILED_CASE(9) ABS_TILED_CASE(10) ABS_TILED_CASE(11) ABS_TILED_CASE(12)
    ABS_TILED_CASE(13) ABS_TILED_CASE(14) ABS_TILED_CASE(15)
#undef ABS_TILED_CASE
    default: return launch_variant<T, 16, true, false>(ctx, tmap, prm, grid, smem, stream);
  }
}

}  // namespace

int plan_stats_tiled(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, abs_stats_plan* out) {
  if (b < 2 || b > kMaxFastRows) return ABS_ERR_UNSUPPORTED;
  TileChoice c;
  if (!tiled_choice(t, smem_optin, dtype == ABS_F32 ? 4 : 8, b, &c)) return ABS_ERR_UNSUPPORTED;
  memset(out, 0, sizeof(*out));
  out->route = 2;
  out->lanes_per_row = 1 << c.lpr_log2;
  out->warps_per_box = 1 << c.rs_log2;
  out->boxes_per_stage = c.bx;
  out->stages = c.stages;
  out->box_rows = c.box_rows;
  out->row_boxes = c.n_row_boxes;
  out->rows_per_thread = c.rmax;
  out->keep_in_registers = c.keep ? 1 : 0;
  out->full = c.full ? 1 : 0;
  out->cluster_size = 1;
  out->rows_per_cta = static_cast<int>(b);
  out->stage_bytes = c.stage_bytes;
  out->smem_bytes = c.smem_bytes;
  return ABS_OK;
}

bool stats_tiled_feasible(abs_ctx* ctx, const StatsLaunch& a) {
  if (a.b > kMaxFastRows || !tma_addressable(a)) return false;
  TileChoice c;
  if (!tiled_choice(ctx->tuning, ctx->smem_optin, a.dtype == ABS_F32 ? 4 : 8, a.b, &c)) return false;
  // the launcher never uses more than two CTAs per SM
  const size_t worst = static_cast<size_t>(ctx->sm_count) * 2 + static_cast<size_t>(a.M);
  return worst * (a.b + 2) * sizeof(double) <= ctx->workspace_bytes;
}

int launch_stats_tiled(abs_ctx* ctx, const StatsLaunch& a, int* P_out) {
  const int es = a.dtype == ABS_F32 ? 4 : 2;
  const int ve = 16 / es;
  if (a.b > kMaxFastRows || !tma_addressable(a)) return ABS_ERR_UNSUPPORTED;

  TileChoice c;
  if (!tiled_choice(ctx->tuning, ctx->smem_optin, ve, a.b, &c)) return ABS_ERR_UNSUPPORTED;

  const int lpr = 1 << c.lpr_log2;
  const long long box_cols = static_cast<long long>(lpr) * ve;
  const long long n_boxes = (a.d + box_cols - 1) / box_cols;
  const long long n_iters = (n_boxes + c.bx - 1) / c.bx;

  int ctas_per_sm = static_cast<int>(ctx->smem_optin / (c.smem_bytes + 1024));
  if (ctas_per_sm < 1) ctas_per_sm = 1;
  if (ctas_per_sm > 2 || (ctas_per_sm == 2 && c.rmax > 8)) ctas_per_sm = c.rmax > 8 ? 1 : 2;
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
  int boxes_per_copy = 1, segment_map = 0;
  {
    // Very small batches: all boxes of a stage in one copy through the segment map when d allows it,
    // else (4-byte elements) two boxes per copy, the widest a plain box can be.
    if (c.small_rows && a.d % kSegElems == 0) {
      boxes_per_copy = c.bx;
      segment_map = 1;
    } else if (c.small_rows && ve == 4) {
      boxes_per_copy = 2;
    }
    const int rc = segment_map
                       ? encode_g_segment_map(ctx, a, static_cast<int>(boxes_per_copy * box_cols / kSegElems), c.box_rows, &tmap)
                       : encode_g_tensor_map(ctx, a, boxes_per_copy * box_cols, c.box_rows, &tmap);
    if (rc != ABS_OK) return rc;
  }

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
  prm.flush_every = static_cast<int>(ctx->tuning.stats_flush_every > 0 ? ctx->tuning.stats_flush_every : 64);
  prm.ws = static_cast<double*>(ctx->workspace);
  prm.gbar_out = a.gbar_out;
  prm.flags = ctx->flags;
  prm.drop_loads = ctx->tuning.stats_fault_drop_loads ? 1 : 0;
  prm.boxes_per_copy = boxes_per_copy;
  prm.segment_map = segment_map;
  prm.guard = a.guard;
  prm.timeout_cycles = ctx->tuning.stats_timeout_cycles > 0 ? ctx->tuning.stats_timeout_cycles : kDefaultTimeoutCycles;

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
