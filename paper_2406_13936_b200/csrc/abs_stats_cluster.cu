// Cluster variant of the single-pass statistics kernel for large batches (256 < b <= 4096).
//
// A column strip with all b rows does not fit one SM's shared memory at a row width that the
// memory system likes (>= 256 bytes), and a CTA that touches a thousand far-apart rows per tile
// runs into address-translation misses.  So the rows are split over a thread-block cluster of
// C = 2, 4, 8 or 16 CTAs: CTA `rank` holds rows [rank*RC, rank*RC + RC) of the strip,
// RC = ceil(b/C) <= 256.  Each CTA sums its rows' columns; the per-CTA column sums (lpr*VE
// floats) are shipped to every peer with one bulk shared-to-shared copy that signals the peer's
// mbarrier; after that every CTA knows gbar for the strip and runs the centred sweep on its rows
// (Eq. batch_grad, Eq. def_var as in the tiled kernel).  G is still read exactly once.
//
// The loop is software pipelined: a step moves the rows of tile i from shared memory into
// registers (so the tile buffer goes straight back to the loader), sends the column sums round
// the cluster, and then finishes tile i-1 from a second register set, whose sums have had a
// whole step to arrive.  Four exchange buffers / barriers are in flight.  There is no separate
// loader warp: after the CTA-wide barrier that follows the register load, thread 0 re-arms the
// buffer and issues the next TMA load into it.  All waits are bounded.
#include "abs_pipeline.cuh"

namespace absk {
namespace {

constexpr int kCW = 8;                         // warps
constexpr int kThreadsC = kCW * 32;
constexpr int kMaxCluster = 16;                // 16 needs the non-portable cluster size opt-in
constexpr int kDepth = 4;                      // column-sum exchange buffers in flight (power of two)

struct ClusterParams {
  long long b, d;
  int rows_per_cta;      // RC
  int lpr_log2;
  int stages;
  int box_rows, n_row_boxes;
  unsigned stage_bytes;  // rows_pad * lpr * 16
  long long col_begin;   // first column of this launch's share of the row (a multiple of the strip width)
  long long n_iters;     // column strips of that share, per worker
  int n_clusters;        // clusters per worker in this launch
  int rec_base;          // first partial record of this launch (a second launch appends its records)
  int rec_total;         // partial records per worker over all launches
  int wait_primary;      // this launch runs beside the one before it in the stream: wait for that one before exit
  int flush_every;
  double* ws;
  float* gbar_out;
  unsigned* flags;
  long long timeout_cycles;
  int drop_loads;        // fault injection for the bounded waits: no tile load is issued
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// RMAX: rows per thread and register set, ceil(rows per CTA / row groups) (two sets alternate);
// FULL: every thread of every CTA owns exactly RMAX rows, so nothing is predicated.  Otherwise
// a thread owns n_rows_mine <= RMAX rows -- the cluster's last CTA holds b - (C-1)*RC rows, which
// can be several row groups short of RC -- and every row index is checked against that count.
template <typename T, int RMAX, bool FULL>
__global__ void __launch_bounds__(kThreadsC, 1)
abs_stats_cluster_kernel(const __grid_constant__ CUtensorMap tmap, const ClusterParams prm) {
  constexpr int VE = Vec<T>::VE;
  extern __shared__ __align__(128) unsigned char smem_raw[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = blockIdx.y;
  const int C = static_cast<int>(cluster_nctarank());
  const int rank = static_cast<int>(cluster_ctarank());
  const int cl = blockIdx.x / C;                 // cluster index within the worker
  const int b = static_cast<int>(prm.b);
  const int RC = prm.rows_per_cta;
  const int row0 = rank * RC;
  const int b_loc = max(0, min(RC, b - row0));   // rows this CTA owns
  const int S = prm.stages;
  const int lpr = 1 << prm.lpr_log2;
  const unsigned row_bytes = static_cast<unsigned>(lpr) * 16u;
  const int cols = lpr * VE;                     // columns of a strip

  unsigned char* stage_mem = smem_raw;
  float* part = reinterpret_cast<float*>(stage_mem + static_cast<size_t>(S) * prm.stage_bytes);   // [2][8][cols]
  float* xsum = part + 2 * kCW * cols;                                                             // [kDepth][16][cols]
  double* e_acc = reinterpret_cast<double*>(xsum + kDepth * kMaxCluster * cols);                   // [RC]
  double* red = e_acc + RC;                                                                        // [16]
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(red + 2 * kCW);                 // full[S] x[kDepth]
  volatile unsigned* abort_flag = reinterpret_cast<volatile unsigned*>(bars + S + kDepth);

  const uint32_t stage_u32 = smem_u32(stage_mem);
  const uint32_t full_u32 = smem_u32(bars);
  const uint32_t xbar_u32 = smem_u32(bars + S);
  const uint32_t xsum_u32 = smem_u32(xsum);

  const long long n_mine = (prm.n_iters > cl) ? (prm.n_iters - cl + prm.n_clusters - 1) / prm.n_clusters : 0;

  // Loads tile i of this cluster (rows of this CTA) into its ring buffer; thread 0 only.  After a
  // wait has run out nothing more is issued, so the loads that were issued are a prefix 0..issued-1.
  long long issued = 0;
  auto issue_load = [&](long long i) {
    if (prm.drop_loads || *abort_flag) return;     // drop_loads: test hook, the waits must run out, not hang
    ++issued;
    const int s = static_cast<int>(i % S);
    const uint32_t full = full_u32 + 8u * s;
    mbar_expect_tx(full, prm.stage_bytes);
    const long long x = prm.col_begin + (cl + i * prm.n_clusters) * cols;
    const uint32_t dst0 = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes;
    for (int rb = 0; rb < prm.n_row_boxes; ++rb)
      tma_load_3d(dst0 + static_cast<uint32_t>(rb * prm.box_rows) * row_bytes, &tmap, static_cast<int>(x),
                  row0 + rb * prm.box_rows, m, full);
  };

  if (tid == 0) {
    for (int s = 0; s < S; ++s) mbar_init(full_u32 + 8u * s, 1);
    for (int q = 0; q < kDepth; ++q) mbar_init(xbar_u32 + 8u * q, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i < RC; i += kThreadsC) e_acc[i] = 0.0;
  cluster_sync_all();      // every CTA's barriers exist before anybody signals them
  pdl_launch_dependents(); // the finalisation kernel may be scheduled; it waits for this grid to complete
  if (tid == 0)
    for (long long i = 0; i < S && i < n_mine; ++i) issue_load(i);

  const int sub = lane >> prm.lpr_log2;          // sub-row-group within the warp
  const int cv = lane & (lpr - 1);               // 16-byte column vector within the strip row
  const int subs = 32 >> prm.lpr_log2;
  const int RG = kCW * subs;                     // row groups
  const int rg = warp * subs + sub;
  const int n_rows_mine = (b_loc > rg) ? (b_loc - rg + RG - 1) / RG : 0;
  const unsigned row_step = static_cast<unsigned>(RG) * row_bytes;
  const uint32_t my_off = static_cast<uint32_t>(rg) * row_bytes + static_cast<uint32_t>(cv) * 16u;
  const float inv_b = 1.0f / static_cast<float>(b);
  const bool writes_mean = (rank == 0 && rg == 0);

  double vacc = 0.0, nacc = 0.0;
  float e[RMAX];
#pragma unroll
  for (int k = 0; k < RMAX; ++k) e[k] = 0.f;
  int since_flush = 0;

  uint4 va[RMAX], vb[RMAX];
  auto step = [&](uint4 (&cur)[RMAX], uint4 (&prev)[RMAX], const long long i) {
    if (i < n_mine) {
      // ---- first half: tile i into registers, its column sums round the cluster ----
      const int s = static_cast<int>(i % S);
      mbar_wait(full_u32 + 8u * s, static_cast<uint32_t>((i / S) & 1), abort_flag, prm.timeout_cycles);
      const uint32_t base = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + my_off;
      const uint32_t base0 = stage_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + static_cast<uint32_t>(cv) * 16u;
      float cs[VE];
#pragma unroll
      for (int j = 0; j < VE; ++j) cs[j] = 0.f;
#pragma unroll
      for (int k = 0; k < RMAX; ++k) {
        // rows past the batch: safe address, zeroed by a select (no branch around the loads)
        const bool ok = FULL || k < n_rows_mine;
        uint4 u = lds128(ok ? base + static_cast<uint32_t>(k) * row_step : base0);
        if (!ok) u = make_uint4(0u, 0u, 0u, 0u);
        cur[k] = u;
        float x[VE];
        Vec<T>::unpack(u, x);
#pragma unroll
        for (int j = 0; j < VE; ++j) cs[j] += x[j];
      }
      for (int off = lpr; off < 32; off <<= 1) {
#pragma unroll
        for (int j = 0; j < VE; ++j) cs[j] += __shfl_xor_sync(0xffffffffu, cs[j], off);
      }
      float* buf = part + static_cast<size_t>(i & 1) * (kCW * cols);
      if (sub == 0) {
        smem_store_vec<VE>(buf + warp * cols + cv * VE, cs);
      }
      __syncthreads();     // partial sums visible; every thread has its rows in registers
      if (tid == 0 && i + S < n_mine) issue_load(i + S);     // the buffer is free: refill it
      // Warp 0 folds the 8 warps' sums (one lane per 16-byte column vector) into this CTA's own
      // slot, arms its own barrier for the bytes the peers will send, and lane `peer` ships the
      // slot to that peer with one bulk copy that signals the peer's barrier.
      if (warp == 0) {
        const int q = static_cast<int>(i & (kDepth - 1));
        float* mine = xsum + (q * kMaxCluster + rank) * cols;
        if (lane < lpr) {
          float tot[VE];
#pragma unroll
          for (int j = 0; j < VE; ++j) tot[j] = 0.f;
          for (int w = 0; w < kCW; ++w) {
            smem_add_vec<VE>(buf + w * cols + lane * VE, tot);
          }
          smem_store_vec<VE>(mine + lane * VE, tot);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads what was just written
        }
        __syncwarp();
        const uint32_t bytes = static_cast<uint32_t>(cols) * 4u;
        if (lane == 0) mbar_expect_tx(xbar_u32 + 8u * q, static_cast<uint32_t>(C - 1) * bytes);
        if (lane < C && lane != rank) {
          const uint32_t slot = xsum_u32 + static_cast<uint32_t>((q * kMaxCluster + rank) * cols * 4);
          bulk_copy_to_peer(map_to_rank(slot, static_cast<uint32_t>(lane)), slot, bytes,
                            map_to_rank(xbar_u32 + 8u * q, static_cast<uint32_t>(lane)));
        }
      }
    }
    if (i >= 1) {
      // ---- second half: finish tile i-1 from the other register set ----
      const long long t = i - 1;
      const int q = static_cast<int>(t & (kDepth - 1));
      mbar_wait(xbar_u32 + 8u * q, static_cast<uint32_t>((t / kDepth) & 1), abort_flag, prm.timeout_cycles);
      float g[VE];
#pragma unroll
      for (int j = 0; j < VE; ++j) g[j] = 0.f;
      for (int peer = 0; peer < C; ++peer) {      // fixed order: the same mean in every CTA
        const float* src = xsum + (q * kMaxCluster + peer) * cols + cv * VE;
        smem_add_vec<VE>(src, g);
      }
#pragma unroll
      for (int j = 0; j < VE; ++j) g[j] *= inv_b;

      if (writes_mean) {
        float nl = 0.f;
#pragma unroll
        for (int j = 0; j < VE; ++j) nl = fmaf(g[j], g[j], nl);
        nacc += static_cast<double>(nl);
        if (prm.gbar_out != nullptr) {
          const long long col = prm.col_begin + ((cl + t * prm.n_clusters) * static_cast<long long>(lpr) + cv) * VE;
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

      float vl[VE];
#pragma unroll
      for (int j = 0; j < VE; ++j) vl[j] = 0.f;
#pragma unroll
      for (int k = 0; k < RMAX; ++k) {
        const bool ok = FULL || k < n_rows_mine;
        float x[VE];
        Vec<T>::unpack(prev[k], x);
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
      if (++since_flush >= prm.flush_every || i == n_mine) {
        since_flush = 0;
#pragma unroll
        for (int k = 0; k < RMAX; ++k) {
          float ek = e[k];
          for (int off = 1; off < lpr; off <<= 1) ek += __shfl_xor_sync(0xffffffffu, ek, off);
          if (cv == 0 && (FULL || k < n_rows_mine)) e_acc[rg + k * RG] += static_cast<double>(ek);
          e[k] = 0.f;
        }
      }
    }
  };
  for (long long i = 0; i <= n_mine; i += 2) {
    step(va, vb, i);
    if (i + 1 <= n_mine) step(vb, va, i + 1);
  }

  // ------------------------------ CTA epilogue ------------------------------
  vacc = warp_sum(vacc);
  nacc = warp_sum(nacc);
  if (lane == 0) {
    red[warp] = vacc;
    red[kCW + warp] = nacc;
  }
  __syncthreads();
  double* out = prm.ws + (static_cast<size_t>(m) * prm.rec_total + prm.rec_base + blockIdx.x) * (static_cast<size_t>(b) + 2);
  for (int r = tid; r < b; r += kThreadsC) {
    const int loc = r - row0;
    out[r] = (loc >= 0 && loc < b_loc) ? e_acc[loc] : 0.0;     // rows of other CTAs: their records carry them
  }
  if (tid == 0) {
    double vs = 0.0, ns = 0.0;
    for (int w = 0; w < kCW; ++w) {
      vs += red[w];
      ns += red[kCW + w];
    }
    out[b] = vs;
    out[b + 1] = ns;
    if (*abort_flag) atomicOr(prm.flags, 1u);
    // Leave no copy in flight into this CTA's shared memory: every armed phase of the tile ring and
    // of the exchange barriers must have completed before the CTA may exit.  Normally all of them
    // have been waited for already; after a wait that ran out these are bounded waits of their own.
    volatile unsigned ignore = 0u;
    for (int s = 0; s < S && s < issued; ++s)
      mbar_wait(full_u32 + 8u * s, static_cast<uint32_t>(((issued - 1 - s) / S) & 1), &ignore, prm.timeout_cycles);
    for (int q = 0; q < kDepth && q < n_mine; ++q)
      mbar_wait(xbar_u32 + 8u * q, static_cast<uint32_t>(((n_mine - 1 - q) / kDepth) & 1), &ignore, prm.timeout_cycles);
  }
  cluster_sync_all();      // nobody leaves while a peer could still address its shared memory
  // A launch that ran beside its predecessor (on the SMs that one cannot use) must not complete before
  // it: the finalisation waits for this grid only.
  if (prm.wait_primary) pdl_wait();
}

// What one launch of the kernel covers.  n_clusters == 0 asks only how many clusters of this size
// can be resident at once (*max_clusters_out), without launching.
struct ClusterShare {
  int n_clusters = 0;
  bool beside_previous = false;   // programmatic dependent launch that starts while the launch before it runs
  int* max_clusters_out = nullptr;
};

template <typename T, int RMAX, bool FULL>
int launch_cluster_variant(abs_ctx* ctx, const CUtensorMap& tmap, ClusterParams prm, const StatsLaunch& a, int C,
                           size_t smem, const ClusterShare& share) {
  auto kern = abs_stats_cluster_kernel<T, RMAX, FULL>;
  ABS_CUDA_TRY(ctx, ensure_dynamic_smem(ctx, kern, smem));
  if (C > 8 && cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    cudaGetLastError();
    return ABS_ERR_UNSUPPORTED;
  }
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(C);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3(kThreadsC);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = a.stream;
  cfg.attrs = attr;
  cfg.numAttrs = share.beside_previous ? 2 : 1;
  if (share.n_clusters == 0) {
    const int slot = ctx->fn_cache.slot(reinterpret_cast<const void*>(kern));
    if (slot >= 0 && ctx->fn_cache.cluster_size[slot] == C && ctx->fn_cache.cluster_smem[slot] == smem) {
      *share.max_clusters_out = ctx->fn_cache.max_clusters[slot];     // asked before: the answer cannot change
      return ABS_OK;
    }
    cfg.gridDim = dim3(static_cast<unsigned>(C), 1, 1);
    cfg.numAttrs = 1;
    int max_clusters = 0;
    const cudaError_t occ = cudaOccupancyMaxActiveClusters(&max_clusters, kern, &cfg);
    if (occ != cudaSuccess || max_clusters < 1) {
      cudaGetLastError();
      set_error(ctx, ABS_ERR_UNSUPPORTED, "a cluster of %d CTAs cannot be scheduled (%s, %d clusters)", C,
                cudaGetErrorString(occ), max_clusters);
      return ABS_ERR_UNSUPPORTED;
    }
    if (slot >= 0) {
      ctx->fn_cache.cluster_size[slot] = C;
      ctx->fn_cache.cluster_smem[slot] = smem;
      ctx->fn_cache.max_clusters[slot] = max_clusters;
    }
    *share.max_clusters_out = max_clusters;
    return ABS_OK;
  }
  cfg.gridDim = dim3(static_cast<unsigned>(share.n_clusters * C), static_cast<unsigned>(a.M), 1);
  ABS_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, kern, tmap, prm));
  return ABS_OK;
}

// One attempt with a given cluster size; ABS_ERR_UNSUPPORTED if that size cannot be used.
struct ClusterGeom {
  int RC, lpr_log2, RG, rmax, n_row_boxes, box_rows, stages, cols;
  unsigned stage_bytes;
  size_t smem;
  bool full;
};

// Tile geometry of a cluster of C CTAs for b rows; false if that size cannot be used.
bool cluster_geometry(const Tuning& t, size_t smem_optin, int es, long long b, int C, ClusterGeom* g) {
  const int ve = 16 / es;
  g->RC = static_cast<int>((b + C - 1) / C);
  if (g->RC > 512) return false;
  g->lpr_log2 = g->RC <= 256 ? 4 : 3;                       // 256-byte rows; 128-byte for 257..512 rows
  const int lpr = 1 << g->lpr_log2;
  const int subs = 32 / lpr;
  g->RG = kCW * subs;
  g->rmax = (g->RC + g->RG - 1) / g->RG;                    // rows per thread, <= 16
  g->n_row_boxes = (g->RC + 255) / 256;
  g->box_rows = (g->RC + g->n_row_boxes - 1) / g->n_row_boxes;
  const int rows_pad = g->box_rows * g->n_row_boxes;
  g->stage_bytes = static_cast<unsigned>(rows_pad) * lpr * 16u;
  g->cols = lpr * ve;
  const size_t extras = static_cast<size_t>(2 * kCW * g->cols + kDepth * kMaxCluster * g->cols) * 4 +
                        static_cast<size_t>(g->RC) * 8 + 2 * kCW * 8 + kDepth * 8 + 16 + 128;
  g->stages = static_cast<int>(t.stats_stages > 0 ? t.stats_stages : 4);
  while (g->stages > 2 && g->stages * static_cast<size_t>(g->stage_bytes) + extras + g->stages * 8 > smem_optin)
    --g->stages;
  g->smem = g->stages * static_cast<size_t>(g->stage_bytes) + extras + g->stages * 8;
  if (g->smem > smem_optin) return false;
  g->full = (b % C == 0) && (g->RC % g->RG == 0) && (g->rmax == 8 || g->rmax == 16);
  return true;
}

// Up to 2048 rows: at most 256 rows of 256 bytes per CTA.  Beyond: clusters of 8 with up to 512
// rows of 128 bytes (a cluster of 16 leaves too many SMs without a cluster; tried: 3.9 vs 4.6 TB/s
// at b = 4096).  Direct st.shared::cluster stores with cluster-scope fences instead of the bulk
// copies were also tried: 40 % slower.
int preferred_cluster_size(const Tuning& t, long long b) {
  const int want_rows = t.stats_cluster_rows > 0 ? static_cast<int>(t.stats_cluster_rows) : (b > 2048 ? 512 : 256);
  // the fewest CTAs that leave each at most want_rows rows: any size from 2 to 8 (not only powers of
  // two), because fuller tiles matter more than how evenly the clusters tile the GPU
  long long C = (b + want_rows - 1) / want_rows;
  if (C < 2) C = 2;
  if (C > kMaxCluster) C = kMaxCluster;
  return static_cast<int>(C);
}

// One launch (or one occupancy query) of the variant that fits the geometry.
int cluster_dispatch(abs_ctx* ctx, const StatsLaunch& a, int C, const ClusterGeom& geo, ClusterParams prm,
                     const ClusterShare& share) {
  CUtensorMap tmap;
  int rc = encode_g_tensor_map(ctx, a, geo.cols, geo.box_rows, &tmap);
  if (rc != ABS_OK) return rc;
  prm.b = a.b;
  prm.d = a.d;
  prm.rows_per_cta = geo.RC;
  prm.lpr_log2 = geo.lpr_log2;
  prm.stages = geo.stages;
  prm.box_rows = geo.box_rows;
  prm.n_row_boxes = geo.n_row_boxes;
  prm.stage_bytes = geo.stage_bytes;
  prm.flush_every = static_cast<int>(ctx->tuning.stats_flush_every > 0 ? ctx->tuning.stats_flush_every : 64);
  prm.ws = static_cast<double*>(ctx->workspace);
  prm.gbar_out = a.gbar_out;
  prm.flags = ctx->flags;
  prm.timeout_cycles = ctx->tuning.stats_timeout_cycles > 0 ? ctx->tuning.stats_timeout_cycles : kDefaultTimeoutCycles;
  prm.drop_loads = ctx->tuning.stats_fault_drop_loads ? 1 : 0;
  prm.n_clusters = share.n_clusters;
  prm.wait_primary = share.beside_previous ? 1 : 0;
  const int rmax = geo.rmax;
  const size_t smem = geo.smem;
  const bool full = geo.full;
#define ABS_CLUSTER_CASE(T, R) \
  case R: return launch_cluster_variant<T, R, false>(ctx, tmap, prm, a, C, smem, share);
#define ABS_CLUSTER_DISPATCH(T)                                                                        \
  if (full) {                                                                                          \
    return rmax == 8 ? launch_cluster_variant<T, 8, true>(ctx, tmap, prm, a, C, smem, share)           \
                     : launch_cluster_variant<T, 16, true>(ctx, tmap, prm, a, C, smem, share);         \
  }                                                                                                    \
  switch (rmax) {                                                                                      \
    ABS_CLUSTER_CASE(T, 1) ABS_CLUSTER_CASE(T, 2) ABS_CLUSTER_CASE(T, 3) ABS_CLUSTER_CASE(T, 4)        \
    ABS_CLUSTER_CASE(T, 5) ABS_CLUSTER_CASE(T, 6) ABS_CLUSTER_CASE(T, 7) ABS_CLUSTER_CASE(T, 8)        \
    ABS_CLUSTER_CASE(T, 9) ABS_CLUSTER_CASE(T, 10) ABS_CLUSTER_CASE(T, 11) ABS_CLUSTER_CASE(T, 12)     \
    ABS_CLUSTER_CASE(T, 13) ABS_CLUSTER_CASE(T, 14) ABS_CLUSTER_CASE(T, 15)                            \
    default: return launch_cluster_variant<T, 16, false>(ctx, tmap, prm, a, C, smem, share);           \
  }
  if (a.dtype == ABS_F32) { ABS_CLUSTER_DISPATCH(float) }
  ABS_CLUSTER_DISPATCH(__nv_bfloat16)
#undef ABS_CLUSTER_DISPATCH
#undef ABS_CLUSTER_CASE
}

// One attempt with a given cluster size; ABS_ERR_UNSUPPORTED if that size cannot be used.
//
// Clusters of C CTAs cannot be placed on every SM (a cluster lives inside one GPC, and a GPC's SM
// count need not be a multiple of C: 33 clusters of 4 occupy 132 of 148 SMs).  The SMs that are left
// over come in pairs, so a second launch of the same kernel with clusters of half the size (twice the
// rows per CTA, half the row width) takes a share of the columns of its own: it is enqueued as a
// programmatic dependent of the first launch, starts as soon as that one is resident, finds only
// the left-over SMs free, and waits for the first launch before it completes.  Its partial records
// follow the first launch's in the workspace, and the finalisation folds them all.
int try_cluster_size(abs_ctx* ctx, const StatsLaunch& a, int C, int* P_out) {
  const int es = a.dtype == ABS_F32 ? 4 : 2;
  ClusterGeom geo;
  if (!cluster_geometry(ctx->tuning, ctx->smem_optin, es, a.b, C, &geo)) return ABS_ERR_UNSUPPORTED;
  int max_clusters = 0;
  ClusterShare query;
  query.max_clusters_out = &max_clusters;
  int rc = cluster_dispatch(ctx, a, C, geo, ClusterParams(), query);
  if (rc != ABS_OK) return rc;

  const long long strips = (a.d + geo.cols - 1) / geo.cols;
  long long n1 = ctx->tuning.stats_ctas_per_worker > 0 ? ctx->tuning.stats_ctas_per_worker
                                                       : static_cast<long long>(max_clusters) / a.M;
  if (n1 < 1) n1 = 1;
  if (n1 > strips) n1 = strips;
  if (n1 * C > 65535) n1 = 65535 / C;

  // the second launch: clusters of two on the SMs the first cannot use
  ClusterGeom geo2;
  long long n2 = 0, cols_second = 0;
  const long long idle = ctx->sm_count - n1 * a.M * C;
  // Only pairs are known to fit what clusters of three or four leave over; clusters of four beside
  // clusters of eight were tried (b = 2048) and mostly ran after the first launch instead of beside
  // it: 6.7 -> 8.8 ms.
  const int C2 = 2;
  if ((C == 3 || C == 4) && !ctx->tuning.stats_no_secondary && ctx->tuning.stats_ctas_per_worker == 0 && idle >= C2 &&
      n1 * a.M == (static_cast<long long>(max_clusters) / a.M) * a.M &&
      cluster_geometry(ctx->tuning, ctx->smem_optin, es, a.b, C2, &geo2)) {
    n2 = (idle / C2) / a.M;
    // its share of the columns: in proportion to its SMs, each counted at `pct` per cent of an SM of
    // the first launch (measured: the two finish together at about 100, and every per cent beyond
    // that costs a per cent of the whole call, so the default stays a little below); at least 64
    // strips per cluster
    // (beside clusters of three the pairs were worth 60: b = 768, 6.09 -> 6.39 TB/s, and 95 lost; rows
    // further apart than about 64 MB: a CTA of the second launch touches 512 of them per tile and
    // misses the TLB more often than one of the first with its 256; measured at a 102 MB row stride the
    // two finish together at 80)
    const long long row_bytes = a.row_stride * es;
    const long long pct = ctx->tuning.stats_secondary_pct > 0 ? ctx->tuning.stats_secondary_pct
                                                               : (C == 3 ? 60 : (row_bytes > (64ll << 20) ? 80 : 95));
    const double w2 = static_cast<double>(n2 * C2) * pct / 100.0;
    cols_second = static_cast<long long>(static_cast<double>(a.d) * w2 / (static_cast<double>(n1 * C) + w2));
    if (n2 < 1 || cols_second < 64 * n2 * geo2.cols) n2 = 0;
  }
  long long cols_first = a.d;
  if (n2 > 0) {
    cols_first = (a.d - cols_second) / geo.cols * geo.cols;      // whole strips of the first launch
    if (cols_first <= 0 || cols_first >= a.d) n2 = 0, cols_first = a.d;
  }
  const long long strips1 = (cols_first + geo.cols - 1) / geo.cols;
  if (n1 > strips1) n1 = strips1;
  const long long strips2 = n2 > 0 ? (a.d - cols_first + geo2.cols - 1) / geo2.cols : 0;
  const long long records = n1 * C + n2 * C2;
  const size_t need = static_cast<size_t>(a.M) * records * (a.b + 2) * sizeof(double);
  if (need > ctx->workspace_bytes)
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_test_stats needs %zu workspace bytes, context has %zu", need,
                     ctx->workspace_bytes);

  ClusterParams prm;
  prm.col_begin = 0;
  prm.n_iters = strips1;
  prm.rec_base = 0;
  prm.rec_total = static_cast<int>(records);
  ClusterShare first;
  first.n_clusters = static_cast<int>(n1);
  rc = cluster_dispatch(ctx, a, C, geo, prm, first);
  if (rc != ABS_OK) return rc;
  if (n2 > 0) {
    prm.col_begin = cols_first;
    prm.n_iters = strips2;
    prm.rec_base = static_cast<int>(n1 * C);
    ClusterShare second;
    second.n_clusters = static_cast<int>(n2);
    second.beside_previous = true;
    rc = cluster_dispatch(ctx, a, C2, geo2, prm, second);
    if (rc != ABS_OK) return rc;
  }
  *P_out = static_cast<int>(records);
  return ABS_OK;
}

}  // namespace

// Takes the call when 256 < b <= 4096 and the tiled loads can address G.  Prefers the cluster
// size that leaves each CTA at most 256 rows (64 KiB tiles of 256-byte rows); falls back to
// smaller clusters when the larger one cannot be scheduled.
int launch_stats_cluster(abs_ctx* ctx, const StatsLaunch& a, int* P_out) {
  if (a.b <= 256 || a.b > kMaxFastRows || !tma_addressable(a)) return ABS_ERR_UNSUPPORTED;
  for (int C = preferred_cluster_size(ctx->tuning, a.b); C >= 2; --C) {
    const int rc = try_cluster_size(ctx, a, C, P_out);
    if (rc != ABS_ERR_UNSUPPORTED) return rc;
  }
  return ABS_ERR_UNSUPPORTED;
}

int plan_stats_cluster(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, int cluster_size,
                       abs_stats_plan* out) {
  if (b <= 256 || b > kMaxFastRows) return ABS_ERR_UNSUPPORTED;
  const int C = cluster_size > 0 ? cluster_size : preferred_cluster_size(t, b);
  ClusterGeom g;
  if (!cluster_geometry(t, smem_optin, dtype == ABS_F32 ? 4 : 2, b, C, &g)) return ABS_ERR_UNSUPPORTED;
  memset(out, 0, sizeof(*out));
  out->route = 1;
  out->lanes_per_row = 1 << g.lpr_log2;
  out->warps_per_box = kCW;
  out->boxes_per_stage = 1;
  out->stages = g.stages;
  out->box_rows = g.box_rows;
  out->row_boxes = g.n_row_boxes;
  out->rows_per_thread = g.rmax;
  out->keep_in_registers = 1;
  out->full = g.full ? 1 : 0;
  out->cluster_size = C;
  out->rows_per_cta = g.RC;
  out->stage_bytes = g.stage_bytes;
  out->smem_bytes = g.smem;
  return ABS_OK;
}

}  // namespace absk
