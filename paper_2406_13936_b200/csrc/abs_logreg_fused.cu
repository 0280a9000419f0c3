// Whole communication rounds of local SGD on the logistic problem in ONE cooperative launch
// (Algorithm 2's structure with Algorithm 1's per-sample statistic once per round, Section 4.3).
//
// The round driver abs_logreg_round enqueues about four small kernels per local step; for a
// problem of a few hundred parameters every one of them is pure launch latency.  Here each
// worker is ONE thread-block cluster of P CTAs (P = 16, 8, ... - the largest that leaves all M
// clusters co-resident), every CTA keeps the worker's parameters in shared memory, and a local
// step needs nothing outside the cluster's shared memory:
//
//   phase A   every warp takes samples of the step's batch: z = <a_i, x>, r_i = sigmoid(z) - y_i,
//             and adds r_i a_i to its partial batch gradient; the CTA's partial goes into the
//             shared memory of every CTA of the cluster by one bulk copy per peer
//             (cp.async.bulk shared::cta -> shared::cluster) that signals the peer's mbarrier
//   wait      on the CTA's own mbarrier until the partials of all peers have arrived (bounded)
//   phase B   every CTA of the worker adds the P partials it received in a fixed order -> gbar
//             (Eq. batch_grad), then takes the step x <- x - lr gbar (Eq. local_sgd_alt); all
//             CTAs of a worker do the same arithmetic, so their copies of x stay bit-identical
//   last step of a round, between B and the update:
//   phase C   the CTA's samples again (from L1/L2): sum_i ||g_i - gbar||^2, e_i = <g_i - gbar, gbar>
//             (Eq. def_var, centred), partial sums per CTA in fp64, to global memory
//   grid barrier (the only one of the round: the workers meet here)
//   phase D   model averaging over the M workers (Eq. local_sgd_alt, second line), the records,
//             T per worker, b <- min(b_max, max(b, max_m T_m)) (Algorithm 1) - computed by every
//             CTA from the same numbers, so the next round's batch size needs no further barrier
//             and never leaves the device.
//
// The per-sample gradient matrix is never written.  A local step has no cluster-wide barrier:
// the received partials (and the copies' source) alternate between two buffers by step, and a
// peer can only send the partial of step h + 2 after it has received this CTA's partial of step
// h + 1, which is sent after the buffer of step h has been read.  A wait that runs out raises a
// flag, all later waits of the CTA return at once, the barriers that follow are still reached,
// and the round's records carry ABS_STATUS_TIMEOUT.  No CTA leaves while a peer may still copy
// into it: a grid barrier follows the last exchange.
// Data that crosses clusters inside the launch goes through L2 only (st.cg / ld.cg).  A round has
// one grid barrier, between the writers of S / Xpre and their readers (phase D); nothing holds a
// fast worker back from running the next round's local steps and writing its sums again while a
// slow CTA of another worker is still in phase D.  So S and Xpre exist twice and alternate by round:
// the copy read in round r is written again in round r + 2, whose writers have passed the barrier
// of round r + 1, which every CTA reaches only after its phase D of round r.  Every CTA executes the same sequence of barriers:
// the trip counts depend only on (rounds, H) and on b, which all CTAs derive from the same values.
#include <cooperative_groups.h>

#include "abs_pipeline.cuh"

namespace cg = cooperative_groups;

namespace absk {
namespace {

constexpr int kMaxWorkersFused = 64;
constexpr int kMaxDimFused = 1024;
constexpr int kMaxCtasPerWorker = 16;        // = the largest cluster (16 needs the non-portable opt-in)

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
  unsigned* flag;   // device word, zero at launch: set when a wait for the peers' partials ran out
  long long timeout_cycles;
  int drop_copies;  // test hook: the partials are not sent, so the waits run out
  double* S;        // [2][M][P][4]   V, sum e, sum e^2, N           (two copies that alternate by round:
  float* Xpre;      // [2][M][d]      parameters before the averaging  see the note on the grid barrier)
  long long* Sx;    // [2][M]         samples each worker used in the round (counter B of Alg. 1 / Alg. 2)
  long long* Bx;    // [2][M]         sizes the workers ask for after a step (per-step cadence, shared size)
  // cadence and bookkeeping (all zero / NULL: the test once per round, one size shared by all workers)
  int every_step;   // the test after every local step (Algorithm 1)
  int per_worker;   // every worker keeps its own size (Eq. test_stat); else the maximum over workers
  int sizes_per_worker;   // b_dev / b_hist hold one value per worker
  const double* eta_m;    // [M] norm-test constants per worker, or NULL
  abs_round_ctl* ctl;     // sample counter and stop rule, or NULL
  int workers_test;       // Algorithm 2 as printed: no per-sample statistics; the norm test on the workers'
                          // batch gradients of the round's last local step, after the averaging
  float* Gpre;            // [2][M][d]  those batch gradients (alternating by round like Xpre)
};

__device__ __forceinline__ void st_cluster_f64(uint32_t addr, double v) {
  asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
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
// sigmoid(z) - label.  For the labels 1 and 0 nothing is subtracted (sigmoid(z) - 1 = -sigmoid(-z)),
// so a well-fitted sample, whose residual is tiny, keeps its relative accuracy.
__device__ __forceinline__ float residual(float z, float label) {
  const float ez = expf(-fabsf(z));
  const float big = 1.f / (1.f + ez), small = ez * big;          // sigmoid(|z|), sigmoid(-|z|)
  const float p = z >= 0.f ? big : small, q = z >= 0.f ? small : big;   // sigmoid(z), sigmoid(-z)
  return label == 1.f ? -q : (label == 0.f ? p : p - label);
}

__device__ __forceinline__ void prefetch_l1(const void* p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

// KV: 16-byte column vectors per lane (slot k of a lane is vector k*32 + lane of the row).
// NW: warps per CTA (16 for narrow rows, where a warp's registers allow it: fewer samples per warp).
// EVERY: the per-step cadence of Algorithm 1 (statistics, T and the size update after every local
// step; one cluster barrier per step for the statistics' partial sums, and a grid barrier per step
// when all workers share one size).
template <int KV, int NW, bool EVERY>
__global__ void __launch_bounds__(NW * 32, 1) logreg_rounds_kernel(const FusedParams prm) {
  constexpr int NT = NW * 32;
  constexpr int U = (NW > 8 ? 8 : 16) / KV;   // samples a warp keeps in flight (8 or 16 row vectors in registers)
  cg::grid_group grid = cg::this_grid();
  extern __shared__ __align__(16) float smem_f[];
  const int d = prm.d, DV = d >> 2;
  float4* x4 = reinterpret_cast<float4*>(smem_f);              // [DV] parameters of this worker
  float4* g4 = x4 + DV;                                         // [DV] batch gradient of the step
  float4* wacc4 = g4 + DV;                                      // [NW][DV] per-warp partial sums
  float4* inbox4 = wacc4 + NW * DV;                            // [2][P][DV] the partial batch gradients of all
                                                                // CTAs of the cluster, written by their owners
  float4* outbox4 = inbox4 + 2 * prm.P * DV;                    // [2][DV] this CTA's partial, source of the copies
  __shared__ __align__(8) unsigned long long xbar[2];           // "all partials of the step have arrived"
  __shared__ unsigned abort_s;
  volatile unsigned* abort_flag = &abort_s;
  const uint32_t xbar_u32 = smem_u32(xbar);
  __shared__ double red[NW][3];
  __shared__ double N_s;
  __shared__ long long T_s[kMaxWorkersFused];
  __shared__ long long b_s;
  __shared__ __align__(16) double sbox[2][kMaxCtasPerWorker][4];   // per-step cadence: V, sum e, sum e^2, abort
                                                                    // of every CTA of the cluster, by step parity

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int M = prm.M, P = prm.P;
  const int m = blockIdx.x / P, p = blockIdx.x % P;
  const float4* A4 = reinterpret_cast<const float4*>(prm.A);
  float4* X4 = reinterpret_cast<float4*>(prm.X);
  float4* Xpre4 = reinterpret_cast<float4*>(prm.Xpre);
  const float lr = prm.lr;

  for (int j = tid; j < DV; j += NT) x4[j] = X4[static_cast<long long>(m) * DV + j];
  long long b = prm.b_dev[prm.sizes_per_worker ? m : 0];
  if (b > prm.cfg.b_max) b = prm.cfg.b_max;
  if (b < 2) b = 2;                        // the variance needs two rows
  if (blockIdx.x == 0 && tid == 0 && prm.b_hist != nullptr && !prm.sizes_per_worker) prm.b_hist[0] = b;
  abs_test_cfg cfg_m = prm.cfg;            // this worker's constants (eta_m of Eq. approx_norm_local)
  if (prm.eta_m != nullptr) cfg_m.eta = prm.eta_m[m];
  long long B = 0, n_stop = 0;             // the counter B and the N of "while B < N"; the same in every CTA
  if (prm.ctl != nullptr) {
    B = prm.ctl->samples;
    n_stop = prm.ctl->n_stop;
  }
  int rounds_done = 0;
  if (tid == 0) {
    mbar_init(xbar_u32, 1);
    mbar_init(xbar_u32 + 8u, 1);
    abort_s = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  cg::this_cluster().sync();               // every CTA's barriers exist before a peer signals them

  // Sample i of a step belongs to CTA i % P and there to warp (i / P) % NW.  The row index of the
  // warp's t-th sample is fetched by lane t % 32 ahead of the loop over the samples; for the
  // first 32 samples of a warp (all of them unless b > 32 NW P) that load is issued a whole local
  // step earlier, and the rows themselves are prefetched before the partials are exchanged.
  const long long first = p + static_cast<long long>(P) * warp;     // this warp's first sample
  const long long hop = static_cast<long long>(P) * NW;
  auto clamp_row = [&](int raw) -> long long {                       // indices outside the data are clamped
    return raw < 0 ? 0 : (raw >= prm.n ? prm.n - 1 : static_cast<long long>(raw));
  };
  auto fetch_row = [&](const int* idx_step, long long t) { return clamp_row(idx_step[first + t * hop]); };
  const int lines_per_row = (d * 4 + 127) >> 7;
  long long chunk0_row = 0;                                          // row of sample `lane` of the current step

  for (int r = 0; r < prm.rounds; ++r) {
    if (n_stop > 0 && B >= n_stop) break;                           // Alg. 1 / Alg. 2: while B < N
    long long used = 0;                                             // samples of this worker in this round
    int Pa = static_cast<int>(b < P ? b : P);                       // CTAs of a worker that have samples
    long long n_mine = b > first ? (b - first + hop - 1) / hop : 0;
    float inv_b = 1.0f / static_cast<float>(b);
    chunk0_row = lane < n_mine ? fetch_row(prm.idx + (static_cast<long long>(r) * prm.H * M + m) * prm.idx_stride, lane) : 0;
    for (int h = 0; h < prm.H; ++h) {
      const long long gstep = static_cast<long long>(r) * prm.H + h;
      const bool last = h == prm.H - 1;
      const bool workers = !EVERY && prm.workers_test != 0;         // Algorithm 2: the test is on batch gradients
      const bool test_now = EVERY || (last && !workers);            // per-sample statistics on this step's gradients
      const int* idx_m = prm.idx + (gstep * M + m) * prm.idx_stride;
      float4* part4 = inbox4 + (gstep & 1) * static_cast<long long>(P) * DV;
      if (EVERY && h > 0) {
        // the size may have grown since the last step: the step's quantities again, and the first
        // chunk of row indices now (nothing was fetched ahead for lanes that had no sample before)
        Pa = static_cast<int>(b < P ? b : P);
        n_mine = b > first ? (b - first + hop - 1) / hop : 0;
        inv_b = 1.0f / static_cast<float>(b);
        chunk0_row = lane < n_mine ? fetch_row(idx_m, lane) : 0;
      }
      used += b;

      // ---- phase A: partial batch gradient of this CTA ------------------------------------
      float4 acc[KV];
#pragma unroll
      for (int k = 0; k < KV; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      // the row indices of the NEXT local step's first chunk: the load is issued here and used after
      // this step's samples, so it costs nothing
      // (the value is not touched before the samples of this step are done: an instruction that
      // used it here would make the warp wait for the load)
      int ahead_raw = 0;
      if (!EVERY && !last && lane < n_mine) ahead_raw = (idx_m + static_cast<long long>(M) * prm.idx_stride)[first + lane * hop];
      for (long long t0 = 0; t0 < n_mine; t0 += 32) {
        const int cnt = static_cast<int>(n_mine - t0 < 32 ? n_mine - t0 : 32);
        long long my_row = chunk0_row;
        if (t0 > 0 && lane < cnt) my_row = fetch_row(idx_m, t0 + lane);
        for (int t = 0; t < cnt; t += U) {
          // U samples in flight: all their loads are issued before anything is reduced.  A slot past
          // the end repeats sample t with weight 0.
          long long rows[U];
          float lab[U], z[U];
          float4 a[U][KV];
#pragma unroll
          for (int u = 0; u < U; ++u) rows[u] = __shfl_sync(0xffffffffu, my_row, t + u < cnt ? t + u : t);
#pragma unroll
          for (int u = 0; u < U; ++u) {
            lab[u] = __ldg(prm.y + rows[u]);                                  // one address per warp
#pragma unroll
            for (int k = 0; k < KV; ++k) {
              const int j = k * 32 + lane;
              a[u][k] = j < DV ? __ldg(A4 + rows[u] * DV + j) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            z[u] = 0.f;
          }
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              const float4 xv = x4[j];
#pragma unroll
              for (int u = 0; u < U; ++u) z[u] = dot4(a[u][k], xv, z[u]);
            }
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
            for (int u = 0; u < U; ++u) z[u] += __shfl_xor_sync(0xffffffffu, z[u], off);
          }
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const float rr = t + u < cnt ? residual(z[u], lab[u]) : 0.f;
#pragma unroll
            for (int k = 0; k < KV; ++k) {
              acc[k].x = fmaf(rr, a[u][k].x, acc[k].x);
              acc[k].y = fmaf(rr, a[u][k].y, acc[k].y);
              acc[k].z = fmaf(rr, a[u][k].z, acc[k].z);
              acc[k].w = fmaf(rr, a[u][k].w, acc[k].w);
            }
          }
        }
      }
#pragma unroll
      for (int k = 0; k < KV; ++k) {
        const int j = k * 32 + lane;
        if (j < DV) wacc4[warp * DV + j] = acc[k];
      }
      if (!EVERY && !last) {
        // the next step's rows on their way into L1 while the barrier is crossed
        const long long ahead_row = clamp_row(ahead_raw);
        const int cnt0 = static_cast<int>(n_mine < 32 ? n_mine : 32);
        const int total = cnt0 * lines_per_row;
        for (int q0 = 0; q0 < total; q0 += 32) {
          const int q = q0 + lane, t = q / lines_per_row;
          const long long row = __shfl_sync(0xffffffffu, ahead_row, t < cnt0 ? t : 0);
          if (q < total) prefetch_l1(reinterpret_cast<const char*>(prm.A + row * d) + (q - t * lines_per_row) * 128);
        }
        chunk0_row = ahead_row;
      }
      __syncthreads();
      // The CTA's partial goes into its own slot of the inbox and, by one bulk copy per peer that
      // signals the peer's barrier, into the same slot of every other CTA of the cluster.  Nobody
      // waits for anybody but the data: there is no cluster-wide barrier in a step.
      const uint32_t par = static_cast<uint32_t>(gstep & 1);
      const uint32_t bytes = static_cast<uint32_t>(DV) * 16u;
      if (p < Pa) {
        for (int j = tid; j < DV; j += NT) {
          float4 s = wacc4[j];
#pragma unroll
          for (int w = 1; w < NW; ++w) {
            const float4 v = wacc4[w * DV + j];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          outbox4[par * DV + j] = s;
          part4[p * DV + j] = s;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the copies read what was just written
      }
      __syncthreads();
      // After a wait has run out this CTA takes no further part in the exchange: its barrier's
      // phase never completed, and a second arrival in the same phase is not allowed.  Its peers
      // then run into their own limits.
      if (warp == 0 && *abort_flag == 0u) {
        if (lane == 0) mbar_expect_tx(xbar_u32 + 8u * par, static_cast<uint32_t>(Pa - (p < Pa ? 1 : 0)) * bytes);
        __syncwarp();
        if (p < Pa && lane < P && lane != p && !prm.drop_copies)
          bulk_copy_to_peer(map_to_rank(smem_u32(part4 + p * DV), static_cast<uint32_t>(lane)),
                            smem_u32(outbox4 + par * DV), bytes,
                            map_to_rank(xbar_u32 + 8u * par, static_cast<uint32_t>(lane)));
      }
      // barrier `par` is used every other step: its phase bit is bit 1 of the step count
      mbar_wait(xbar_u32 + 8u * par, static_cast<uint32_t>((gstep >> 1) & 1), abort_flag, prm.timeout_cycles);

      // ---- phase B: batch gradient of the worker; the step unless statistics come first -----
      // The P partials are split over thread groups (group q takes partials q, q + groups, ...),
      // then the groups' sums are added in group order.
      {
        const int groups = NT / DV >= NW ? NW : (NT / DV > 0 ? NT / DV : 1);   // wacc4 has NW rows
        const int grp = tid / DV, j = tid - grp * DV;
        if (grp < groups) {
          float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
          for (int q = grp; q < Pa; q += groups) {
            const float4 v = part4[q * DV + j];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          wacc4[grp * DV + j] = s;
        }
        __syncthreads();
        for (int jj = tid; jj < DV; jj += NT) {
          float4 s = wacc4[jj];
          for (int q = 1; q < groups; ++q) {
            const float4 v = wacc4[q * DV + jj];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          s.x *= inv_b; s.y *= inv_b; s.z *= inv_b; s.w *= inv_b;
          g4[jj] = s;
          if (!test_now) {
            float4 xv = x4[jj];
            xv.x = fmaf(-lr, s.x, xv.x); xv.y = fmaf(-lr, s.y, xv.y);
            xv.z = fmaf(-lr, s.z, xv.z); xv.w = fmaf(-lr, s.w, xv.w);
            x4[jj] = xv;
          }
        }
        __syncthreads();
      }
      if (!test_now && !(last && workers)) continue;

      if (last && workers) {
        // ---- Algorithm 2: the step is taken; publish the parameters and the batch gradient -----------
        float4* Gpre4 = reinterpret_cast<float4*>(prm.Gpre);
        if (p == 0) {
          for (int j = tid; j < DV; j += NT) {
            __stcg(Xpre4 + (static_cast<long long>(r & 1) * M + m) * DV + j, x4[j]);
            __stcg(Gpre4 + (static_cast<long long>(r & 1) * M + m) * DV + j, g4[j]);
          }
          if (tid == 0 && prm.ctl != nullptr) __stcg(prm.Sx + static_cast<long long>(r & 1) * M + m, used);
        }
      } else {
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
        long long my_row = chunk0_row;
        if (t0 > 0 && lane < cnt) my_row = fetch_row(idx_m, t0 + lane);
        for (int t = 0; t < cnt; t += U) {
          long long rows[U];
          float lab[U], z[U], s1[U], s2[U];
          float4 a[U][KV];
#pragma unroll
          for (int u = 0; u < U; ++u) rows[u] = __shfl_sync(0xffffffffu, my_row, t + u < cnt ? t + u : t);
#pragma unroll
          for (int u = 0; u < U; ++u) {
            lab[u] = __ldg(prm.y + rows[u]);
#pragma unroll
            for (int k = 0; k < KV; ++k) {
              const int j = k * 32 + lane;
              a[u][k] = j < DV ? __ldg(A4 + rows[u] * DV + j) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            z[u] = s1[u] = s2[u] = 0.f;
          }
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              const float4 xv = x4[j];
#pragma unroll
              for (int u = 0; u < U; ++u) z[u] = dot4(a[u][k], xv, z[u]);
            }
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
            for (int u = 0; u < U; ++u) z[u] += __shfl_xor_sync(0xffffffffu, z[u], off);
          }
#pragma unroll
          for (int u = 0; u < U; ++u) z[u] = residual(z[u], lab[u]);           // from here on z holds r_i
#pragma unroll
          for (int k = 0; k < KV; ++k) {
            const int j = k * 32 + lane;
            if (j < DV) {
              const float4 gv = g4[j];
#pragma unroll
              for (int u = 0; u < U; ++u) {
                const float tx = fmaf(z[u], a[u][k].x, -gv.x), ty = fmaf(z[u], a[u][k].y, -gv.y);
                const float tz = fmaf(z[u], a[u][k].z, -gv.z), tw = fmaf(z[u], a[u][k].w, -gv.w);
                s1[u] = fmaf(tx, tx, s1[u]); s1[u] = fmaf(ty, ty, s1[u]);
                s1[u] = fmaf(tz, tz, s1[u]); s1[u] = fmaf(tw, tw, s1[u]);
                s2[u] = fmaf(tx, gv.x, s2[u]); s2[u] = fmaf(ty, gv.y, s2[u]);
                s2[u] = fmaf(tz, gv.z, s2[u]); s2[u] = fmaf(tw, gv.w, s2[u]);
              }
            }
          }
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
              s1[u] += __shfl_xor_sync(0xffffffffu, s1[u], off);
              s2[u] += __shfl_xor_sync(0xffffffffu, s2[u], off);
            }
          }
#pragma unroll
          for (int u = 0; u < U; ++u) {
            if (t + u < cnt) {
              V += static_cast<double>(s1[u]);
              se += static_cast<double>(s2[u]);
              see += static_cast<double>(s2[u]) * static_cast<double>(s2[u]);
            }
          }
        }
      }
      if (lane == 0) {
        red[warp][0] = V;
        red[warp][1] = se;
        red[warp][2] = see;
      }
      __syncthreads();
      if (EVERY) {
        // ---- per-step cadence: the cluster's sums, this worker's record, T and the size update ----
        // Every CTA puts its three partial sums (and whether one of its waits ran out) into its slot
        // of every CTA of the cluster; the cluster barrier makes them visible; every CTA then adds
        // the P slots in slot order, so all of them take the same decision.  The slots alternate by
        // step: a peer writes step h + 2 only after the barrier of step h + 1, which this CTA reaches
        // after it has read the slots of step h.
        const int par2 = static_cast<int>(gstep & 1);
        if (tid < P) {
          double a0 = 0.0, a1 = 0.0, a2 = 0.0;
          for (int w = 0; w < NW; ++w) {
            a0 += red[w][0];
            a1 += red[w][1];
            a2 += red[w][2];
          }
          const uint32_t slot = map_to_rank(smem_u32(&sbox[par2][p][0]), static_cast<uint32_t>(tid));
          st_cluster_f64(slot, a0);
          st_cluster_f64(slot + 8u, a1);
          st_cluster_f64(slot + 16u, a2);
          st_cluster_f64(slot + 24u, abort_s != 0u ? 1.0 : 0.0);
        }
        cluster_barrier();
        if (tid == 0) {
          double V = 0.0, se = 0.0, see = 0.0, ab = 0.0;
          for (int q = 0; q < P; ++q) {
            V += sbox[par2][q][0];
            se += sbox[par2][q][1];
            see += sbox[par2][q][2];
            ab += sbox[par2][q][3];
          }
          const bool timed_out = ab != 0.0;
          if (timed_out && p == 0) atomicOr(prm.flag, 1u);
          const abs_stats rec = record_from_sums(V, N_s, se, see, b, timed_out);
          const long long T = test_size_from_record(rec, cfg_m);
          long long want = T > b ? T : b;                             // Alg. 1: b <- max{T, b}
          want = want < prm.cfg.b_max ? want : prm.cfg.b_max;
          if (p == 0) {
            const long long slot = gstep * M + m;
            prm.stats[slot] = rec;
            if (prm.T_out != nullptr) prm.T_out[slot] = T;
            if (prm.b_hist != nullptr) prm.b_hist[slot] = b;          // the size this step ran with
            if (!prm.per_worker) __stcg(prm.Bx + static_cast<long long>(par2) * M + m, want);
          }
          b_s = want;
        }
        // the step that was held back
        for (int j = tid; j < DV; j += NT) {
          const float4 s = g4[j];
          float4 xv = x4[j];
          xv.x = fmaf(-lr, s.x, xv.x); xv.y = fmaf(-lr, s.y, xv.y);
          xv.z = fmaf(-lr, s.z, xv.z); xv.w = fmaf(-lr, s.w, xv.w);
          x4[j] = xv;
          if (last && p == 0) __stcg(Xpre4 + (static_cast<long long>(r & 1) * M + m) * DV + j, xv);
        }
        if (!prm.per_worker) {
          // one size for all workers: the maximum of what they ask for (display below Eq. test_stat),
          // taken after every step, which costs a grid barrier per step
          grid.sync();
          if (tid == 0) {
            long long best = 0;
            for (int w = 0; w < M; ++w) {
              const long long v = __ldcg(prm.Bx + static_cast<long long>(par2) * M + w);
              best = v > best ? v : best;
            }
            b_s = best;
          }
        }
        __syncthreads();
        b = b_s;
        if (!last) continue;
        if (tid == 0 && p == 0 && prm.ctl != nullptr) __stcg(prm.Sx + static_cast<long long>(r & 1) * M + m, used);
      } else {
        if (tid == 0) {
          // CTAs without samples contribute zeros, so that a reader need not know how many CTAs of
          // another worker (whose size may differ) were active
          double a0 = 0.0, a1 = 0.0, a2 = 0.0;
          for (int w = 0; w < NW; ++w) {
            a0 += red[w][0];
            a1 += red[w][1];
            a2 += red[w][2];
          }
          double* dst = prm.S + ((static_cast<long long>(r & 1) * M + m) * P + p) * 4;
          __stcg(dst + 0, a0);
          __stcg(dst + 1, a1);
          __stcg(dst + 2, a2);
          __stcg(dst + 3, N_s);
          if (p == 0) {
            if (prm.ctl != nullptr) __stcg(prm.Sx + static_cast<long long>(r & 1) * M + m, used);
            if (prm.per_worker) __stcg(prm.Bx + static_cast<long long>(r & 1) * M + m, b);
          }
        }
        // the step that was held back, and this worker's parameters for the averaging
        for (int j = tid; j < DV; j += NT) {
          const float4 s = g4[j];
          float4 xv = x4[j];
          xv.x = fmaf(-lr, s.x, xv.x); xv.y = fmaf(-lr, s.y, xv.y);
          xv.z = fmaf(-lr, s.z, xv.z); xv.w = fmaf(-lr, s.w, xv.w);
          x4[j] = xv;
          if (p == 0) __stcg(Xpre4 + (static_cast<long long>(r & 1) * M + m) * DV + j, xv);
        }
      }
      }   // per-sample statistics
      if (tid == 0 && abort_s != 0u) atomicOr(prm.flag, 1u);
      grid.sync();
      const bool timed_out = __ldcg(prm.flag) != 0u;

      // ---- phase D: averaging, records, next batch size ---------------------------------------
      // The loads of this phase come from L2 and nothing else is left to overlap them with, so
      // they are spread over the threads and issued together: the records by one warp per worker
      // (lane q reads the sums of CTA q; the shuffle tree adds them in a fixed order), the
      // parameters by thread groups that split the workers and are added in group order.
      if (workers) {
        // The rows are the M workers' batch gradients (Eq. test_stat_actual): gbar = mean_m g^m,
        // V = sum_m ||g^m - gbar||^2, N = ||gbar||^2, by every CTA from the same numbers in the same order.
        const float4* Gpre4 = reinterpret_cast<const float4*>(prm.Gpre) + static_cast<long long>(r & 1) * M * DV;
        const float inv_M = 1.0f / static_cast<float>(M);
        double v_loc = 0.0, n_loc = 0.0;
        for (int jj = tid; jj < DV; jj += NT) {
          float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int w = 0; w < M; ++w) {
            const float4 v = __ldcg(Gpre4 + static_cast<long long>(w) * DV + jj);
            mean.x += v.x; mean.y += v.y; mean.z += v.z; mean.w += v.w;
          }
          mean.x *= inv_M; mean.y *= inv_M; mean.z *= inv_M; mean.w *= inv_M;
          float vs = 0.f;
          for (int w = 0; w < M; ++w) {
            const float4 v = __ldcg(Gpre4 + static_cast<long long>(w) * DV + jj);
            const float dx = v.x - mean.x, dy = v.y - mean.y, dz = v.z - mean.z, dw = v.w - mean.w;
            vs = fmaf(dx, dx, vs); vs = fmaf(dy, dy, vs); vs = fmaf(dz, dz, vs); vs = fmaf(dw, dw, vs);
          }
          v_loc += static_cast<double>(vs);
          n_loc += static_cast<double>(fmaf(mean.x, mean.x, fmaf(mean.y, mean.y, fmaf(mean.z, mean.z, mean.w * mean.w))));
        }
        v_loc = warp_sum_dd(v_loc);
        n_loc = warp_sum_dd(n_loc);
        if (lane == 0) {
          red[warp][0] = v_loc;
          red[warp][1] = n_loc;
        }
        __syncthreads();
        if (tid == 0) {
          double V = 0.0, N = 0.0;
          for (int w = 0; w < NW; ++w) {
            V += red[w][0];
            N += red[w][1];
          }
          abs_stats rec = record_from_sums(V, N, 0.0, 0.0, M, timed_out);
          rec.status |= ABS_STATUS_NORM_ONLY;            // the per-worker inner products are not formed
          abs_test_cfg c = prm.cfg;
          c.kind = ABS_TEST_NORM;
          c.row_weight = static_cast<double>(b);          // a row is the mean of b samples (Section 4.3)
          c.divisor = static_cast<double>(M);             // Eq. test_stat_actual
          const long long T = test_size_from_record(rec, c);
          for (int w = 0; w < M; ++w) T_s[w] = T;
          if (blockIdx.x == 0) {
            prm.stats[static_cast<long long>(r) * M] = rec;
            if (prm.T_out != nullptr) prm.T_out[static_cast<long long>(r) * M] = T;
            if (prm.b_hist != nullptr && prm.sizes_per_worker)
              for (int w = 0; w < M; ++w) prm.b_hist[static_cast<long long>(r) * M + w] = b;
          }
        }
      } else if (!EVERY) {
        for (int w = warp; w < M; w += NW) {
          double a0 = 0.0, a1 = 0.0, a2 = 0.0, nn = 0.0;
          if (lane < P) {
            const double* src = prm.S + ((static_cast<long long>(r & 1) * M + w) * P + lane) * 4;
            a0 = __ldcg(src + 0);
            a1 = __ldcg(src + 1);
            a2 = __ldcg(src + 2);
            nn = __ldcg(src + 3);
          }
          a0 = warp_sum_dd(a0);
          a1 = warp_sum_dd(a1);
          a2 = warp_sum_dd(a2);
          nn = __shfl_sync(0xffffffffu, nn, 0);
          if (lane == 0) {
            const long long b_w = prm.per_worker ? __ldcg(prm.Bx + static_cast<long long>(r & 1) * M + w) : b;
            abs_test_cfg cfg_w = prm.cfg;
            if (prm.eta_m != nullptr) cfg_w.eta = prm.eta_m[w];
            const abs_stats rec = record_from_sums(a0, nn, a1, a2, b_w, timed_out);
            const long long T = test_size_from_record(rec, cfg_w);
            T_s[w] = T;
            if (blockIdx.x == 0) {
              prm.stats[static_cast<long long>(r) * M + w] = rec;
              if (prm.T_out != nullptr) prm.T_out[static_cast<long long>(r) * M + w] = T;
              if (prm.b_hist != nullptr && prm.sizes_per_worker) prm.b_hist[static_cast<long long>(r) * M + w] = b_w;
            }
          }
        }
      }
      {
        const float inv_M = 1.0f / static_cast<float>(M);
        const int groups = NT / DV >= NW ? NW : (NT / DV > 0 ? NT / DV : 1);
        const int grp = tid / DV, j = tid - grp * DV;
        if (grp < groups) {
          float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
          for (int w = grp; w < M; w += groups) {
            const float4 v = __ldcg(Xpre4 + (static_cast<long long>(r & 1) * M + w) * DV + j);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          wacc4[grp * DV + j] = s;
        }
        __syncthreads();
        for (int jj = tid; jj < DV; jj += NT) {
          float4 s = wacc4[jj];
          for (int q = 1; q < groups; ++q) {
            const float4 v = wacc4[q * DV + jj];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
          }
          s.x *= inv_M; s.y *= inv_M; s.z *= inv_M; s.w *= inv_M;
          x4[jj] = s;
        }
      }
      __syncthreads();
      if (tid == 0) {
        long long best = b;
        if (!EVERY) {
          if (prm.per_worker) {
            best = T_s[m] > best ? T_s[m] : best;                    // Eq. test_stat: the worker's own T
          } else {
            for (int w = 0; w < M; ++w) best = T_s[w] > best ? T_s[w] : best;
          }
          best = best < prm.cfg.b_max ? best : prm.cfg.b_max;
        }
        b_s = best;
        if (blockIdx.x == 0 && prm.b_hist != nullptr && !prm.sizes_per_worker) prm.b_hist[r + 1] = best;
        // the round's term of the sample counter: sum_m sum_h b^m_{k,h} (Alg. 1), which is H M b_k when
        // the size is shared and constant over the round (Alg. 2)
        long long tot = 0;
        if (prm.ctl != nullptr)
          for (int w = 0; w < M; ++w) tot += __ldcg(prm.Sx + static_cast<long long>(r & 1) * M + w);
        T_s[0] = tot;       // T_s is free again: every thread is past the loop above (barrier before this block)
      }
      __syncthreads();
      b = b_s;
      B += T_s[0];
      ++rounds_done;
      __syncthreads();      // T_s[0] is overwritten by the next round's records
    }
  }
  // the parameters after the last round that ran (x^m_{K,0}: the output of Alg. 1 / Alg. 2 is replica 1)
  if (p == 0 && rounds_done > 0)
    for (int jj = tid; jj < DV; jj += NT) X4[static_cast<long long>(m) * DV + jj] = x4[jj];
  if (tid == 0 && p == 0 && (prm.sizes_per_worker || m == 0)) prm.b_dev[prm.sizes_per_worker ? m : 0] = b;
  if (blockIdx.x == 0 && tid == 0 && prm.ctl != nullptr) {
    prm.ctl->samples = B;
    prm.ctl->rounds += rounds_done;
  }
}

using KernelFn = void (*)(const FusedParams);
struct KernelChoice {
  KernelFn fn;
  int warps;
};
KernelChoice pick_kernel(int DV, bool every) {
  if (every) {
    if (DV <= 32) return {logreg_rounds_kernel<1, 16, true>, 16};
    if (DV <= 64) return {logreg_rounds_kernel<2, 16, true>, 16};
    if (DV <= 128) return {logreg_rounds_kernel<4, 8, true>, 8};
    return {logreg_rounds_kernel<8, 8, true>, 8};
  }
  if (DV <= 32) return {logreg_rounds_kernel<1, 16, false>, 16};
  if (DV <= 64) return {logreg_rounds_kernel<2, 16, false>, 16};
  if (DV <= 128) return {logreg_rounds_kernel<4, 8, false>, 8};
  return {logreg_rounds_kernel<8, 8, false>, 8};
}

}  // namespace
}  // namespace absk

using namespace absk;

extern "C" int abs_logreg_rounds_fused_opts(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                            const int* idx, long long idx_stride, int rounds, float* X, int M, int H,
                                            float lr, const abs_test_cfg* cfg, const abs_round_opts* opts,
                                            abs_stats* stats, long long* T_out, long long* b_hist, long long* b_dev,
                                            void* stream) {
  if (ctx == nullptr) return ABS_ERR_INVALID_ARG;
  if (A == nullptr || y == nullptr || idx == nullptr || X == nullptr || cfg == nullptr || stats == nullptr ||
      b_dev == nullptr)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "null pointer argument");
  if (n < 1 || d < 1 || M < 1 || H < 1 || rounds < 1)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need n, d, M, H, rounds >= 1");
  const bool workers_test = cfg->kind == ABS_TEST_NORM_WORKERS;
  if (workers_test && (M < 2 || (opts != nullptr && (opts->test_every_step != 0 || opts->per_worker != 0))))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "the test on the workers' batch gradients (Algorithm 2) needs M >= 2, runs once "
                                               "per round and gives all workers one size");
  if (cfg->kind != ABS_TEST_NORM && cfg->kind != ABS_TEST_AUG_INNER_PRODUCT && !workers_test)
    return set_error(ctx, ABS_ERR_INVALID_ARG, "unknown test kind %d", cfg->kind);
  if (cfg->b_max < 2 || !(cfg->row_weight > 0.0) || !(cfg->divisor > 0.0))
    return set_error(ctx, ABS_ERR_INVALID_ARG, "need b_max >= 2, row_weight > 0, divisor > 0");
  if (cfg->kind != ABS_TEST_AUG_INNER_PRODUCT ? !(cfg->eta > 0.0 || (opts != nullptr && opts->eta_m != nullptr))
                                 : !(cfg->theta > 0.0 && cfg->nu > 0.0))
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

  const bool every = opts != nullptr && opts->test_every_step != 0;
  const int DV = static_cast<int>(d / 4);
  const KernelChoice choice = pick_kernel(DV, every);
  KernelFn kernel = choice.fn;
  const size_t smem_fixed = static_cast<size_t>(2 + choice.warps + 2) * d * sizeof(float);   // + 2 P d floats of inboxes

  // One cluster per worker: the largest cluster size that leaves all M clusters co-resident.
  cudaLaunchConfig_t lc = {};
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeClusterDimension;
  attrs[1].id = cudaLaunchAttributeCooperative;
  attrs[1].val.cooperative = 1;
  lc.blockDim = dim3(static_cast<unsigned>(choice.warps * 32));
  lc.stream = static_cast<cudaStream_t>(stream);
  lc.attrs = attrs;
  lc.numAttrs = 2;
  ABS_CUDA_TRY(ctx, cudaFuncSetAttribute(reinterpret_cast<const void*>(kernel),
                                         cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
  int P = 0;
  for (int cand = kMaxCtasPerWorker; cand >= 1 && P == 0; cand >>= 1) {
    const size_t smem = smem_fixed + 2ull * cand * d * sizeof(float);
    if (smem + 2048 > ctx->smem_optin) continue;      // 2 KiB for the static shared variables
    // (always the most this kernel can have, so that calls from other contexts or threads never lower it)
    ABS_CUDA_TRY(ctx, cudaFuncSetAttribute(reinterpret_cast<const void*>(kernel),
                                           cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           static_cast<int>(ctx->smem_optin - 2048)));
    lc.dynamicSmemBytes = smem;
    attrs[0].val.clusterDim.x = static_cast<unsigned>(cand);
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    lc.gridDim = dim3(static_cast<unsigned>(M * cand));
    int clusters = 0;
    const cudaError_t e = cudaOccupancyMaxActiveClusters(&clusters, reinterpret_cast<const void*>(kernel), &lc);
    if (e != cudaSuccess) {
      cudaGetLastError();        // this cluster size is not available on the device: try the next
      continue;
    }
    if (clusters >= M) P = cand;
  }
  if (P == 0) return set_error(ctx, ABS_ERR_UNSUPPORTED, "%d workers do not fit a co-resident grid", M);

  // scratch in the context's workspace: statistics partials, pre-average parameters, sample counts, sizes
  const size_t S_bytes = 2 * static_cast<size_t>(M) * P * 4 * sizeof(double);       // two copies each,
  const size_t xpre_bytes = 2 * static_cast<size_t>(M) * d * sizeof(float);          // alternating by round
  const size_t cnt_bytes = 2 * static_cast<size_t>(M) * sizeof(long long);
  if (S_bytes + 2 * xpre_bytes + 2 * cnt_bytes > ctx->workspace_bytes)      // Xpre and Gpre have the same size
    return set_error(ctx, ABS_ERR_WORKSPACE, "workspace of %zu bytes is too small (%zu needed)", ctx->workspace_bytes,
                     S_bytes + 2 * xpre_bytes + 2 * cnt_bytes);
  unsigned char* ws = static_cast<unsigned char*>(ctx->workspace);

  FusedParams prm;
  prm.A = A; prm.y = y; prm.n = n; prm.d = static_cast<int>(d);
  prm.idx = idx; prm.idx_stride = idx_stride;
  prm.rounds = rounds; prm.M = M; prm.H = H; prm.P = P;
  prm.lr = lr; prm.cfg = *cfg;
  prm.X = X; prm.stats = stats; prm.T_out = T_out; prm.b_hist = b_hist; prm.b_dev = b_dev;
  prm.flag = ctx->flags + 2;
  prm.drop_copies = ctx->tuning.stats_fault_drop_loads != 0 ? 1 : 0;
  prm.timeout_cycles = ctx->tuning.stats_timeout_cycles > 0 ? ctx->tuning.stats_timeout_cycles : kDefaultTimeoutCycles;
  ABS_CUDA_TRY(ctx, cudaMemsetAsync(prm.flag, 0, sizeof(unsigned), static_cast<cudaStream_t>(stream)));
  prm.S = reinterpret_cast<double*>(ws);
  prm.Sx = reinterpret_cast<long long*>(ws + S_bytes);
  prm.Bx = reinterpret_cast<long long*>(ws + S_bytes + cnt_bytes);
  prm.Xpre = reinterpret_cast<float*>(ws + S_bytes + 2 * cnt_bytes);
  prm.every_step = every ? 1 : 0;
  prm.per_worker = opts != nullptr && opts->per_worker != 0 ? 1 : 0;
  prm.sizes_per_worker = opts != nullptr ? 1 : 0;
  prm.eta_m = opts != nullptr ? opts->eta_m : nullptr;
  prm.ctl = opts != nullptr ? opts->ctl : nullptr;
  prm.workers_test = workers_test ? 1 : 0;
  prm.Gpre = reinterpret_cast<float*>(ws + S_bytes + 2 * cnt_bytes + xpre_bytes);
  ABS_CUDA_TRY(ctx, cudaLaunchKernelEx(&lc, kernel, prm));
  return ABS_OK;
}

extern "C" int abs_logreg_rounds_fused(abs_ctx* ctx, const float* A, const float* y, long long n, long long d,
                                       const int* idx, long long idx_stride, int rounds, float* X, int M, int H,
                                       float lr, const abs_test_cfg* cfg, abs_stats* stats, long long* T_out,
                                       long long* b_hist, long long* b_dev, void* stream) {
  return abs_logreg_rounds_fused_opts(ctx, A, y, n, d, idx, idx_stride, rounds, X, M, H, lr, cfg, nullptr, stats,
                                      T_out, b_hist, b_dev, stream);
}
