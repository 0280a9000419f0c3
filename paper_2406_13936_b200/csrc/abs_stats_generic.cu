// Alignment-free statistics kernel and the fp64 finalisation of the batch-size test.
//
// The generic kernel takes any base address, any strides and any b.  A CTA owns a
// strip of 256 columns at a time: sweep A sums the strip's columns over all rows
// (Eq. batch_grad), sweep B re-reads the strip (from L2 when it is still there) and
// forms the centred sums of Eq. def_var.  Loads are scalar and coalesced across a
// warp.  It reads G twice and is the fallback of the tiled kernel, not the fast path.
#include <cuda_bf16.h>

#include "abs_internal.cuh"

namespace absk {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kStrip = 256;
constexpr int kChain = 16;            // rows a thread adds up in fp32 before the sum moves on

__device__ __forceinline__ float load_elt(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_elt(const __nv_bfloat16* p) {
  return __uint_as_float(static_cast<unsigned>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// E_SMEM: the per-row sums e_r live in (dynamic) shared memory until the end, which is possible up
// to kGenericSmemRows rows; beyond, they are updated in the CTA's workspace record strip by strip.
constexpr int kGenericSmemRows = 4096;

template <typename T, bool E_SMEM>
__global__ void __launch_bounds__(kThreads)
abs_stats_generic_kernel(const T* __restrict__ G, long long b, long long d, long long row_stride,
                         long long worker_stride, long long n_strips, int P, double* __restrict__ ws,
                         float* __restrict__ gbar_out) {
  __shared__ float colpart[kWarps][kStrip];
  __shared__ float gbar_s[kStrip];
  __shared__ double red[2 * kWarps];
  extern __shared__ double e_rows[];            // [b] when E_SMEM

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = blockIdx.y, p = blockIdx.x;
  const T* Gm = G + static_cast<long long>(m) * worker_stride;
  double* out = ws + (static_cast<size_t>(m) * P + p) * (static_cast<size_t>(b) + 2);
  double* e_acc = E_SMEM ? e_rows : out;        // one warp owns a row: a single writer either way
  const float inv_b = 1.0f / static_cast<float>(b);
  pdl_launch_dependents();      // the finalisation kernel may be scheduled; it waits for this grid to complete

  for (long long r = tid; r < b; r += kThreads) e_acc[r] = 0.0;
  __syncthreads();

  double vacc = 0.0, nacc = 0.0;
  for (long long it = p; it < n_strips; it += P) {
    const long long j0 = it * kStrip;
    // sweep A: column sums, rows split over the warps
    // (no fp32 sum takes more than kChain terms in a row: a thread's rows are summed in groups, and
    // the groups' sums are added to a second accumulator, so that thousands of rows of one sign or
    // one large entry among tiny ones do not wear the low bits away)
    float cs[kStrip / 32], cg[kStrip / 32];
#pragma unroll
    for (int c = 0; c < kStrip / 32; ++c) cs[c] = cg[c] = 0.f;
    int chain = 0;
    for (long long r = warp; r < b; r += kWarps) {
      const T* row = Gm + r * row_stride + j0;
#pragma unroll
      for (int c = 0; c < kStrip / 32; ++c) {
        const long long col = j0 + c * 32 + lane;
        if (col < d) cg[c] += load_elt(row + c * 32 + lane);
      }
      if (++chain == kChain) {
        chain = 0;
#pragma unroll
        for (int c = 0; c < kStrip / 32; ++c) {
          cs[c] += cg[c];
          cg[c] = 0.f;
        }
      }
    }
#pragma unroll
    for (int c = 0; c < kStrip / 32; ++c) cs[c] += cg[c];
#pragma unroll
    for (int c = 0; c < kStrip / 32; ++c) colpart[warp][c * 32 + lane] = cs[c];
    __syncthreads();
    {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) s += colpart[w][tid];
      const float g = s * inv_b;
      gbar_s[tid] = g;
      if (j0 + tid < d) {
        nacc += static_cast<double>(g * g);
        if (gbar_out != nullptr) gbar_out[static_cast<long long>(m) * d + j0 + tid] = g;
      }
    }
    __syncthreads();
    // sweep B: centred sums; one warp owns a row, so e_r has a single writer
    float gl[kStrip / 32];
#pragma unroll
    for (int c = 0; c < kStrip / 32; ++c) gl[c] = gbar_s[c * 32 + lane];
    float vl = 0.f;
    chain = 0;
    for (long long r = warp; r < b; r += kWarps) {
      const T* row = Gm + r * row_stride + j0;
      float el = 0.f;
#pragma unroll
      for (int c = 0; c < kStrip / 32; ++c) {
        const long long col = j0 + c * 32 + lane;
        if (col < d) {
          const float dlt = load_elt(row + c * 32 + lane) - gl[c];
          vl = fmaf(dlt, dlt, vl);
          el = fmaf(dlt, gl[c], el);
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) el += __shfl_xor_sync(0xffffffffu, el, off);
      if (lane == 0) e_acc[r] += static_cast<double>(el);
      if (++chain == kChain) {
        chain = 0;
        vacc += static_cast<double>(vl);
        vl = 0.f;
      }
    }
    vacc += static_cast<double>(vl);
    __syncthreads();
  }

  vacc = warp_sum_d(vacc);
  nacc = warp_sum_d(nacc);
  if (lane == 0) {
    red[warp] = vacc;
    red[kWarps + warp] = nacc;
  }
  __syncthreads();
  if (E_SMEM)
    for (long long r = tid; r < b; r += kThreads) out[r] = e_rows[r];
  if (tid == 0) {
    double vs = 0.0, ns = 0.0;
    for (int w = 0; w < kWarps; ++w) {
      vs += red[w];
      ns += red[kWarps + w];
    }
    out[b] = vs;
    out[b + 1] = ns;
  }
}

// Folds the P partial records of every worker in a fixed order and writes abs_stats.  Grid
// (M, nb): the rows of a worker are split over nb CTAs (one when b < 128), because a single CTA
// that reads P x b sums takes long for large batches.  CTA y sums e_r
// over the records for its rows and leaves sum e, sum e^2 (CTA 0 also V and N) in the first words
// of its own rows of record 0 - rows no other CTA reads; the worker's last CTA to arrive (ticket
// counter) adds the nb pairs in the order of y and writes the record, so the result does not
// depend on which CTA that is.
constexpr int kFinalThreads = 1024;
constexpr int kFinalMaxSplit = 16;
constexpr int kFinalRowsPerCta = 64;      // at least this many rows per CTA (>= 4: the words it borrows)

__global__ void __launch_bounds__(kFinalThreads)
abs_stats_finalize_kernel(double* ws, long long b, int P, unsigned* __restrict__ flags,
                          unsigned* __restrict__ tickets, abs_stats* __restrict__ stats_out, const Recheck rk) {
  __shared__ double red[4][kFinalThreads / 32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = blockIdx.x, y = blockIdx.y, nb = gridDim.y;
  const size_t rec = static_cast<size_t>(b) + 2;
  double* base = ws + static_cast<size_t>(m) * P * rec;
  const long long rows_per = (b + nb - 1) / nb;
  const long long r_begin = y * rows_per;
  const long long r_end = r_begin + rows_per < b ? r_begin + rows_per : b;
  pdl_wait();                    // the statistics kernel's partial records
  pdl_launch_dependents();
  // the finalisation of a recomputation that was not needed: the records stand as they are
  if (rk.second && *reinterpret_cast<volatile unsigned*>(rk.redo) == 0u) return;
  // Loads whose values are only needed at the end are issued here, so that they are in flight
  // while the rows are summed: the time-out flag, and the first V and N of every thread.
  unsigned timeout_word = 0u;
  if (tid == 0) timeout_word = *reinterpret_cast<volatile unsigned*>(flags);
  double vn = 0.0, nn = 0.0;
  if (y == 0 && tid < P) {
    vn = base[tid * rec + b];
    nn = base[tid * rec + b + 1];
  }

  // Rows are spread over the threads; when the CTA has fewer than 1024 rows several threads share
  // a row and split the P records between them (record p goes to thread group p mod tpr), then
  // the groups' sums are added in group order: the order of additions is fixed, the loads run in
  // parallel.
  __shared__ double esum[kFinalThreads];
  int rb = 1;
  while (rb < kFinalThreads && rb < r_end - r_begin) rb <<= 1;   // rows handled per pass (power of two)
  const int tpr = kFinalThreads / rb;                     // threads per row
  const int col = tid & (rb - 1), grp = tid / rb;
  double se = 0.0, see = 0.0;
  for (long long r0 = r_begin; r0 < r_end; r0 += rb) {
    const long long r = r0 + col;
    double e = 0.0;
    if (r < r_end) {
      // sixteen loads are issued before the first sum needs one (a load per iteration would cost a
      // round trip to L2 each; so would a scalar tail, hence the predicated last batch: adding 0.0
      // changes nothing); the sums are still taken in the order of p
      for (int p0 = grp; p0 < P; p0 += 16 * tpr) {
        double v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int p = p0 + u * tpr;
          v[u] = p < P ? base[static_cast<size_t>(p) * rec + r] : 0.0;
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) e += v[u];
      }
    }
    esum[tid] = e;
    __syncthreads();
    if (grp == 0 && r < r_end) {
      double tot = 0.0;
      for (int g2 = 0; g2 < tpr; ++g2) tot += esum[g2 * rb + col];
      se += tot;
      see += tot * tot;
    }
    __syncthreads();
  }
  // V and N (CTA 0 of the worker): thread t takes the records p = t, t + 1024, ...
  if (y == 0) {
    for (int p = tid + kFinalThreads; p < P; p += kFinalThreads) {
      vn += base[p * rec + b];
      nn += base[p * rec + b + 1];
    }
  }
  const double a0 = warp_sum_d(se), a1 = warp_sum_d(see), a2 = warp_sum_d(vn), a3 = warp_sum_d(nn);
  if (lane == 0) {
    red[0][warp] = a0;
    red[1][warp] = a1;
    red[2][warp] = a2;
    red[3][warp] = a3;
  }
  __syncthreads();
  if (warp != 0) return;
  // one value per warp and 32 warps: the first warp adds them with the same shuffle tree
  double s_e = warp_sum_d(red[0][lane]), s_ee = warp_sum_d(red[1][lane]);
  double V = warp_sum_d(red[2][lane]), N = warp_sum_d(red[3][lane]);
  if (tid == 0) {
    if (nb > 1) {
      // every read of this CTA's rows is done (the barriers above): borrow their first words
      double* mine = base + r_begin;
      __stcg(mine + 0, s_e);
      __stcg(mine + 1, s_ee);
      if (y == 0) {
        __stcg(mine + 2, V);
        __stcg(mine + 3, N);
      }
      __threadfence();
      if (atomicAdd(tickets + m, 1u) != static_cast<unsigned>(nb - 1)) return;   // not the worker's last CTA
      __threadfence();
      tickets[m] = 0u;                                   // for the next call
      double pe[kFinalMaxSplit], pee[kFinalMaxSplit];
#pragma unroll
      for (int y2 = 0; y2 < kFinalMaxSplit; ++y2) {       // all loads first, then the sums in CTA order
        pe[y2] = y2 < nb ? __ldcg(base + y2 * rows_per + 0) : 0.0;
        pee[y2] = y2 < nb ? __ldcg(base + y2 * rows_per + 1) : 0.0;
      }
      V = __ldcg(base + 2);
      N = __ldcg(base + 3);
      s_e = 0.0;
      s_ee = 0.0;
#pragma unroll
      for (int y2 = 0; y2 < kFinalMaxSplit; ++y2) {
        s_e += pe[y2];
        s_ee += pee[y2];
      }
    }
    const bool timed_out = timeout_word != 0u;
    // The last worker to get here clears the time-out flag (flags[0]) and the arrival counter
    // (flags[1]) for the next call, which saves a memset per call.
    abs_stats rec = record_from_sums(V, N, s_e, s_ee, b, timed_out);
    if (rk.second) rec.recomputed = 1u;
    if (!rk.second && rk.redo != nullptr && (rec.status & (ABS_STATUS_NONFINITE | ABS_STATUS_TIMEOUT)) == 0u) {
      const double bd = static_cast<double>(b);
      if (bd * N > rk.max_kv * (bd - 1.0) * rec.var_norm || N * N > rk.max_kip * rk.max_kip * rec.var_ip)
        atomicOr(rk.redo, 1u);
    }
    __threadfence();
    if (atomicAdd(flags + 1, 1u) == gridDim.x - 1) {
      flags[0] = 0u;
      flags[1] = 0u;
      if (rk.second) *rk.redo = 0u;
    }
    stats_out[m] = rec;
  }
}

}  // namespace

int launch_stats_generic(abs_ctx* ctx, const StatsLaunch& a, int* P_out) {
  const long long n_strips = (a.d + kStrip - 1) / kStrip;
  long long P = (static_cast<long long>(ctx->sm_count) * 4) / a.M;
  if (P < 1) P = 1;
  if (P > n_strips) P = n_strips;
  if (P > 65535) P = 65535;
  if (a.M > 65535) return set_error(ctx, ABS_ERR_UNSUPPORTED, "M = %d exceeds 65535", a.M);
  // fit the workspace: fewer CTAs per worker if b is very large
  const size_t rec = (static_cast<size_t>(a.b) + 2) * sizeof(double);
  while (P > 1 && static_cast<size_t>(a.M) * P * rec > ctx->workspace_bytes) P = (P + 1) / 2;
  if (static_cast<size_t>(a.M) * P * rec > ctx->workspace_bytes)
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_test_stats needs %zu workspace bytes, context has %zu",
                     static_cast<size_t>(a.M) * P * rec, ctx->workspace_bytes);
  const dim3 grid(static_cast<unsigned>(P), static_cast<unsigned>(a.M));
  double* ws = static_cast<double*>(ctx->workspace);
  const bool e_smem = a.b <= kGenericSmemRows;
  const size_t smem = e_smem ? static_cast<size_t>(a.b) * sizeof(double) : 0;
#define ABS_GENERIC_LAUNCH(T, E)                                                                                 \
  abs_stats_generic_kernel<T, E><<<grid, kThreads, smem, a.stream>>>(static_cast<const T*>(a.G), a.b, a.d,       \
                                                                     a.row_stride, a.worker_stride, n_strips,    \
                                                                     static_cast<int>(P), ws, a.gbar_out)
  if (a.dtype == ABS_F32) {
    if (e_smem) ABS_GENERIC_LAUNCH(float, true); else ABS_GENERIC_LAUNCH(float, false);
  } else {
    if (e_smem) ABS_GENERIC_LAUNCH(__nv_bfloat16, true); else ABS_GENERIC_LAUNCH(__nv_bfloat16, false);
  }
#undef ABS_GENERIC_LAUNCH
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  *P_out = static_cast<int>(P);
  return ABS_OK;
}

int launch_stats_finalize(abs_ctx* ctx, const StatsLaunch& a, int P, const Recheck& rk) {
  // the rows of a worker are split over several CTAs when the context has a ticket word per worker
  long long nb = a.M <= ctx->ticket_slots ? a.b / kFinalRowsPerCta : 1;
  nb = nb < 1 ? 1 : (nb > kFinalMaxSplit ? kFinalMaxSplit : nb);
  while (nb > 1 && (nb - 1) * ((a.b + nb - 1) / nb) + 4 > a.b) --nb;     // the last CTA keeps at least 4 rows
  ABS_CUDA_TRY(ctx, launch_dependent(abs_stats_finalize_kernel, dim3(a.M, static_cast<unsigned>(nb)),
                                     dim3(kFinalThreads), 0, a.stream, static_cast<double*>(ctx->workspace), a.b, P,
                                     ctx->flags, ctx->flags + kFlagWords, a.stats_out, rk));
  return ABS_OK;
}

}  // namespace absk
