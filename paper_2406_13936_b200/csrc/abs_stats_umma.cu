// Gram-matrix statistics kernel for bf16 rows and 32 < b <= 256 on the tcgen05 tensor cores, sm_100a.
//
// As in the small-batch Gram kernel, K = G G^T carries everything the batch-size test needs
// (Eq. batch_grad and Eq. def_var expanded):
//   N = 1^T K 1 / b^2,  c_i = (K 1)_i / b,  sum_i ||g_i - gbar||^2 = tr K - 1^T K 1 / b.
// The CUDA-core route needs about six instructions per bf16 element and stalls near 4 TB/s for
// these batch sizes; a 128 x b x 16 tcgen05.mma takes the 4 KiB it consumes off the critical path.
// Products of two bf16 values are exact in fp32; the tensor core adds them in fp32 over about
// 4096 columns in TMEM (a fold), then four warps read the accumulator back (tcgen05.ld),
// reduce each row to (K 1)_i and K_ii and add those to fp64 registers, which is where the
// cancellation in c_i - N happens.  Two accumulators alternate, so the read-back overlaps the
// next fold's MMAs.
//
// Operands: both A and B are the same shared-memory tile (K-major, 128-byte swizzle): rows of G,
// 64 columns per k-block, four k-blocks per row segment of 256 columns.  A tensor-map copy into
// that layout is limited to 128-byte box rows, which the copy engine serves at about two thirds
// of the HBM rate, so the tile is filled by four loader warps with 16-byte cp.async copies (a warp
// covers 512 contiguous bytes of one row) that apply the swizzle themselves and signal the
// stage's mbarrier through cp.async.mbarrier.arrive, so they never wait for their own copies.
//
// Measured here, an MMA of this shape costs about (128 + N) / 2 clocks whatever M and the
// arithmetic are (the operands arrive at about 64 bytes per clock), i.e. about 100 clocks per 16
// columns.  For b <= 64 that is slower than HBM delivers 16 columns, so two or three column
// segments are stacked as extra operand rows: the tile [s * ceil8(b) rows] x [256 columns] holds
// segment t in rows t * ceil8(b) ..., one MMA then covers 16 columns of every segment, and the
// diagonal blocks of its s x s block result are the segments' Gram matrices (the off-diagonal
// blocks are never read).  A k-block holds stack * ceil8(b) rows; the A descriptor always spans
// 128 rows and the B descriptor ceil16(.), so both may run into the next k-block: what they pick
// up there lands in rows / columns of the accumulator that nobody reads.
//
// 128 < b <= 256: the rows form two blocks of 128.  A tile is then 128 columns (two k-blocks, so that
// three stages still fit), and each k-step issues two MMAs: rows 0..127 against all rows
// (K00 | K01, N = ceil16(b)) and rows 128.. against rows 128.. (K11, N = ceil16(b) - 128).  K10 is
// not computed: the row sums of rows >= 128 take its part from the column sums of K01, which the
// read-back warps form with a halving butterfly of shuffles (16 per 16 columns).  Both
// accumulators of a fold take 2 ceil16(b) - 128 TMEM columns, so they alternate with a second
// pair only while ceil16(b) <= 192; above, the MMAs wait while a fold is read back, and folds are
// twice as long.
//
// Warp roles: 0-3 loaders, 4-7 accumulator read-back (warp w owns TMEM lanes 32 (w % 4) ..),
// 8 MMA issue (one elected lane) and TMEM allocation, 9-12 column means on the CUDA cores when
// gbar is wanted.  Every wait is bounded; a wait that runs out raises the CTA's abort flag, every
// role falls through its loop, TMEM is freed and the records come back flagged ABS_STATUS_TIMEOUT.
#include <cuda_bf16.h>

#include "abs_pipeline.cuh"

namespace absk {
namespace {

constexpr int kLoadWarps = 4;
constexpr int kFoldCols = 4096;       // columns added up in fp32 (TMEM) before the fold into fp64
constexpr int kMaxStagesU = 8;
constexpr int kBarsU = 2 * kMaxStagesU + 5;

struct UmmaParams {
  const __nv_bfloat16* G;
  long long b, d, row_stride, worker_stride;   // strides in elements
  int stack;              // column segments stacked as extra rows of the operand (1..3; 1 when b > 128)
  int rows_blk;           // ceil8(b): rows one segment takes in a k-block
  int nkb;                // k-blocks (64 columns each) per segment: 4, or 2 when b > 128
  int n_dim;              // N of the MMA on rows 0..127: ceil16(stack * rows_blk)
  int n1_dim;             // N of the MMA on rows 128..: n_dim - 128 (0 when b <= 128)
  int nbuf;               // accumulator sets that alternate between folds (2, or 1 when they do not fit twice)
  int buf_stride;         // TMEM columns from one accumulator set to the next
  int acc1_off;           // TMEM column of the second row block's accumulator inside a set
  int tmem_cols;          // TMEM columns allocated (a power of two)
  int stages;
  int fold_tiles;         // stages accumulated in TMEM before the fold into fp64
  unsigned kb_bytes;      // stack * rows_blk * 128
  unsigned stage_bytes;   // nkb k-blocks
  long long n_tiles;
  int P;
  double* ws;
  float* gbar_out;
  unsigned* flags;
  long long timeout_cycles;
  int drop_loads;         // fault injection for the bounded waits: the loaders issue nothing
};

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Bounded wait for barriers that are expected to stay closed for a while: sleeps between polls so
// that the waiting warps leave the issue slots to the loaders and the MMA thread.
__device__ __forceinline__ bool mbar_wait_backoff(uint32_t bar, uint32_t parity, volatile unsigned* abort_flag,
                                                  long long limit, unsigned sleep_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*abort_flag) return false;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag || clock64() - t0 > limit) {
      *abort_flag = 1u;
      return false;
    }
    __nanosleep(sleep_ns);
  }
  return true;
}
// True in exactly one lane of the (converged) warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t is_leader;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(is_leader));
  return is_leader != 0;
}
// D (fp32, TMEM) (+)= A (bf16, smem) * B^T (bf16, smem); issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive accumulator columns of this thread's TMEM lane: two loads in flight, one wait.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[2][16]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%32];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%33];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr), "r"(taddr + 16u)
      : "memory");
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    v[0][j] = __uint_as_float(r[j]);
    v[1][j] = __uint_as_float(r[16 + j]);
  }
}

// Sum over the 32 lanes of a warp of each of 16 per-lane values with a halving butterfly (16
// shuffles): afterwards every lane holds the total of value index 8 b4 + 4 b3 + 2 b2 + b1, where
// b4..b1 are bits 4..1 of its lane number (lanes 2k and 2k+1 hold the same total).
__device__ __forceinline__ float warp_sum_16_values(const float (&v)[16], int lane) {
  float w[8], x[4], y[2];
  const bool h16 = (lane & 16) != 0, h8 = (lane & 8) != 0, h4 = (lane & 4) != 0, h2 = (lane & 2) != 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) w[i] = (h16 ? v[8 + i] : v[i]) + __shfl_xor_sync(0xffffffffu, h16 ? v[i] : v[8 + i], 16);
#pragma unroll
  for (int i = 0; i < 4; ++i) x[i] = (h8 ? w[4 + i] : w[i]) + __shfl_xor_sync(0xffffffffu, h8 ? w[i] : w[4 + i], 8);
#pragma unroll
  for (int i = 0; i < 2; ++i) y[i] = (h4 ? x[2 + i] : x[i]) + __shfl_xor_sync(0xffffffffu, h4 ? x[i] : x[2 + i], 4);
  float z = (h2 ? y[1] : y[0]) + __shfl_xor_sync(0xffffffffu, h2 ? y[0] : y[1], 2);
  z += __shfl_xor_sync(0xffffffffu, z, 1);
  return z;
}

// red[] layout (doubles) in the CTA's tail of shared memory
constexpr int kRedRow = 0;        // [256] row sums per TMEM-lane owner (second row block at +128)
constexpr int kRedDiag = 256;     // [256] diagonal entries
constexpr int kRedCol = 512;      // [4][128] column sums of K01 per read-back warp
constexpr int kRedTot = 1024;     // total, trace
constexpr int kRedRs = 1026;      // [256] (K 1)_i per row of G
constexpr int kRedDg = 1282;      // [256] K_ii per row of G
constexpr int kRedDoubles = 1538;

// MB: row blocks of 128 (1: b <= 128, 2: b <= 256)
template <int MB, bool WANT_GBAR>
__global__ void __launch_bounds__(WANT_GBAR ? 416 : 288, 1)
abs_stats_umma_kernel(const UmmaParams prm) {
  extern __shared__ unsigned char smem_dyn[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m = blockIdx.y, p = blockIdx.x;
  const int b = static_cast<int>(prm.b);
  const int S = prm.stages;

  // the swizzle is a function of the address: k-blocks start on 1024-byte boundaries
  const uint32_t raw_u32 = smem_u32(smem_dyn);
  const uint32_t ring_u32 = (raw_u32 + 1023u) & ~1023u;
  unsigned char* ring = smem_dyn + (ring_u32 - raw_u32);
  // room the operand descriptors (128 * MB rows from the start of a k-block) may run into
  const uint32_t pad = (static_cast<uint32_t>(128 * MB) - prm.kb_bytes / 128u) * 128u;
  unsigned char* tail = ring + static_cast<size_t>(S) * prm.stage_bytes + pad;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tail);
  volatile unsigned* abort_flag = reinterpret_cast<volatile unsigned*>(bars + kBarsU);
  unsigned* tmem_slot = const_cast<unsigned*>(abort_flag) + 1;
  double* red = reinterpret_cast<double*>(bars + kBarsU + 1);
  const uint32_t full_u32 = smem_u32(bars);
  const uint32_t empty_u32 = full_u32 + 8u * kMaxStagesU;
  const uint32_t accfull_u32 = empty_u32 + 8u * kMaxStagesU;      // 2
  const uint32_t accempty_u32 = accfull_u32 + 16u;                // 2
  const uint32_t done_u32 = accempty_u32 + 16u;                   // 1

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(full_u32 + 8u * s, kLoadWarps * 32);
      mbar_init(empty_u32 + 8u * s, WANT_GBAR ? 5 : 1);
    }
    for (int k = 0; k < 2; ++k) {
      mbar_init(accfull_u32 + 8u * k, 1);
      mbar_init(accempty_u32 + 8u * k, 128);
    }
    mbar_init(done_u32, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const uint32_t tmem_cols = static_cast<uint32_t>(prm.tmem_cols);
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();      // the finalisation kernel may be scheduled; it waits for this grid to complete

  const long long n_mine = (prm.n_tiles > p) ? (prm.n_tiles - p + prm.P - 1) / prm.P : 0;
  const __nv_bfloat16* Gm = prm.G + static_cast<long long>(m) * prm.worker_stride;
  const int seg_cols = prm.nkb * 64;                                // columns of one row segment
  const long long tile_cols = static_cast<long long>(prm.stack) * seg_cols;
  double row_sum[MB], row_diag[MB], col_sum[MB == 2 ? 8 : 1];
#pragma unroll
  for (int k = 0; k < MB; ++k) row_sum[k] = row_diag[k] = 0.0;
#pragma unroll
  for (int k = 0; k < (MB == 2 ? 8 : 1); ++k) col_sum[k] = 0.0;

  if (warp < kLoadWarps) {
    // ---- loaders: a row segment is nkb * 8 chunks of 16 bytes; a warp instruction covers one segment
    // row (nkb = 4) or two (nkb = 2); a thread keeps its chunk and walks down the rows.  The swizzle
    // term depends on row % 8, which takes at most two values along a thread's rows. ----
    const int cpr = prm.nkb * 8;
    const int rstep = kLoadWarps * (32 / cpr);                      // 4 or 8
    const int r0 = warp * (32 / cpr) + lane / cpr;
    const int ch = lane % cpr;
    const uint32_t kb_off = static_cast<uint32_t>(ch >> 3) * prm.kb_bytes + static_cast<uint32_t>(r0) * 128u;
    const uint32_t swz_a = static_cast<uint32_t>((ch & 7) ^ (r0 & 7)) << 4;
    const uint32_t swz_b = (static_cast<uint32_t>((ch & 7) ^ ((r0 + rstep) & 7)) << 4) + static_cast<uint32_t>(rstep) * 128u;
    const long long step_b = static_cast<long long>(rstep) * prm.row_stride, step_a = 2 * step_b;
    const __nv_bfloat16* row0 = Gm + static_cast<long long>(r0) * prm.row_stride;
    const uint32_t seg_bytes = static_cast<uint32_t>(prm.rows_blk) * 128u;
    long long col0 = static_cast<long long>(p) * tile_cols + ch * 8;
    int s = 0;
    uint32_t pass = 0;
    for (long long i = 0; i < n_mine; ++i) {
      if (pass > 0) mbar_wait_backoff(empty_u32 + 8u * s, (pass - 1) & 1u, abort_flag, prm.timeout_cycles, 64);
      for (int t = 0; t < (prm.drop_loads ? 0 : prm.stack); ++t) {  // test hook: no copies, no arrival; the waits run out
        const long long col = col0 + t * seg_cols;
        const long long left = prm.d - col;                         // elements of a row from this chunk on
        const uint32_t bytes = left >= 8 ? 16u : (left > 0 ? static_cast<uint32_t>(left) * 2u : 0u);
        const __nv_bfloat16* src = row0 + (left > 0 ? col : 0);
        uint32_t dst = ring_u32 + static_cast<uint32_t>(s) * prm.stage_bytes + static_cast<uint32_t>(t) * seg_bytes + kb_off;
        for (int row = r0; row < b; row += 2 * rstep) {
          cp_async_16(dst + swz_a, src, bytes);                     // bytes past `bytes` are zero-filled
          if (row + rstep < b) cp_async_16(dst + swz_b, src + step_b, bytes);
          src += step_a;
          dst += static_cast<uint32_t>(2 * rstep) * 128u;
        }
      }
      // one arrival on the stage's barrier once this thread's copies have landed; nothing here
      // waits for them, so the loaders run a whole ring ahead of the tensor core
      if (!prm.drop_loads)
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full_u32 + 8u * s) : "memory");
      col0 += static_cast<long long>(prm.P) * tile_cols;
      if (++s == S) {
        s = 0;
        ++pass;
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");                // nothing in flight at exit
  } else if (warp == 8) {
    // ---- MMA issue: the whole warp walks the loop (uniform control flow keeps the descriptors in
    // uniform registers), one elected lane issues ----
    // instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, N / 8 at bit 17, M / 16 = 8 at bit 24
    const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | (8u << 24);
    const uint32_t idesc0 = idesc_base | (static_cast<uint32_t>(prm.n_dim >> 3) << 17);
    const uint32_t idesc1 = idesc_base | (static_cast<uint32_t>(prm.n1_dim >> 3) << 17);
    // operand descriptor, K-major with 128-byte swizzle: start address / 16, 8-row groups 1024 bytes
    // apart (64 << 32), descriptor version 1 (bit 46), swizzle mode 2 (bits 61-63)
    const uint64_t desc_hi = (64ull << 32) | (1ull << 46) | (2ull << 61) | (1ull << 16);
    const uint32_t kb16 = prm.kb_bytes >> 4;
    int s = 0, fold_pos = 0;
    uint32_t pass = 0, fold = 0;
    for (long long i = 0; i < n_mine; ++i) {
      const uint32_t buf = prm.nbuf == 2 ? (fold & 1u) : 0u;
      const uint32_t use = prm.nbuf == 2 ? (fold >> 1) : fold;      // how often this accumulator set was used before
      if (fold_pos == 0 && use > 0)
        mbar_wait(accempty_u32 + 8u * buf, (use - 1) & 1u, abort_flag, prm.timeout_cycles);
      mbar_wait(full_u32 + 8u * s, pass & 1u, abort_flag, prm.timeout_cycles);
      fence_async_smem();                                           // the copies' writes, before the tensor core reads
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * static_cast<uint32_t>(prm.buf_stride);
      const uint32_t lo = ((ring_u32 + static_cast<uint32_t>(s) * prm.stage_bytes) & 0x3ffffu) >> 4;
      const bool last_of_fold = fold_pos == prm.fold_tiles - 1 || i == n_mine - 1;
      if (elect_one()) {
        for (int kb = 0; kb < prm.nkb; ++kb) {
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t acc = (fold_pos == 0 && kb == 0 && k == 0) ? 0u : 1u;
            const uint64_t desc = desc_hi | static_cast<uint64_t>(lo + static_cast<uint32_t>(kb) * kb16 + 2u * k);
            umma_bf16(d_tmem, desc, desc, idesc0, acc);
            if (MB == 2) {
              const uint64_t desc1 = desc + 1024u;                  // rows 128..: 128 rows * 128 bytes / 16
              umma_bf16(d_tmem + static_cast<uint32_t>(prm.acc1_off), desc1, desc1, idesc1, acc);
            }
          }
        }
        umma_commit(empty_u32 + 8u * s);                            // the stage may be refilled
        if (last_of_fold) umma_commit(accfull_u32 + 8u * buf);
      }
      __syncwarp();
      if (last_of_fold) {
        fold_pos = 0;
        ++fold;
      } else {
        ++fold_pos;
      }
      if (++s == S) {
        s = 0;
        ++pass;
      }
    }
    if (elect_one()) umma_commit(done_u32);
    __syncwarp();
    volatile unsigned ignore = 0u;
    mbar_wait(done_u32, 0u, &ignore, prm.timeout_cycles);           // no MMA in flight when TMEM is freed
  } else if (warp < 8) {
    // ---- accumulator read-back: this thread owns TMEM lane r = 32 (warp % 4) + lane.
    // MB = 1: lane r is row r % rows_blk of the Gram matrix of column segment r / rows_blk, whose
    //         columns sit at [c_first, c_first + b) of the lane.
    // MB = 2: lane r of the first accumulator is row r of (K00 | K01), lane r of the second is row
    //         128 + r of K11 (its columns start at 128). ----
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const int c_first = MB == 1 ? row / prm.rows_blk * prm.rows_blk : 0;
    const bool live = MB == 1 ? (row < prm.stack * prm.rows_blk && row - c_first < b) : true;
    const int c_last = live ? c_first + b : 0;                      // columns [c_first, c_last) of this lane count
    const long long n_folds = (n_mine + prm.fold_tiles - 1) / prm.fold_tiles;
    for (long long f = 0; f < n_folds; ++f) {
      const uint32_t buf = prm.nbuf == 2 ? (static_cast<uint32_t>(f) & 1u) : 0u;
      const uint32_t use = prm.nbuf == 2 ? static_cast<uint32_t>(f >> 1) : static_cast<uint32_t>(f);
      mbar_wait_backoff(accfull_u32 + 8u * buf, use & 1u, abort_flag, prm.timeout_cycles, 256);
      tc_fence_after();
      const uint32_t taddr = tmem_base + buf * static_cast<uint32_t>(prm.buf_stride) + (static_cast<uint32_t>(q * 32) << 16);
      float diag = 0.f;
      for (int c32 = 0; c32 < prm.n_dim; c32 += 32) {               // n_dim is a multiple of 16: the last pair may
        float v[2][16];                                             // read 16 columns past it, inside the allocation
        tmem_ld32(taddr + static_cast<uint32_t>(c32), v);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int c0 = c32 + 16 * h;
          float part = 0.f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const bool in = c0 + j >= c_first && c0 + j < c_last;
            part += in ? v[h][j] : 0.f;
            diag = (c0 + j == row) ? v[h][j] : diag;
            if (MB == 2 && !in) v[h][j] = 0.f;                      // columns >= b hold whatever the operand ran into
          }
          row_sum[0] += static_cast<double>(part);
          if (MB == 2 && c0 >= 128 && c0 < prm.n_dim) {
            // column sums of K01 = row sums of K10: over this warp's 32 rows here, over the warps at the end
            col_sum[(c0 - 128) >> 4] += static_cast<double>(warp_sum_16_values(v[h], lane));
          }
        }
      }
      row_diag[0] += static_cast<double>(diag);
      if (MB == 2) {
        float diag1 = 0.f;
        for (int c32 = 0; c32 < prm.n1_dim; c32 += 32) {
          float v[2][16];
          tmem_ld32(taddr + static_cast<uint32_t>(prm.acc1_off + c32), v);
          float part = 0.f;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int c = c32 + 16 * h + j;
              part += (128 + c < b) ? v[h][j] : 0.f;
              diag1 = (c == row) ? v[h][j] : diag1;
            }
          }
          row_sum[MB - 1] += static_cast<double>(part);
        }
        row_diag[MB - 1] += static_cast<double>(diag1);
      }
      tc_fence_before();
      mbar_arrive(accempty_u32 + 8u * buf);
    }
  } else if (WANT_GBAR) {
    // ---- column means on the CUDA cores: the four warps split a segment's nkb * 8 chunks of 16
    // bytes; lane = (row phase, chunk); the row phases are folded with shuffles ----
    const int w = warp - 9;
    const int cw = prm.nkb * 2;                                     // chunks per warp: 8 or 4
    const int nph = 32 / cw;                                        // row phases: 4 or 8
    const int rph = lane / cw;
    const int gch = w * cw + lane % cw;                             // chunk of the segment
    const int kb = gch >> 3, ch = gch & 7;
    const float inv_b = 1.0f / static_cast<float>(b);
    long long col0 = static_cast<long long>(p) * tile_cols + gch * 8;
    int s = 0;
    uint32_t pass = 0;
    for (long long i = 0; i < n_mine; ++i) {
      mbar_wait_backoff(full_u32 + 8u * s, pass & 1u, abort_flag, prm.timeout_cycles, 32);
      for (int t = 0; t < prm.stack; ++t) {
        const long long col = col0 + t * seg_cols;
        const uint32_t base = ring_u32 + static_cast<uint32_t>(s) * prm.stage_bytes +
                              static_cast<uint32_t>(kb) * prm.kb_bytes + static_cast<uint32_t>(t * prm.rows_blk) * 128u;
        float cs[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = 0.f;
        for (int r = rph; r < b; r += nph) {
          const uint4 u = lds128(base + static_cast<uint32_t>(r) * 128u + (static_cast<uint32_t>(ch ^ (r & 7)) << 4));
          float x[8];
          Vec<__nv_bfloat16>::unpack(u, x);
#pragma unroll
          for (int j = 0; j < 8; ++j) cs[j] += x[j];
        }
        for (int off = cw; off < 32; off <<= 1) {
#pragma unroll
          for (int j = 0; j < 8; ++j) cs[j] += __shfl_xor_sync(0xffffffffu, cs[j], off);
        }
        if (rph == 0) {
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
      if (lane == 0) mbar_arrive(empty_u32 + 8u * s);                // this warp's reads of the stage are done
      col0 += static_cast<long long>(prm.P) * tile_cols;
      if (++s == S) {
        s = 0;
        ++pass;
      }
    }
  }

  // ---- CTA epilogue: (e_r, V, N) from the row sums and the diagonal of K ----
  if (warp >= 4 && warp < 8) {
    const int q = warp & 3;
    const int row = q * 32 + lane;
#pragma unroll
    for (int k = 0; k < MB; ++k) {
      red[kRedRow + 128 * k + row] = row_sum[k];
      red[kRedDiag + 128 * k + row] = row_diag[k];
    }
    if (MB == 2 && (lane & 1) == 0) {
      const int c = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
#pragma unroll
      for (int g = 0; g < 8; ++g) red[kRedCol + q * 128 + g * 16 + c] = col_sum[g];
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
  if (tid < b) {
    double rs = 0.0, dg = 0.0;
    if (MB == 1) {                                  // the segments' Gram matrices add up to the tile's
      for (int t = 0; t < prm.stack; ++t) {
        rs += red[kRedRow + t * prm.rows_blk + tid];
        dg += red[kRedDiag + t * prm.rows_blk + tid];
      }
    } else {
      rs = red[kRedRow + tid];
      dg = red[kRedDiag + tid];
      if (tid >= 128)
        for (int wq = 0; wq < 4; ++wq) rs += red[kRedCol + wq * 128 + tid - 128];
    }
    red[kRedRs + tid] = rs;
    red[kRedDg + tid] = dg;
  }
  __syncthreads();
  if (tid == 0) {
    double total = 0.0, trace = 0.0;
    for (int i = 0; i < b; ++i) {
      total += red[kRedRs + i];
      trace += red[kRedDg + i];
    }
    red[kRedTot] = total;
    red[kRedTot + 1] = trace;
  }
  __syncthreads();
  {
    const double bd = static_cast<double>(b);
    const double total = red[kRedTot], trace = red[kRedTot + 1];
    const double Ncta = total / (bd * bd);
    double* out = prm.ws + (static_cast<size_t>(m) * prm.P + p) * (static_cast<size_t>(b) + 2);
    for (int i = tid; i < b; i += blockDim.x) out[i] = red[kRedRs + i] / bd - Ncta;   // sum_j (g_ij - gbar_j) gbar_j
    if (tid == 0) {
      out[b] = trace - total / bd;                                                   // sum_ij (g_ij - gbar_j)^2
      out[b + 1] = Ncta;
      if (*abort_flag) atomicOr(prm.flags, 1u);
    }
  }
}

struct UmmaGeom {
  int mblocks, rows_blk, stack, nkb, n_dim, n1_dim, nbuf, buf_stride, acc1_off, tmem_cols, stages, fold_tiles;
  unsigned kb_bytes, stage_bytes;
  size_t smem;
};

bool umma_geometry(const Tuning& t, size_t smem_optin, long long b, UmmaGeom* g) {
  if (b <= 32 || b > 256) return false;
  g->rows_blk = static_cast<int>((b + 7) / 8 * 8);
  if (b <= 128) {
    g->mblocks = 1;
    g->nkb = 4;
    g->stack = 128 / g->rows_blk;                 // 1 (b > 64), 2 (40 < b <= 64) or 3 (b <= 40)
    g->n_dim = (g->stack * g->rows_blk + 15) / 16 * 16;
    g->n1_dim = 0;
    g->nbuf = 2;
    g->buf_stride = g->n_dim <= 64 ? 64 : 128;
    g->acc1_off = 0;
    g->tmem_cols = 2 * g->buf_stride;
  } else {
    g->mblocks = 2;
    g->nkb = 2;                                   // 128-column tiles, so that three stages of 256 rows fit
    g->stack = 1;
    g->n_dim = static_cast<int>((b + 15) / 16 * 16);
    g->n1_dim = g->n_dim - 128;
    g->nbuf = g->n_dim <= 192 ? 2 : 1;            // n_dim + n1_dim columns per set, 512 in all
    g->buf_stride = 256;
    g->acc1_off = g->nbuf == 2 ? 192 : 256;
    g->tmem_cols = 512;
  }
  g->kb_bytes = static_cast<unsigned>(g->stack * g->rows_blk) * 128u;
  g->stage_bytes = static_cast<unsigned>(g->nkb) * g->kb_bytes;
  const size_t pad = static_cast<size_t>(128 * g->mblocks - g->stack * g->rows_blk) * 128;
  const size_t fixed = 1024 + pad + static_cast<size_t>(kBarsU + 1) * 8 + kRedDoubles * sizeof(double) + 128;
  int stages = static_cast<int>(t.stats_stages > 0 ? t.stats_stages : kMaxStagesU);
  if (stages > kMaxStagesU) stages = kMaxStagesU;
  while (stages > 2 && static_cast<size_t>(stages) * g->stage_bytes + fixed > smem_optin) --stages;
  g->stages = stages;
  g->smem = static_cast<size_t>(stages) * g->stage_bytes + fixed;
  if (g->smem > smem_optin) return false;
  // about kFoldCols columns are added up in fp32 before the fold into fp64; twice as many where the
  // MMAs have to wait for the read-back
  const int tile_cols = g->stack * g->nkb * 64;
  int fold = (g->nbuf == 2 ? kFoldCols : 2 * kFoldCols) / tile_cols;
  if (t.stats_flush_every > 0) fold = static_cast<int>(t.stats_flush_every > 64 ? 64 : t.stats_flush_every);
  g->fold_tiles = fold < 1 ? 1 : fold;
  return true;
}

template <int MB, bool WANT_GBAR>
int launch_umma_variant(abs_ctx* ctx, const UmmaParams& prm, dim3 grid, size_t smem, cudaStream_t stream) {
  auto kern = abs_stats_umma_kernel<MB, WANT_GBAR>;
  ABS_CUDA_TRY(ctx, ensure_dynamic_smem(ctx, kern, smem));
  kern<<<grid, WANT_GBAR ? 416 : 288, smem, stream>>>(prm);
  ABS_CUDA_TRY(ctx, cudaGetLastError());
  return ABS_OK;
}

}  // namespace

int plan_stats_umma(const Tuning& t, size_t smem_optin, abs_dtype dtype, long long b, abs_stats_plan* out) {
  UmmaGeom g;
  if (dtype != ABS_BF16 || !umma_geometry(t, smem_optin, b, &g)) return ABS_ERR_UNSUPPORTED;
  memset(out, 0, sizeof(*out));
  out->route = 4;
  out->lanes_per_row = 8;                    // a k-block row: 128 bytes
  out->warps_per_box = kLoadWarps;
  out->boxes_per_stage = g.nkb;              // k-blocks
  out->stages = g.stages;
  out->box_rows = g.stack * g.rows_blk;
  out->row_boxes = 1;
  out->rows_per_thread = 0;
  out->cluster_size = 1;
  out->rows_per_cta = static_cast<int>(b);
  out->stage_bytes = g.stage_bytes;
  out->smem_bytes = g.smem;
  return ABS_OK;
}

// Takes the call for bf16 rows with 32 < b <= 256 whose base and strides are multiples of 16 bytes.
int launch_stats_umma(abs_ctx* ctx, const StatsLaunch& a, int* P_out) {
  if (a.dtype != ABS_BF16) return ABS_ERR_UNSUPPORTED;
  UmmaGeom g;
  if (!umma_geometry(ctx->tuning, ctx->smem_optin, a.b, &g)) return ABS_ERR_UNSUPPORTED;
  const unsigned long long row_b = static_cast<unsigned long long>(a.row_stride) * 2;
  const unsigned long long wrk_b = static_cast<unsigned long long>(a.M > 1 ? a.worker_stride : 0) * 2;
  if ((reinterpret_cast<uintptr_t>(a.G) & 15u) || (row_b & 15u) || (wrk_b & 15u) || a.M > 65535)
    return ABS_ERR_UNSUPPORTED;

  const long long tile_cols = static_cast<long long>(g.stack) * g.nkb * 64;
  const long long n_tiles = (a.d + tile_cols - 1) / tile_cols;
  long long P = ctx->tuning.stats_ctas_per_worker > 0 ? ctx->tuning.stats_ctas_per_worker
                                                      : static_cast<long long>(ctx->sm_count) / a.M;
  if (P < 1) P = 1;
  if (P > n_tiles) P = n_tiles;
  if (P > 65535) P = 65535;
  const size_t need = static_cast<size_t>(a.M) * P * (a.b + 2) * sizeof(double);
  if (need > ctx->workspace_bytes)
    return set_error(ctx, ABS_ERR_WORKSPACE, "abs_test_stats needs %zu workspace bytes, context has %zu", need,
                     ctx->workspace_bytes);
  UmmaParams prm;
  prm.G = static_cast<const __nv_bfloat16*>(a.G);
  prm.b = a.b;
  prm.d = a.d;
  prm.row_stride = a.row_stride;
  prm.worker_stride = a.M > 1 ? a.worker_stride : 0;
  prm.stack = g.stack;
  prm.rows_blk = g.rows_blk;
  prm.nkb = g.nkb;
  prm.n_dim = g.n_dim;
  prm.n1_dim = g.n1_dim;
  prm.nbuf = g.nbuf;
  prm.buf_stride = g.buf_stride;
  prm.acc1_off = g.acc1_off;
  prm.tmem_cols = g.tmem_cols;
  prm.stages = g.stages;
  prm.fold_tiles = g.fold_tiles;
  prm.kb_bytes = g.kb_bytes;
  prm.stage_bytes = g.stage_bytes;
  prm.n_tiles = n_tiles;
  prm.P = static_cast<int>(P);
  prm.ws = static_cast<double*>(ctx->workspace);
  prm.gbar_out = a.gbar_out;
  prm.flags = ctx->flags;
  prm.timeout_cycles = ctx->tuning.stats_timeout_cycles > 0 ? ctx->tuning.stats_timeout_cycles : kDefaultTimeoutCycles;
  prm.drop_loads = ctx->tuning.stats_fault_drop_loads ? 1 : 0;
  const dim3 grid(static_cast<unsigned>(P), static_cast<unsigned>(a.M));
  const bool gb = a.gbar_out != nullptr;
  int rc;
  if (g.mblocks == 1)
    rc = gb ? launch_umma_variant<1, true>(ctx, prm, grid, g.smem, a.stream)
            : launch_umma_variant<1, false>(ctx, prm, grid, g.smem, a.stream);
  else
    rc = gb ? launch_umma_variant<2, true>(ctx, prm, grid, g.smem, a.stream)
            : launch_umma_variant<2, false>(ctx, prm, grid, g.smem, a.stream);
  if (rc != ABS_OK) return rc;
  *P_out = static_cast<int>(P);
  return ABS_OK;
}

}  // namespace absk
