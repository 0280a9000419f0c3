// The MLP producer's batched GEMM on the tcgen05 tensor cores (sm_100a): C = epilogue(A B) for
// fp32 operands with fp32-grade accuracy.
//
// A TF32 tensor-core product keeps 11 significant bits of each operand.  Every fp32 operand is
// therefore split in the loaders into hi = the value rounded to 11 bits and lo = the exact
// remainder, and one product a b becomes three tensor-core products a_hi b_hi + a_hi b_lo + a_lo b_hi
// (what is dropped is below 2^-22 |a b|).  The tensor core accumulates in fp32 in tensor memory
// without rounding to nearest, so a long sum would drift: a main accumulator only ever takes 32
// values of k (four additions) and is then added, rounded to nearest, to a running fp32 sum in the
// registers of the epilogue warps; three of them rotate so that this overlaps the products of the
// next two k-blocks.  The cross terms (2^-11 of the main term) have one accumulator of their own for
// the whole of K, read once at the end: what their additions lose stays below 1e-8 of the result.
// Measured against fp64 on the first layer of the MLP (K = 784, values up to 11): rms error 4.4e-7
// with all three products in one accumulator of 32 values of k, 1e-5 (max) with 128 values; the
// CUDA-core kernels (fp32 slices folded into fp64) have 1.3e-7.
//
// CTA = one 128 x 128 tile of C.  Warp roles: 0-7 loaders in two sets that take alternate k-blocks
// (global -> registers -> split -> shared memory with the 128-byte swizzle: K-major when k is the
// operand's contiguous index in global memory, MN-major when the tile's rows are, so every global
// load and every shared-memory store moves whole 16-byte pieces and nothing is transposed; a set
// issues the loads of its next k-block right after it has handed over the current one, so they are
// in flight while the other set works and while the stage is waited for), 8-15 epilogue
// (tcgen05.ld, running sum; two warps share a quarter of the TMEM lanes and take 64 columns each;
// at the end the tile goes through shared memory so that a warp stores whole rows of C), 16 MMA
// issue and TMEM allocation.  Every wait is bounded: one that runs out raises the CTA's abort flag,
// every role falls through its loop, tensor memory is freed and the device flag word is set.
//
// Where the time goes (M = 8 workers, b = 4096, the 784-1024-1024-10 network; per k-block of a
// CTA, measured by leaving parts out): products alone about 870 clocks, the loads 880, split and
// stores 540, the hand-overs between the roles 500, and they overlap only partly (about 2000 per
// k-block in all); a hand-over from the tensor core to a loader and back costs about a
// microsecond, which is what three stages of 64 KiB barely cover.
#include "abs_gemm.cuh"
#include "abs_pipeline.cuh"

namespace absk {
namespace {

constexpr int kTM = 128, kTN = 128;             // tile of C
constexpr int kTK = 32;                         // k-block: 32 floats = one 128-byte swizzled row
constexpr int kStagesT = 3;
constexpr uint32_t kAccBufs = 3;                // main accumulators in tensor memory, one k-block (32 values of k) each
constexpr int kOperandBytes = kTM * 128;        // one 128 x 32 fp32 operand tile
constexpr int kStageBytesT = 4 * kOperandBytes; // A_hi, A_lo, B_hi, B_lo
constexpr int kLoaders = 128;                   // threads of one loader set
constexpr int kLoaderSets = 2;
constexpr int kEpiWarps = 8;
constexpr int kMmaWarp = kLoaderSets * 4 + kEpiWarps;
constexpr int kThreadsT = (kMmaWarp + 1) * 32;  // 544
constexpr int kTmemCols = 512;                  // three main accumulators and one for the cross terms, 128 columns each
constexpr size_t kSmemT = static_cast<size_t>(kStagesT) * kStageBytesT + 1024 + 256;

struct TcParams {
  GemmArgs g;
  unsigned* flag;
  long long timeout_cycles;
  int drop_loads;       // fault injection for the bounded waits: the loaders fill nothing and never arrive
};

__device__ __forceinline__ void fence_async_smem_t() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ bool elect_one_t() {
  uint32_t is_leader;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(is_leader));
  return is_leader != 0;
}
// D (fp32, TMEM) (+)= A (tf32, smem, K-major) * B^T (tf32, smem, K-major); issued by one thread.
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit_t(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive columns of this thread's TMEM lane from each of two accumulators: both loads in
// flight, one wait.
__device__ __forceinline__ void tmem_ld16x2_t(uint32_t taddr0, uint32_t taddr1, float (&v)[16], float (&w)[16]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%32];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%33];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr0), "r"(taddr1)
      : "memory");
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    v[j] = __uint_as_float(r[j]);
    w[j] = __uint_as_float(r[16 + j]);
  }
}
// Bounded wait that sleeps between polls, for the warps that wait long (they leave the issue slots
// to the loaders and the MMA thread).
__device__ __forceinline__ bool mbar_wait_sleep(uint32_t bar, uint32_t parity, volatile unsigned* abort_flag,
                                                long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  if (*abort_flag) return false;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag || clock64() - t0 > limit) {
      *abort_flag = 1u;
      return false;
    }
    __nanosleep(64);
  }
  return true;
}
__device__ __forceinline__ void sts128(uint32_t addr, float4 v) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// hi: the value rounded to 11 significant bits (its low 13 mantissa bits are zero, so the tensor
// core's own conversion changes nothing); lo: the exact remainder, of which the tensor core keeps
// the leading 11 bits.
__device__ __forceinline__ void split_tf32(float a, float& hi, float& lo) {
  hi = __uint_as_float((__float_as_uint(a) + 0x1000u) & 0xffffe000u);
  lo = a - hi;
}
__device__ __forceinline__ void split4(const float4 a, float4& hi, float4& lo) {
  split_tf32(a.x, hi.x, lo.x);
  split_tf32(a.y, hi.y, lo.y);
  split_tf32(a.z, hi.z, lo.z);
  split_tf32(a.w, hi.w, lo.w);
}

// Four consecutive elements starting at p; elements at or past `left` read as zero.  `vec`: p is
// 16-byte aligned; else 8-byte alignment is tried (odd replicas of a parameter vector of odd
// half-length are 8 bytes off).
__device__ __forceinline__ float4 load4_guard(const float* p, long long left, bool vec) {
  if (left >= 4 && vec) return __ldg(reinterpret_cast<const float4*>(p));
  if (left >= 4 && (reinterpret_cast<uintptr_t>(p) & 7u) == 0) {
    const float2 a = __ldg(reinterpret_cast<const float2*>(p)), b = __ldg(reinterpret_cast<const float2*>(p) + 1);
    return make_float4(a.x, a.y, b.x, b.y);
  }
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (left > 0) v.x = __ldg(p);
  if (left > 1) v.y = __ldg(p + 1);
  if (left > 2) v.z = __ldg(p + 2);
  if (left > 3) v.w = __ldg(p + 3);
  return v;
}

// One operand tile [128 rows of the tile] x [32 values of k] of a k-block, into registers.
//   KC (k contiguous):  element (row, k) at P[row * rs + k];   piece e -> row e / 8, k quad e % 8
//   else (row contiguous): element (row, k) at P[k * ks + row]; piece e -> k = e / 32, row quad e % 32
// Either way a warp instruction reads whole 128-byte lines.
template <bool KC>
__device__ __forceinline__ void fetch_operand(const float* P, long long rs_or_ks, long long row_base, long long n_rows,
                                              int k0, int K, bool vec, int t, float4 (&r)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int e = t + kLoaders * i;
    if (KC) {
      const long long row = row_base + (e >> 3);
      const int k = k0 + 4 * (e & 7);
      r[i] = load4_guard(P + row * rs_or_ks + k, row < n_rows ? K - k : 0, vec);
    } else {
      const int k = k0 + (e >> 5);
      const long long row = row_base + 4 * (e & 31);
      r[i] = load4_guard(P + k * rs_or_ks + row, k < K ? n_rows - row : 0, vec);
    }
  }
}
// ... and from registers into the hi and lo tiles, 16 bytes at a time, in the layout the tensor core
// reads with the 128-byte swizzle:
//   KC:   K-major.  Row r of the tile is 128 bytes (its 32 values of k); the 16-byte chunk c of row r
//         sits at chunk position c ^ (r % 8); 8-row groups are 1024 bytes apart.
//   else: MN-major, for which TF32 operands have one layout: the 128-byte swizzle with a 32-byte base.
//         The tile is cut into blocks of [4 values of k] x [32 rows] (512 bytes): inside a block the 32
//         rows of one k are 128 contiguous bytes, and the 32-byte piece p of k-line kr sits at piece
//         position p ^ kr; the four row blocks of one k-quad are 512 bytes apart, the k-quads 2048.
template <bool KC>
__device__ __forceinline__ void stash_operand(uint32_t hi_tile, uint32_t lo_tile, int t, const float4 (&r)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int e = t + kLoaders * i;
    float4 hi, lo;
    split4(r[i], hi, lo);
    uint32_t off;
    if (KC) {
      const uint32_t row = static_cast<uint32_t>(e >> 3), ch = static_cast<uint32_t>(e & 7);
      off = row * 128u + ((ch ^ (row & 7u)) << 4);
    } else {
      const uint32_t k = static_cast<uint32_t>(e >> 5), rq = static_cast<uint32_t>(e & 31);
      const uint32_t kr = k & 3u, c16 = rq & 7u;
      off = (k >> 2) * 2048u + (rq >> 3) * 512u + kr * 128u + (((c16 >> 1) ^ kr) << 5) + ((c16 & 1u) << 4);
    }
    sts128(hi_tile + off, hi);
    sts128(lo_tile + off, lo);
  }
}

template <bool A_KC, bool B_KC>
__global__ void __launch_bounds__(kThreadsT, 1)
gemm_tc_kernel(const TcParams prm) {
  extern __shared__ unsigned char smem_dyn[];
  const GemmArgs& g = prm.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int z = blockIdx.z;
  const long long r0 = static_cast<long long>(blockIdx.y) * kTM, c0 = static_cast<long long>(blockIdx.x) * kTN;

  const uint32_t raw_u32 = smem_u32(smem_dyn);
  const uint32_t ring_u32 = (raw_u32 + 1023u) & ~1023u;            // the swizzle is a function of the address
  unsigned char* tail = smem_dyn + (ring_u32 - raw_u32) + static_cast<size_t>(kStagesT) * kStageBytesT;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tail);   // full[3] empty[3] accfull[3] accempty[3] done
  volatile unsigned* abort_flag = reinterpret_cast<volatile unsigned*>(bars + 14);
  unsigned* tmem_slot = const_cast<unsigned*>(abort_flag) + 1;
  const uint32_t full_u32 = smem_u32(bars);
  const uint32_t empty_u32 = full_u32 + 8u * kStagesT;
  const uint32_t accfull_u32 = empty_u32 + 8u * kStagesT;
  const uint32_t accempty_u32 = accfull_u32 + 8u * kAccBufs;
  const uint32_t done_u32 = accempty_u32 + 8u * kAccBufs;

  if (tid == 0) {
    for (int s = 0; s < kStagesT; ++s) {
      mbar_init(full_u32 + 8u * s, kLoaders);
      mbar_init(empty_u32 + 8u * s, 1);
    }
    for (int k = 0; k < kAccBufs; ++k) {
      mbar_init(accfull_u32 + 8u * k, 1);
      mbar_init(accempty_u32 + 8u * k, kEpiWarps * 32);
    }
    mbar_init(done_u32, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(static_cast<uint32_t>(kTmemCols))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_before();
  __syncthreads();
  tc_after();
  const uint32_t tmem_base = *tmem_slot;

  const int n_kb = (g.K + kTK - 1) / kTK;

  if (warp < kLoaderSets * 4) {
    // ---- loaders: set `set` takes the k-blocks kb = set, set + 2, ... ---------------------------
    const int set = warp >> 2, t = tid & (kLoaders - 1);
    const float* A = g.A + z * g.a_bs;
    const float* B = g.B + z * g.b_bs;
    const long long a_str = A_KC ? g.a_rs : g.a_cs, b_str = B_KC ? g.b_cs : g.b_rs;
    const bool a_vec = (reinterpret_cast<uintptr_t>(A) & 15u) == 0 && (a_str & 3) == 0;
    const bool b_vec = (reinterpret_cast<uintptr_t>(B) & 15u) == 0 && (b_str & 3) == 0;
    // Software pipeline: the loads of a set's next k-block are issued as soon as this one is handed
    // over (after the arrive, so that neither the fence nor the arrive has loads ahead of it), into the
    // same 16 vector registers; they are in flight while the other set works and the stage is waited for.
    float4 ra[8], rb[8];
    if (set < n_kb && !prm.drop_loads) {
      fetch_operand<A_KC>(A, a_str, r0, g.rows, set * kTK, g.K, a_vec, t, ra);
      fetch_operand<B_KC>(B, b_str, c0, g.cols, set * kTK, g.K, b_vec, t, rb);
    }
    for (int kb = set; kb < n_kb; kb += kLoaderSets) {
      if (prm.drop_loads) break;                   // test hook: the waits of the other roles must run out, not hang
      const int k_next = (kb + kLoaderSets) * kTK;                          // past K: reads nothing, gives zeros
      const int s = kb % kStagesT;
      const uint32_t pass = static_cast<uint32_t>(kb / kStagesT);
      if (pass > 0) mbar_wait(empty_u32 + 8u * s, (pass - 1) & 1u, abort_flag, prm.timeout_cycles);
      const uint32_t stage = ring_u32 + static_cast<uint32_t>(s) * kStageBytesT;
      stash_operand<A_KC>(stage, stage + kOperandBytes, t, ra);
      stash_operand<B_KC>(stage + 2 * kOperandBytes, stage + 3 * kOperandBytes, t, rb);
      fence_async_smem_t();                        // these stores, before the tensor core reads them
      mbar_arrive(full_u32 + 8u * s);
      fetch_operand<A_KC>(A, a_str, r0, g.rows, k_next, g.K, a_vec, t, ra);
      fetch_operand<B_KC>(B, b_str, c0, g.cols, k_next, g.K, b_vec, t, rb);
    }
  } else if (warp == kMmaWarp) {
    // ---- MMA issue ----------------------------------------------------------------------------
    // instruction descriptor: fp32 accumulate (bit 4), tf32 x tf32 (2 at bits 7 and 10), operand
    // majors (bit 15 / 16: 1 = the rows of the tile, not k, are contiguous in shared memory), N / 8 at
    // bit 17, M / 16 at bit 24
    const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | (A_KC ? 0u : (1u << 15)) | (B_KC ? 0u : (1u << 16)) |
                           (static_cast<uint32_t>(kTN >> 3) << 17) | (static_cast<uint32_t>(kTM >> 4) << 24);
    // operand descriptors (version 1 at bit 46, swizzle mode at bits 61-63), offsets in units of 16 bytes.
    // K-major, 128-byte swizzle (mode 2): 8-row groups 1024 bytes apart (stride offset 64); a k-step of
    // 8 values is 32 bytes further along the row.  MN-major, 128-byte swizzle with 32-byte base (mode 1):
    // row blocks 512 bytes apart (leading offset 32), k-quads 2048 bytes apart (stride offset 128); a
    // k-step of 8 values is two k-quads, 4096 bytes.
    const uint64_t desc_k = (64ull << 32) | (1ull << 46) | (2ull << 61) | (1ull << 16);
    const uint64_t desc_mn = (128ull << 32) | (1ull << 46) | (1ull << 61) | (32ull << 16);
    const uint64_t desc_a = A_KC ? desc_k : desc_mn, desc_b = B_KC ? desc_k : desc_mn;
    const uint32_t step_a = A_KC ? 2u : 256u, step_b = B_KC ? 2u : 256u;
    int s = 0;
    uint32_t pass = 0;
    for (int kb = 0; kb < n_kb; ++kb) {
      const uint32_t buf = static_cast<uint32_t>(kb) % kAccBufs, use = static_cast<uint32_t>(kb) / kAccBufs;
      if (use > 0) mbar_wait(accempty_u32 + 8u * buf, (use - 1) & 1u, abort_flag, prm.timeout_cycles);
      mbar_wait(full_u32 + 8u * s, pass & 1u, abort_flag, prm.timeout_cycles);
      fence_async_smem_t();
      tc_after();
      const uint32_t d_main = tmem_base + buf * static_cast<uint32_t>(kTN), d_cross = tmem_base + kAccBufs * kTN;
      const uint32_t base = ((ring_u32 + static_cast<uint32_t>(s) * kStageBytesT) & 0x3ffffu) >> 4;
      const uint32_t op16 = kOperandBytes >> 4;
      if (elect_one_t()) {
#pragma unroll
        for (int k = 0; k < kTK / 8; ++k) {                          // an instruction takes 8 values of k (32 bytes)
          const uint64_t a_hi = desc_a | static_cast<uint64_t>(base + step_a * k);
          const uint64_t a_lo = desc_a | static_cast<uint64_t>(base + op16 + step_a * k);
          const uint64_t b_hi = desc_b | static_cast<uint64_t>(base + 2u * op16 + step_b * k);
          const uint64_t b_lo = desc_b | static_cast<uint64_t>(base + 3u * op16 + step_b * k);
          // The cross terms are 2^-11 of the main term: they have an accumulator of their own for the
          // whole of K (what their additions lose is below 1e-8 of the result), and a main accumulator
          // takes one addition per 8 values of k, four in all.
          umma_tf32(d_main, a_hi, b_hi, idesc, k == 0 ? 0u : 1u);
          umma_tf32(d_cross, a_lo, b_hi, idesc, (kb == 0 && k == 0) ? 0u : 1u);
          umma_tf32(d_cross, a_hi, b_lo, idesc, 1u);
        }
        umma_commit_t(empty_u32 + 8u * s);                           // the stage may be refilled
        umma_commit_t(accfull_u32 + 8u * buf);
      }
      __syncwarp();
      if (++s == kStagesT) {
        s = 0;
        ++pass;
      }
    }
    if (elect_one_t()) umma_commit_t(done_u32);
    __syncwarp();
    volatile unsigned ignore = 0u;
    mbar_wait(done_u32, 0u, &ignore, prm.timeout_cycles);            // no MMA in flight when TMEM is freed
  } else {
    // ---- epilogue: this thread owns row 32 (warp % 4) + lane of the tile and 64 of its columns ----
    constexpr int kCols = kTN / 2;
    const int q = warp & 3, half = (warp - kLoaderSets * 4) >> 2;
    const int row = q * 32 + lane;
    const int cb = half * kCols;                                     // first column of this thread's share
    float acc[kCols];
#pragma unroll
    for (int j = 0; j < kCols; ++j) acc[j] = 0.f;
    const uint32_t t_row = tmem_base + static_cast<uint32_t>(cb) + (static_cast<uint32_t>(q * 32) << 16);
    for (int kb = 0; kb < n_kb; ++kb) {
      const uint32_t buf = static_cast<uint32_t>(kb) % kAccBufs, use = static_cast<uint32_t>(kb) / kAccBufs;
      mbar_wait_sleep(accfull_u32 + 8u * buf, use & 1u, abort_flag, prm.timeout_cycles);
      tc_after();
      const uint32_t taddr = t_row + buf * static_cast<uint32_t>(kTN);
#pragma unroll
      for (int c32 = 0; c32 < kCols; c32 += 32) {
        float v[16], w[16];
        tmem_ld16x2_t(taddr + static_cast<uint32_t>(c32), taddr + static_cast<uint32_t>(c32 + 16), v, w);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          acc[c32 + j] += v[j];                                      // rounded to nearest
          acc[c32 + 16 + j] += w[j];
        }
      }
      tc_before();
      mbar_arrive(accempty_u32 + 8u * buf);
    }
    if (n_kb > 0) {                                                  // the cross terms of the whole product
#pragma unroll
      for (int c32 = 0; c32 < kCols; c32 += 32) {
        float v[16], w[16];
        tmem_ld16x2_t(t_row + kAccBufs * kTN + static_cast<uint32_t>(c32),
                      t_row + kAccBufs * kTN + static_cast<uint32_t>(c32 + 16), v, w);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          acc[c32 + j] += v[j];
          acc[c32 + 16 + j] += w[j];
        }
      }
    }
    // The thread owns a row of the tile, so stores straight from its registers would touch 32 lines
    // per warp instruction.  The tile goes through shared memory instead (the ring is free: the last
    // accumulator was complete, so every product has read its operands): row r at r * 512 bytes, its
    // 16-byte chunk c at position c ^ (r % 32), which keeps both the row-per-thread stores and the
    // row-per-warp loads free of bank conflicts.  Then a warp instruction moves 512 contiguous bytes
    // of one row of C (and of the mask).
#pragma unroll
    for (int j = 0; j < kCols; j += 4) {
      const uint32_t c = static_cast<uint32_t>((cb + j) >> 2);
      sts128(ring_u32 + static_cast<uint32_t>(row) * 512u + ((c ^ static_cast<uint32_t>(row & 31)) << 4),
             make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]));
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory");   // the epilogue warps only
    const int ew = warp - kLoaderSets * 4;
    const long long c = c0 + 4 * lane;                               // this lane's four columns
    float4 bias4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (g.mode == 1 || g.mode == 2) {
      const float* bias = g.bias + z * g.bias_bs + c;
      if (c < g.cols) bias4.x = bias[0];
      if (c + 1 < g.cols) bias4.y = bias[1];
      if (c + 2 < g.cols) bias4.z = bias[2];
      if (c + 3 < g.cols) bias4.w = bias[3];
    }
    constexpr int kRowsPerWarp = kTM / kEpiWarps;
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
      const int trow = ew * kRowsPerWarp + rr;
      const long long r = r0 + trow;
      if (r >= g.rows || c >= g.cols) break;
      const uint4 u = lds128(ring_u32 + static_cast<uint32_t>(trow) * 512u +
                             ((static_cast<uint32_t>(lane) ^ static_cast<uint32_t>(trow & 31)) << 4));
      float o[4] = {__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w)};
      const bool full = c + 3 < g.cols;
      if (g.mode == 0) {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) o[q4] *= g.alpha;
      } else if (g.mode == 1) {
        o[0] = fmaxf(o[0] + bias4.x, 0.f); o[1] = fmaxf(o[1] + bias4.y, 0.f);
        o[2] = fmaxf(o[2] + bias4.z, 0.f); o[3] = fmaxf(o[3] + bias4.w, 0.f);
      } else if (g.mode == 2) {
        o[0] += bias4.x; o[1] += bias4.y; o[2] += bias4.z; o[3] += bias4.w;
      } else {
        const float* mrow = g.mask + z * g.mask_bs + r * g.mask_rs + c;
        float mk[4] = {0.f, 0.f, 0.f, 0.f};
        if (full && (reinterpret_cast<uintptr_t>(mrow) & 15u) == 0) {
          const float4 m4 = __ldg(reinterpret_cast<const float4*>(mrow));
          mk[0] = m4.x; mk[1] = m4.y; mk[2] = m4.z; mk[3] = m4.w;
        } else {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            if (c + q4 < g.cols) mk[q4] = __ldg(mrow + q4);
        }
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) o[q4] = mk[q4] > 0.f ? o[q4] : 0.f;
      }
      float* Crow = g.C + z * g.c_bs + r * g.c_rs + c;
      if (full && (reinterpret_cast<uintptr_t>(Crow) & 15u) == 0) {
        *reinterpret_cast<float4*>(Crow) = make_float4(o[0], o[1], o[2], o[3]);
      } else {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4)
          if (c + q4 < g.cols) Crow[q4] = o[q4];
      }
    }
  }
  tc_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(kTmemCols))
                 : "memory");
  }
  if (tid == 0 && *abort_flag) atomicOr(prm.flag, 1u);
}

template <bool A_KC, bool B_KC>
bool launch_tc_variant(const TcParams& prm, dim3 grid, cudaStream_t st) {
  auto kern = gemm_tc_kernel<A_KC, B_KC>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemT)) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  kern<<<grid, kThreadsT, kSmemT, st>>>(prm);
  return true;
}

}  // namespace

bool launch_gemm_tc(const GemmArgs& g, int batch, unsigned* flag, long long timeout_cycles, bool drop_loads,
                    cudaStream_t st) {
  const bool a_kc = g.a_cs == 1, a_rc = g.a_rs == 1, b_kc = g.b_rs == 1, b_cc = g.b_cs == 1;
  if (!(a_kc || a_rc) || !(b_kc || b_cc)) return false;
  // a 128 x 128 tile of 32-value k-blocks must be worth it: one large side, and enough work overall
  if ((g.rows < 96 && g.cols < 96) || g.K < 8 ||
      static_cast<long long>(g.rows) * g.cols * g.K < (1ll << 21))
    return false;
  const unsigned gx = static_cast<unsigned>((g.cols + kTN - 1) / kTN), gy = static_cast<unsigned>((g.rows + kTM - 1) / kTM);
  if (gy > 65535u || batch > 65535) return false;
  TcParams prm{g, flag, timeout_cycles, drop_loads ? 1 : 0};
  const dim3 grid(gx, gy, static_cast<unsigned>(batch));
  // the three operand layouts the producer has (A row-contiguous with B k-contiguous does not occur)
  if (a_kc && b_kc) return launch_tc_variant<true, true>(prm, grid, st);
  if (a_kc) return launch_tc_variant<true, false>(prm, grid, st);
  if (b_kc) return false;
  return launch_tc_variant<false, false>(prm, grid, st);
}

}  // namespace absk
