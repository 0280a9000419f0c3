// Device-side helpers for the TMA + mbarrier tile pipelines of the statistics kernels, and the
// host-side tensor-map encoder they share.
#pragma once

#include <cuda_bf16.h>

#include "abs_internal.cuh"

namespace absk {

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
// ---- distributed shared memory ----------------------------------------------------------
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
// Copies `bytes` (a multiple of 16) from this CTA's shared memory into a peer's and adds them to
// the transaction count of the peer's mbarrier.
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes,
                                                  uint32_t mbar_cluster) {
  asm volatile(
      "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_cluster),
      "r"(src_cta), "r"(bytes), "r"(mbar_cluster)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar)
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

// 16-byte shared-memory accesses for per-thread groups of VE floats (VE = 4 or 8): a warp then
// touches 512 contiguous bytes per instruction instead of striding scalars across the banks.
template <int VE>
__device__ __forceinline__ void smem_store_vec(float* dst, const float (&v)[VE]) {
#pragma unroll
  for (int j = 0; j < VE; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
}
template <int VE>
__device__ __forceinline__ void smem_add_vec(const float* src, float (&acc)[VE]) {
#pragma unroll
  for (int j = 0; j < VE; j += 4) {
    const float4 t = *reinterpret_cast<const float4*>(src + j);
    acc[j] += t.x; acc[j + 1] += t.y; acc[j + 2] += t.z; acc[j + 3] += t.w;
  }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
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

// ---- host: 3-D tensor map over G[M][b][d] with a [1][box_rows][box_cols] box ---------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
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

// True when the tiled loads can address G: 16-byte aligned base and strides, extents within the
// tensor-map limits.
inline bool tma_addressable(const StatsLaunch& a) {
  const int es = a.dtype == ABS_F32 ? 4 : 2;
  const unsigned long long row_b = static_cast<unsigned long long>(a.row_stride) * es;
  const unsigned long long wrk_b = static_cast<unsigned long long>(a.M > 1 ? a.worker_stride : a.b * a.row_stride) * es;
  if ((reinterpret_cast<uintptr_t>(a.G) & 15u) || (row_b & 15u) || (wrk_b & 15u)) return false;
  if (a.d > 0x7fff0000ll || a.M > 65535) return false;
  if (row_b >= (1ull << 40) || wrk_b >= (1ull << 40)) return false;
  return encode_tiled_fn() != nullptr;
}

inline int encode_g_tensor_map(abs_ctx* ctx, const StatsLaunch& a, long long box_cols, int box_rows, CUtensorMap* tmap) {
  const int es = a.dtype == ABS_F32 ? 4 : 2;
  const cuuint64_t gdim[3] = {static_cast<cuuint64_t>(a.d), static_cast<cuuint64_t>(a.b), static_cast<cuuint64_t>(a.M)};
  const cuuint64_t gstr[2] = {static_cast<cuuint64_t>(a.row_stride) * es,
                              static_cast<cuuint64_t>(a.M > 1 ? a.worker_stride : a.b * a.row_stride) * es};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows), 1u};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  const CUresult r = encode_tiled_fn()(
      tmap, a.dtype == ABS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
      const_cast<void*>(a.G), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return set_error(ctx, ABS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r));
  return ABS_OK;
}

// 4-D map over the same G for very small batches: a row is cut into segments of 256 elements
// (the widest box a tensor map allows), and one box takes `segs` consecutive segments of each of
// box_rows rows: [1][box_rows][segs][256].  In shared memory a box row is then segs * 256 elements
// long, so one copy moves what several 3-D boxes would.  Needs d to be a multiple of 256.
constexpr int kSegElems = 256;
inline int encode_g_segment_map(abs_ctx* ctx, const StatsLaunch& a, int segs, int box_rows, CUtensorMap* tmap) {
  const int es = a.dtype == ABS_F32 ? 4 : 2;
  const cuuint64_t gdim[4] = {static_cast<cuuint64_t>(kSegElems), static_cast<cuuint64_t>(a.d / kSegElems),
                              static_cast<cuuint64_t>(a.b), static_cast<cuuint64_t>(a.M)};
  const cuuint64_t gstr[3] = {static_cast<cuuint64_t>(kSegElems) * es, static_cast<cuuint64_t>(a.row_stride) * es,
                              static_cast<cuuint64_t>(a.M > 1 ? a.worker_stride : a.b * a.row_stride) * es};
  const cuuint32_t box[4] = {static_cast<cuuint32_t>(kSegElems), static_cast<cuuint32_t>(segs),
                             static_cast<cuuint32_t>(box_rows), 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r = encode_tiled_fn()(
      tmap, a.dtype == ABS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
      const_cast<void*>(a.G), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return set_error(ctx, ABS_ERR_CUDA, "cuTensorMapEncodeTiled (segments) failed with code %d", static_cast<int>(r));
  return ABS_OK;
}

}  // namespace absk
