// mbarrier and TMA (cp.async.bulk.tensor) helpers shared by the kernels that stream cache
// tiles into shared memory, and the host routine that builds the tensor map of a cache.
#pragma once

#include <cuda.h>      // CUtensorMap and its enums only; the encoder is fetched from the driver at run time

#include "common.cuh"

namespace l2kv {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes)
               : "memory");
}
// Waits for the phase with the given parity; gives up after a bounded number of polls (a
// copy that never lands must not hang the GPU) and reports that through the return value.
template <int LOG2_POLLS = 20>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int spin = 0; spin < (1 << LOG2_POLLS); ++spin) {
    uint32_t done;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; "
                 "selp.u32 %0, 1, 0, p; }" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}
// One box of a rank-5 tensor map (dims: head_dim, token, kv head, layer, batch) into shared memory.
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, int c4) {
  asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
               "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
               :: "r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
               : "memory");
}

// Builds the rank-5 tensor map (head_dim, token, kv head, layer, batch) of a bf16, head_dim-128
// cache with a box of 64 elements x box_rows tokens and the 128-byte swizzle.  Returns false
// when the encoder is unavailable or rejects the geometry (callers then use another path).
inline bool make_cache_map(CUtensorMap* map, const void* base, const Geom& g, int box_rows) {
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = []() -> EncodeFn {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) !=
            cudaSuccess || res != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeFn>(fn);
  }();
  if (!encode) return false;
  cuuint64_t dims[5] = {128, (cuuint64_t)g.t_cap, (cuuint64_t)g.H, (cuuint64_t)g.L, (cuuint64_t)g.B};
  cuuint64_t strides[4] = {(cuuint64_t)g.st * 2, (cuuint64_t)g.sh * 2, (cuuint64_t)g.sl * 2,
                           (cuuint64_t)g.sb * 2};
  if (g.row_off) {
    // packed cache: one [H, total_rows, 128] plane; the two outer dimensions have extent 1
    if (g.st <= 0 || g.sh <= 0 || g.total_rows <= 0 || g.total_rows > 0x7fffffffLL) return false;
    dims[1] = (cuuint64_t)g.total_rows; dims[3] = 1; dims[4] = 1;
    strides[2] = strides[1]; strides[3] = strides[1];
  } else if (g.st <= 0 || g.sh <= 0 || g.sl <= 0 || g.sb <= 0) {
    return false;                                                       // broadcast views
  }
  const cuuint32_t box[5] = {64, (cuuint32_t)box_rows, 1, 1, 1};
  const cuuint32_t elem[5] = {1, 1, 1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides,
                box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace l2kv
