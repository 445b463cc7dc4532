// Tensor maps for the tiled copy engine, encoded on the host.  The encoder is a driver entry point
// fetched through the runtime, so nothing of the driver library is linked.
#pragma once
#include <cuda.h>  // CUtensorMap and its enums (types only)
#include <cuda_runtime.h>
#include <stdint.h>

namespace mava {

// Map of a dense row-major matrix [rows][cols] of 4-byte floats or of bytes, for boxes of box_rows x box_cols;
// elements outside the matrix read as zero.  Needs a 16-byte aligned base, a row pitch and a box width that are
// multiples of 16 bytes, and box sides <= 256.
inline bool encode_map_2d(CUtensorMap *map, const void *base, bool bytes, unsigned long long cols, unsigned long long rows,
                          unsigned box_cols, unsigned box_rows, CUtensorMapSwizzle swizzle) {
  using Fn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                          const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                          CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static Fn encode = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<Fn>(p);
  }();
  const unsigned long long esize = bytes ? 1 : 4;
  if (!encode || rows < 1 || cols < 1 || reinterpret_cast<uintptr_t>(base) % 16 != 0 || (cols * esize) % 16 != 0 || box_cols > 256 ||
      box_rows > 256 || (box_cols * esize) % 16 != 0)
    return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * esize};
  const cuuint32_t box[2] = {box_cols, box_rows}, elem[2] = {1, 1};
  return encode(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims,
                strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool encode_f32_map(CUtensorMap *map, const float *base, unsigned long long cols, unsigned long long rows,
                           unsigned box_cols, unsigned box_rows, CUtensorMapSwizzle swizzle) {
  return encode_map_2d(map, base, false, cols, rows, box_cols, box_rows, swizzle);
}

// Tiled 2-D copy global -> shared through a tensor map, completion counted in bytes on an mbarrier; x is the
// innermost coordinate, in elements, and x times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
// The same box, but only as far as L2: nothing to wait for, nothing lands in shared memory.
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap *map, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y)
               : "memory");
}

}  // namespace mava
