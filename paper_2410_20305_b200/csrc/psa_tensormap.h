// Host-side TMA tensor-map encoding.  cuTensorMapEncodeTiled is looked up through
// the runtime so that the library does not link against the driver library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace psa {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Map over a token-major [T, H, D] tensor; box = 128 tokens x 1 head x `box_inner`
// elements, 128-byte swizzle (box_inner * elem_bytes must be 128).  Rows past T
// read as zero and are not written.
inline bool make_tile_map(CUtensorMap* m, const void* base, int64_t T, int H, int D, CUtensorMapDataType dt,
                          int elem_bytes, int box_inner, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || T <= 0) return false;
  cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(H), cuuint64_t(T)};
  cuuint64_t strides[2] = {cuuint64_t(D) * elem_bytes, cuuint64_t(H) * D * elem_bytes};
  cuuint32_t box[3] = {cuuint32_t(box_inner), 1u, cuuint32_t(box_rows)};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(m, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool make_tile_map_bf16(CUtensorMap* m, const void* base, int64_t T, int H, int D) {
  return make_tile_map(m, base, T, H, D, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, 64, 128);
}

}  // namespace psa
