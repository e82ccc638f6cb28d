// Host side of the TMA path: 4-D tiled tensor maps with a 128-byte-swizzled inner box, encoded through the
// driver entry point that the runtime hands out (no link-time dependency on libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace jup {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(ptr);
    (void)cudaGetLastError();
    return static_cast<EncodeTiledFn>(nullptr);
  }();
  return fn;
}

// dims: extents, innermost first; strides_bytes: of dimensions 1..3 (multiples of 16, below 2^40; a dimension of
// extent 1 may pass 0); box: the tile, innermost first (inner box = 128 bytes).  Out-of-range elements of a load
// read as zero, those of a store are not written.
inline bool make_map(CUtensorMap* m, CUtensorMapDataType type, const void* base, const uint64_t dims[4],
                     const uint64_t strides_bytes[3], const uint32_t box[4], CUtensorMapL2promotion promo) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gd[4] = {dims[0], dims[1], dims[2], dims[3]};
  cuuint64_t gs[3];
  for (int i = 0; i < 3; ++i) {
    gs[i] = strides_bytes[i] ? strides_bytes[i] : 16;  // only extent-1 dimensions carry a zero stride
    if (gs[i] % 16 || gs[i] >= (1ull << 40)) return false;
  }
  cuuint32_t bx[4] = {box[0], box[1], box[2], box[3]};
  cuuint32_t es[4] = {1, 1, 1, 1};
  return fn(m, type, 4, const_cast<void*>(base), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline bool make_map_bf16(CUtensorMap* m, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                          const uint32_t box[4]) {
  return make_map(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, dims, strides_bytes, box, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}
inline bool make_map_f32(CUtensorMap* m, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3],
                         const uint32_t box[4]) {
  return make_map(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, base, dims, strides_bytes, box, CU_TENSOR_MAP_L2_PROMOTION_NONE);
}

}  // namespace jup
