// Host helper: build TMA tensor maps through the driver entry point (no link against libcuda).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

namespace diffqkv {

typedef CUresult (*TmapEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline TmapEncodeTiledFn tmap_encode_fn() {
  static TmapEncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      ptr = nullptr;
    return reinterpret_cast<TmapEncodeTiledFn>(ptr);
  }();
  return fn;
}

// bf16 tensor of `rank` dims (dims[0] innermost, contiguous), byte strides for dims 1.., 128-byte swizzle,
// out-of-range elements read as zero.  The inner box extent must be 64 elements (128 bytes).
inline bool make_tmap_bf16_sw128(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                                 const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  TmapEncodeTiledFn fn = tmap_encode_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i + 1 < rank; ++i)
    if (strides_bytes[i] == 0 || strides_bytes[i] % 16 != 0 || strides_bytes[i] >= (1ull << 40)) return false;
  for (int i = 0; i < rank; ++i)
    if (dims[i] == 0 || box[i] == 0 || box[i] > 256) return false;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace diffqkv
