// Host side of the TMA descriptors used by the tensor-core kernels: every tile these kernels load is a box of
// a 4-D bf16 tensor with 128-byte swizzle, so one encoder serves them all.  cuTensorMapEncodeTiled is a driver
// entry point; it is looked up through the runtime, so the library does not link against libcuda.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace dash {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// nullptr when the driver does not offer the entry point (the callers then report the shape as unsupported)
inline EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// dims: extents, innermost first; strides_bytes: byte strides of dimensions 1..3 (multiples of 16);
// box: tile extents (box[0] * 2 bytes = 128, the swizzle span).  Out-of-range elements read as zero.
inline bool encode_bf16_sw128_4d(CUtensorMap* out, const void* base, const cuuint64_t* dims,
                                 const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return false;
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides_bytes, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace dash
