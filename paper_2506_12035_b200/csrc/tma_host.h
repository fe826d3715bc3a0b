// Host-side construction of TMA tensor maps.  The driver entry point is looked up at
// run time through the CUDA runtime, so the library links against no driver stub and
// still loads on a machine without a GPU.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace marche {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tma_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 16-bit (bf16, or fp16 when ieee_half) tensor of `rank` dimensions (innermost first).  strides_bytes has rank-1 entries
// (the innermost stride is the element size).  Out-of-bounds elements read as zero.  swizzle128 / swizzle32: the
// box's rows are 128 / 32 bytes wide and their 16-byte chunks are permuted in shared memory (bank-conflict-free
// ldmatrix); neither: rows packed as they are.
inline bool tma_make_map_bf16(CUtensorMap* map, const void* ptr, int rank, const uint64_t* dims,
                              const uint64_t* strides_bytes, const uint32_t* box, bool swizzle128,
                              bool ieee_half = false, bool swizzle32 = false) {
  EncodeTiledFn fn = tma_encode_fn();
  if (!fn) return false;
  cuuint64_t d[5], s[5];
  cuuint32_t b[5], e[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    e[i] = 1;
    if (i + 1 < rank) s[i] = strides_bytes[i];
  }
  return fn(map, ieee_half ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
            const_cast<void*>(ptr), d, s, b, e,
            CU_TENSOR_MAP_INTERLEAVE_NONE,
            swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : (swizzle32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE),
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major [rows][cols] matrix of bf16 (elem_bytes 2) or fp32 (4) as the target of 32-row boxes
// that are 128 bytes wide (64 bf16 or 32 fp32 columns), 128-byte swizzle.
inline bool tma_make_store_map(CUtensorMap* map, void* ptr, uint64_t rows, uint64_t cols, int elem_bytes) {
  EncodeTiledFn fn = tma_encode_fn();
  if (!fn) return false;
  const cuuint64_t d[2] = {cols, rows};
  const cuuint64_t s[1] = {cols * (uint64_t)elem_bytes};
  const cuuint32_t b[2] = {(cuuint32_t)(128 / elem_bytes), 32};
  const cuuint32_t e[2] = {1, 1};
  return fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, ptr, d, s, b,
            e, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SM count of the current device (looked up once per device).
inline int device_sm_count() {
  static int n[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!n[dev]) {
    cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev);
    if (n[dev] <= 0) n[dev] = 148;
  }
  return n[dev];
}

}  // namespace marche
