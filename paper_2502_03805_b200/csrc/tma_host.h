// Host-side construction of TMA tensor maps (driver entry point resolved at run time, so the library links
// against the CUDA runtime only).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

namespace ckv {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Resolved once per process, whichever thread asks first (handles of different host threads may call concurrently).
inline EncodeTiledFn tma_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// 4-D bf16 tensor map, 128-byte swizzle, out-of-range elements read as zero.  dims[0] is the contiguous dimension;
// strides_elems are the element strides of dims 1..3; box gives the tile extent per dimension.
inline bool make_bf16_map_4d(CUtensorMap* m, const void* base, const cuuint64_t dims[4],
                             const long long strides_elems[3], const cuuint32_t box[4]) {
  EncodeTiledFn fn = tma_encode_fn();
  if (!fn) return false;
  cuuint64_t gstr[3];
  for (int i = 0; i < 3; ++i) {
    gstr[i] = (cuuint64_t)strides_elems[i] * 2;
    if (gstr[i] % 16 != 0 || gstr[i] >= (1ull << 40)) return false;
  }
  if (box[0] * 2 != 128) return false;  // the 128-byte swizzle span
  for (int i = 0; i < 4; ++i)
    if (box[i] < 1 || box[i] > 256) return false;
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace ckv
