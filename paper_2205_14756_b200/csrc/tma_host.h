// Host-side construction of TMA tensor maps (bf16, tiled) without linking libcuda:
// the driver entry point is fetched through the runtime.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <string.h>

namespace msla {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tma_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
    else
      cudaGetLastError();
  }
  return fn;
}

// rank <= 5; dims and box innermost first; strides[i] = byte stride of dimension i+1.
// Reads outside the tensor return zeros.  Encoding costs a driver call of a
// microsecond or two, which dominates small problems, so each thread keeps the
// last few maps it built (a map depends only on the arguments below).
inline bool tma_make_map_bf16(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                              const cuuint64_t* strides, const cuuint32_t* box, CUtensorMapSwizzle swizzle) {
  struct Key {
    const void* base; int rank; int swizzle; cuuint64_t dims[5]; cuuint64_t strides[4]; cuuint32_t box[5];
  };
  struct Entry { Key key; CUtensorMap map; bool used; };
  constexpr int SLOTS = 64;
  static thread_local Entry cache[SLOTS];
  static thread_local int next_slot = 0;
  Key k{};
  k.base = base; k.rank = rank; k.swizzle = (int)swizzle;
  for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
  for (int i = 0; i < SLOTS; ++i)
    if (cache[i].used && memcmp(&cache[i].key, &k, sizeof(Key)) == 0) {
      *map = cache[i].map;
      return true;
    }
  EncodeTiledFn fn = tma_encode_fn();
  if (!fn) return false;
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  Entry& e = cache[next_slot];
  next_slot = (next_slot + 1) % SLOTS;
  e.key = k; e.map = *map; e.used = true;
  return true;
}

}  // namespace msla
