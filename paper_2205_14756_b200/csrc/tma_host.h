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
// Reads outside the tensor return zeros.  Encoding is a driver call of several
// microseconds, which dominates small problems, so each thread keeps the maps it
// built recently (a map depends only on the arguments below): a 4-way
// set-associative table indexed by a hash of the arguments, round-robin within a set.
inline bool tma_make_map_bf16(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                              const cuuint64_t* strides, const cuuint32_t* box, CUtensorMapSwizzle swizzle) {
  struct Key {
    const void* base; int rank; int swizzle; cuuint64_t dims[5]; cuuint64_t strides[4]; cuuint32_t box[5];
  };
  struct Entry { Key key; CUtensorMap map; bool used; };
  constexpr int SETS = 64, WAYS = 4;
  static thread_local Entry cache[SETS][WAYS];
  static thread_local unsigned char next_way[SETS];
  Key k;
  memset(&k, 0, sizeof(Key));  // padding bytes too: the key is hashed and compared as bytes
  k.base = base; k.rank = rank; k.swizzle = (int)swizzle;
  for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
  unsigned long long h = 1469598103934665603ull;  // FNV-1a over the key bytes
  const unsigned char* kb = reinterpret_cast<const unsigned char*>(&k);
  for (size_t i = 0; i < sizeof(Key); ++i) h = (h ^ kb[i]) * 1099511628211ull;
  const int set = (int)((h >> 20) % SETS);
  for (int w = 0; w < WAYS; ++w)
    if (cache[set][w].used && memcmp(&cache[set][w].key, &k, sizeof(Key)) == 0) {
      *map = cache[set][w].map;
      return true;
    }
  EncodeTiledFn fn = tma_encode_fn();
  if (!fn) return false;
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  Entry& e = cache[set][next_way[set]];
  next_way[set] = (unsigned char)((next_way[set] + 1) % WAYS);
  e.key = k; e.map = *map; e.used = true;
  return true;
}

}  // namespace msla
