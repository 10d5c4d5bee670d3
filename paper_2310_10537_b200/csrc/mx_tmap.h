// Tensor-map encoding shared by the kernels that copy with TMA: the driver's encoder is looked up
// at run time (no link against libcuda) and its results are cached.
#pragma once

#include <cuda.h>  // CUtensorMap and enums only
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

namespace mx {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn(cudaError_t* err) {
  static EncodeTiledFn fn = nullptr;
  if (fn) { *err = cudaSuccess; return fn; }
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  *err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
  if (*err != cudaSuccess) return nullptr;
  if (q != cudaDriverEntryPointSuccess || !p) { *err = cudaErrorNotSupported; return nullptr; }
  fn = (EncodeTiledFn)p;
  return fn;
}

typedef CUresult (*Im2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                             CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                             CUtensorMapFloatOOBfill);

// The driver's im2col-mode encoder (convolution: the copy engine walks the input pixels itself).
inline Im2colFn im2col_fn(cudaError_t* err) {
  static Im2colFn fn = nullptr;
  if (fn) { *err = cudaSuccess; return fn; }
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  *err = cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &q);
  if (*err != cudaSuccess) return nullptr;
  if (q != cudaDriverEntryPointSuccess || !p) { *err = cudaErrorNotSupported; return nullptr; }
  fn = (Im2colFn)p;
  return fn;
}

inline EncodeTiledFn encode_fn_cached() {
  cudaError_t e;
  return encode_fn(&e);
}

// Encoding a tensor map is a driver call of about a microsecond, and a GEMM needs five or six; a
// layer that is called again with the same buffers (every step of a training or decoding loop)
// asks for the very same maps.  The encoder's result depends on its arguments only (address,
// extents, strides, box, type, swizzle), so the last results are kept per thread, keyed on all of
// them, in a small direct-mapped table; a repeated GEMM then makes no driver call at all.
struct MapKey {
  uint64_t ptr, dims[3], strides[2];
  uint32_t box[3], dtype, rank, swizzle, promo, pad;
  bool operator==(const MapKey& o) const { return std::memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapSlot {
  MapKey key;
  CUtensorMap map;
  bool used;
};
constexpr int kMapSlots = 64;

inline bool encode_cached(EncodeTiledFn fn, CUtensorMap* map, CUtensorMapDataType dt, uint32_t rank, const void* ptr,
                   const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
                   CUtensorMapSwizzle swz, CUtensorMapL2promotion promo) {
  static thread_local MapSlot slots[kMapSlots];
  MapKey k;
  std::memset(&k, 0, sizeof(k));
  k.ptr = (uint64_t)(uintptr_t)ptr;
  for (uint32_t i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
  for (uint32_t i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
  k.dtype = (uint32_t)dt; k.rank = rank; k.swizzle = (uint32_t)swz; k.promo = (uint32_t)promo;
  uint64_t h = 1469598103934665603ull;  // FNV-1a over the key
  const unsigned char* b = reinterpret_cast<const unsigned char*>(&k);
  for (size_t i = 0; i < sizeof(k); ++i) h = (h ^ b[i]) * 1099511628211ull;
  MapSlot& slot = slots[h % kMapSlots];
  if (slot.used && slot.key == k) {
    *map = slot.map;
    return true;
  }
  const cuuint32_t estr[3] = {1, 1, 1};
  if (fn(map, dt, rank, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
         promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  slot.key = k;
  slot.map = *map;
  slot.used = true;
  return true;
}

}  // namespace mx
