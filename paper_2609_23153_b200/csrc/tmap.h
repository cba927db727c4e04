// Host-side helper shared by every translation unit that builds TMA descriptors: looks the driver's
// tensor-map encoder up once (through the runtime, so that the library needs no link against libcuda)
// and encodes the one kind of map the kernels use: a 4-D tensor of 1- or 2-byte elements whose box is
// `box_rows` rows of one 128-byte-wide slab, 128-byte swizzle, no out-of-bounds fill value (zeros).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sparkattn.h"

namespace sparkattn {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;      // the entry point is a property of the driver, not of a device
  if (fn) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(ptr);
  return fn;
}

// dims[0] is the contiguous dimension (elements); strides are those of dims[1..3], in elements.
inline int make_slab_map(CUtensorMap* map, const void* base, int elt_bytes, const uint64_t (&dims)[4],
                         const uint64_t (&strides_elems)[3], uint32_t box_rows) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return SPARKATTN_E_NO_DEVICE;
  const cuuint64_t d[4] = {dims[0], dims[1], dims[2], dims[3]};
  const cuuint64_t st[3] = {strides_elems[0] * elt_bytes, strides_elems[1] * elt_bytes, strides_elems[2] * elt_bytes};
  const cuuint32_t box[4] = {(cuuint32_t)(128 / elt_bytes), box_rows, 1u, 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r = enc(map, elt_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 4,
                         const_cast<void*>(base), d, st, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

// [B,H,N,d] tensor with the strides of `s`
inline int make_token_map(CUtensorMap* map, const void* base, int elt_bytes, const sparkattn_shape_t& s, int box_rows) {
  const uint64_t dims[4] = {(uint64_t)s.d, (uint64_t)s.N, (uint64_t)s.H, (uint64_t)s.B};
  const uint64_t strides[3] = {(uint64_t)s.stride_n, (uint64_t)s.stride_h, (uint64_t)s.stride_b};
  return make_slab_map(map, base, elt_bytes, dims, strides, (uint32_t)box_rows);
}

// multiprocessor count of the current device (queried per call: devices of one process may differ)
inline int current_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return 0;
  return n;
}

}  // namespace sparkattn
