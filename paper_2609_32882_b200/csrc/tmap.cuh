// Host-side construction of TMA tensor maps over the raster [batch*heads, T, H, W, D] view of Q/K/V-like
// tensors, so that one 5-D box (64 channels x Bw x Bh x Bt x 1) is exactly one cube tile: 64 rows of 128 bytes
// in (bt, bh, bw) order, 128-byte swizzled, with tokens outside the valid grid filled with zeros.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "common.cuh"

namespace vsa2 {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [batch*heads, L, D] in raster token order -> tensor map whose box is one cube, 64 channels wide.
inline bool make_cube_tmap(CUtensorMap* out, const void* base, const Geo& g, int heads) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t D = (cuuint64_t)g.D;
  cuuint64_t dims[5] = {D, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.T, (cuuint64_t)g.batch * heads};
  cuuint64_t strides[4] = {D * 2, (cuuint64_t)g.W * D * 2, (cuuint64_t)g.H * g.W * D * 2, (cuuint64_t)g.S * D * 2};
  cuuint32_t box[5] = {64, (cuuint32_t)g.Bw, (cuuint32_t)g.Bh, (cuuint32_t)g.Bt, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The text rows of the same tensor (rows L .. L + Lt - 1 of every head) as a 5-D map whose box is 64 rows x 64 channels, so
// that the kernels fetch a text block with the same instruction and byte count as a cube; rows beyond Lt are zero-filled.
// Without text tokens (Lt = 0) the map covers one row of the video part and is never used.
inline bool make_text_tmap(CUtensorMap* out, const void* base, const Geo& g, int heads) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t D = (cuuint64_t)g.D;
  const cuuint64_t rows = g.Lt > 0 ? (cuuint64_t)g.Lt : 1;
  const unsigned char* first = reinterpret_cast<const unsigned char*>(base) + (g.Lt > 0 ? (size_t)g.L * g.D * 2 : 0);
  cuuint64_t dims[5] = {D, rows, 1, 1, (cuuint64_t)g.batch * heads};
  cuuint64_t strides[4] = {D * 2, rows * D * 2, rows * D * 2, (cuuint64_t)g.S * D * 2};
  cuuint32_t box[5] = {64, (cuuint32_t)kBlockTokens, 1, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<unsigned char*>(first), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace vsa2
