// Small CTA-level tile GEMM on shared-memory operands (bf16 in, fp32 out) used by the two fall-back kernels:
// the exact-running-maximum forward that redoes rescued query blocks (fine_fwd.cu) and the router for sub-cube
// counts the tensor-core router has no layout for (router.cu).  All warps of the CTA take part; 16x16 output
// tiles are dealt round-robin to the warps.
#pragma once
#include <mma.h>

#include "common.cuh"

namespace vsa2 {

// C[M x N] (+)= A[M x K] * B[K x N]
//   A_COL: A is stored column-major (i.e. the buffer holds A^T row-major), else row-major.
//   B_COL: B is stored column-major (i.e. the buffer holds B^T = [N][K] row-major), else row-major.
template <int M, int N, int K, bool A_COL, bool B_COL, bool ACCUM>
__device__ __forceinline__ void tile_gemm(const bf16* A, int lda, const bf16* B, int ldb, float* C, int ldc) {
  using namespace nvcuda;
  const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  constexpr int TM = M / 16, TN = N / 16;
  for (int t = warp; t < TM * TN; t += nwarps) {
    const int tm = t / TN, tn = t % TN;
    wmma::fragment<wmma::accumulator, 16, 16, 16, float> acc;
    float* cp = C + (size_t)tm * 16 * ldc + tn * 16;
    if (ACCUM) wmma::load_matrix_sync(acc, cp, ldc, wmma::mem_row_major);
    else wmma::fill_fragment(acc, 0.f);
#pragma unroll
    for (int k = 0; k < K; k += 16) {
      if constexpr (A_COL) {
        wmma::fragment<wmma::matrix_a, 16, 16, 16, bf16, wmma::col_major> a;
        wmma::load_matrix_sync(a, A + (size_t)k * lda + tm * 16, lda);
        if constexpr (B_COL) {
          wmma::fragment<wmma::matrix_b, 16, 16, 16, bf16, wmma::col_major> b;
          wmma::load_matrix_sync(b, B + (size_t)tn * 16 * ldb + k, ldb);
          wmma::mma_sync(acc, a, b, acc);
        } else {
          wmma::fragment<wmma::matrix_b, 16, 16, 16, bf16, wmma::row_major> b;
          wmma::load_matrix_sync(b, B + (size_t)k * ldb + tn * 16, ldb);
          wmma::mma_sync(acc, a, b, acc);
        }
      } else {
        wmma::fragment<wmma::matrix_a, 16, 16, 16, bf16, wmma::row_major> a;
        wmma::load_matrix_sync(a, A + (size_t)tm * 16 * lda + k, lda);
        if constexpr (B_COL) {
          wmma::fragment<wmma::matrix_b, 16, 16, 16, bf16, wmma::col_major> b;
          wmma::load_matrix_sync(b, B + (size_t)tn * 16 * ldb + k, ldb);
          wmma::mma_sync(acc, a, b, acc);
        } else {
          wmma::fragment<wmma::matrix_b, 16, 16, 16, bf16, wmma::row_major> b;
          wmma::load_matrix_sync(b, B + (size_t)k * ldb + tn * 16, ldb);
          wmma::mma_sync(acc, a, b, acc);
        }
      }
    }
    wmma::store_matrix_sync(cp, acc, ldc, wmma::mem_row_major);
  }
}

// Loads the 64 x D bf16 tile of block n of one head (a video cube of the raster layout, or a text block) into shared
// memory [64][ld]; padding positions are zero-filled.
template <int D>
__device__ __forceinline__ void load_cube_tile(bf16* dst, int ld, const bf16* head_base, const Geo& g, int n) {
  constexpr int CH = D / 8;
  for (int c = threadIdx.x; c < kBlockTokens * CH; c += blockDim.x) {
    int p = c / CH, ch = c % CH;
    int l = block_token(g, n, p);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (l >= 0) v = __ldg(reinterpret_cast<const uint4*>(head_base + (size_t)l * D + ch * 8));
    *reinterpret_cast<uint4*>(dst + (size_t)p * ld + ch * 8) = v;
  }
}

}  // namespace vsa2
