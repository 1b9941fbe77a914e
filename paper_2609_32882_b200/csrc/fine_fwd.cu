// Fine branch forward (paper Eq. 12) with the gated merge (Eq. 14) in the epilogue, exact-maximum version:
// for query block i, token-level softmax attention over the valid tokens of the KV blocks
// listed in row i of the CSR map; O = gate * O_c_hat[i] + O_f.  Online softmax in fp32,
// bf16 tensor-core products with fp32 accumulation.
#include "wmma_tile.cuh"

namespace vsa2 {

template <int D>
struct FineFwdSmem {
  static constexpr int LDX = D + 8;    // bf16 tiles Q, K, V
  static constexpr int LDS = 64 + 4;   // fp32 scores
  static constexpr int LDP = 64 + 8;   // bf16 probabilities
  static constexpr int LDO = D + 4;    // fp32 output accumulator
  static constexpr size_t bytes = 3 * 64 * LDX * sizeof(bf16) + 64 * LDS * sizeof(float) + 64 * LDP * sizeof(bf16) +
                                  64 * LDO * sizeof(float) + 3 * 64 * sizeof(float) + 64;
};

// One query block (i, hq, b) by a CTA of 256 threads: exact online softmax (running row maximum).
template <int D>
__device__ __forceinline__ void fine_fwd_block(unsigned char* smem_raw, int i, int hq, int b,
                                               const bf16* __restrict__ q, const bf16* __restrict__ k,
                                               const bf16* __restrict__ v, const float* __restrict__ gate,
                                               const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                                               const float* __restrict__ oc_hat, const Geo& g, void* __restrict__ o,
                                               bf16* __restrict__ o_res, float* __restrict__ lse) {
  using SM = FineFwdSmem<D>;
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);
  bf16* Ks = Qs + 64 * SM::LDX;
  bf16* Vs = Ks + 64 * SM::LDX;
  float* S = reinterpret_cast<float*>(Vs + 64 * SM::LDX);
  bf16* P = reinterpret_cast<bf16*>(S + 64 * SM::LDS);
  float* O = reinterpret_cast<float*>(P + 64 * SM::LDP);
  float* row_m = O + 64 * SM::LDO;
  float* row_l = row_m + 64;
  float* row_spare = row_l + 64;
  unsigned char* kvalid = reinterpret_cast<unsigned char*>(row_spare + 64);
  (void)row_spare;

  const int hk = hq / g.rep;
  const size_t bhq = (size_t)b * g.Hq + hq, bhk = (size_t)b * g.Hkv + hk;
  const bf16* qh = q + bhq * g.S * D;
  const bf16* kh = k + bhk * g.S * D;
  const bf16* vh = v + bhk * g.S * D;
  const int* cols = col_idx + bhq * g.nnz_cap;
  const int beg = row_ptr[bhq * (g.N + 1) + i], end = row_ptr[bhq * (g.N + 1) + i + 1];

  load_cube_tile<D>(Qs, SM::LDX, qh, g, i);
  for (int e = threadIdx.x; e < 64 * SM::LDO; e += blockDim.x) O[e] = 0.f;
  if (threadIdx.x < 64) { row_m[threadIdx.x] = -INFINITY; row_l[threadIdx.x] = 0.f; }

  const int r = threadIdx.x >> 2, qd = threadIdx.x & 3;
  constexpr int OC = D / 4;   // output columns rescaled by one thread
  for (int it = beg; it < end; ++it) {
    const int j = cols[it];
    __syncthreads();
    load_cube_tile<D>(Ks, SM::LDX, kh, g, j);
    load_cube_tile<D>(Vs, SM::LDX, vh, g, j);
    if (threadIdx.x < 64) kvalid[threadIdx.x] = block_token(g, j, threadIdx.x) >= 0;
    __syncthreads();
    tile_gemm<64, 64, D, false, true, false>(Qs, SM::LDX, Ks, SM::LDX, S, SM::LDS);
    __syncthreads();
    {
      float x[16];
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        int col = qd * 16 + c;
        x[c] = kvalid[col] ? S[r * SM::LDS + col] * g.scale : -INFINITY;
        mx = fmaxf(mx, x[c]);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_old = row_m[r], m_new = fmaxf(m_old, mx);
      float ps = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        float p = __expf(x[c] - m_new);
        bf16 pb = __float2bfloat16_rn(p);
        P[r * SM::LDP + qd * 16 + c] = pb;
        ps += p;
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      const float alpha = __expf(m_old - m_new);
#pragma unroll 8
      for (int c = 0; c < OC; ++c) O[r * SM::LDO + qd * OC + c] *= alpha;
      __syncwarp();
      if (qd == 0) {
        row_m[r] = m_new;
        row_l[r] = row_l[r] * alpha + ps;
      }
    }
    __syncthreads();
    tile_gemm<64, D, 64, false, false, true>(P, SM::LDP, Vs, SM::LDX, O, SM::LDO);
  }
  __syncthreads();
  // epilogue: normalise, merge with the coarse branch, write valid tokens only
  const int l = block_token(g, i, r);
  if (l >= 0) {
    const float denom = row_l[r];
    const float inv = denom > 0.f ? 1.f / denom : 0.f;
    const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && gate != nullptr && !block_is_text(g, i);
    const float gt = coarse ? gate[bhq * g.L + l] : 0.f;
    const float* oc = oc_hat + (bhq * g.Nvid + i) * D;
    const size_t obase = (bhq * g.S + l) * D;
    for (int c = 0; c < OC; ++c) {
      int d = qd * OC + c;
      float val = O[r * SM::LDO + d] * inv;
      if (coarse) val = fmaf(gt, oc[d], val);
      store_out(o, obase + d, val, g.out_f32);
      if (o_res != nullptr) {
        // what the bf16 rounding of O dropped, for the backward's delta
        float rounded = __bfloat162float(__float2bfloat16_rn(val));
        o_res[obase + d] = __float2bfloat16_rn(val - rounded);
      }
    }
    if (qd == 0) lse[bhq * g.S + l] = denom > 0.f ? row_m[r] + __logf(denom) : -INFINITY;
  }
}

// grid (N, Hq, batch), 256 threads
template <int D>
__global__ void __launch_bounds__(256) fine_fwd_kernel(const bf16* __restrict__ q, const bf16* __restrict__ k,
                                                       const bf16* __restrict__ v, const float* __restrict__ gate,
                                                       const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                                                       const float* __restrict__ oc_hat, Geo g, void* __restrict__ o,
                                                       bf16* __restrict__ o_res, float* __restrict__ lse) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  fine_fwd_block<D>(smem_raw, blockIdx.x, blockIdx.y, blockIdx.z, q, k, v, gate, row_ptr, col_idx, oc_hat, g, o, o_res, lse);
}

// Recomputes the query blocks listed in `items` (flat index (b*Hq + hq)*N + i).  *count may exceed the capacity of the
// list (its producers keep counting after the list is full and report that through the status word): only the `cap`
// entries that were written are read.
template <int D>
__global__ void __launch_bounds__(256) fine_fwd_list_kernel(const int* __restrict__ count, int cap, const int* __restrict__ items,
                                                            const bf16* __restrict__ q, const bf16* __restrict__ k,
                                                            const bf16* __restrict__ v, const float* __restrict__ gate,
                                                            const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                                                            const float* __restrict__ oc_hat, Geo g, void* __restrict__ o,
                                                            bf16* __restrict__ o_res, float* __restrict__ lse) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int n = min(*count, cap);
  for (int e = blockIdx.x; e < n; e += gridDim.x) {
    int item = items[e];
    int i, bh;
    item_block(g, item, bh, i);
    __syncthreads();
    fine_fwd_block<D>(smem_raw, i, bh % g.Hq, bh / g.Hq, q, k, v, gate, row_ptr, col_idx, oc_hat, g, o, o_res, lse);
  }
}

cudaError_t launch_fine_fwd_list(const Geo& g, const int* count, int cap, const int* items, const bf16* q, const bf16* k,
                                 const bf16* v, const float* gate, const int* row_ptr, const int* col_idx,
                                 const float* oc_hat, void* o, bf16* o_res, float* lse, cudaStream_t st) {
  cudaError_t e;
  if (g.D == 128) {
    size_t smb = FineFwdSmem<128>::bytes;
    if ((e = cudaFuncSetAttribute(fine_fwd_list_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_list_kernel<128><<<64, 256, smb, st>>>(count, cap, items, q, k, v, gate, row_ptr, col_idx, oc_hat, g, o, o_res, lse);
  } else {
    size_t smb = FineFwdSmem<64>::bytes;
    if ((e = cudaFuncSetAttribute(fine_fwd_list_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_list_kernel<64><<<64, 256, smb, st>>>(count, cap, items, q, k, v, gate, row_ptr, col_idx, oc_hat, g, o, o_res, lse);
  }
  return cudaGetLastError();
}

cudaError_t launch_fine_fwd(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                            const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                            float* lse, cudaStream_t st) {
  dim3 grid(g.N, g.Hq, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    size_t smb = FineFwdSmem<128>::bytes;
    if ((e = cudaFuncSetAttribute(fine_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_kernel<128><<<grid, 256, smb, st>>>(q, k, v, gate, row_ptr, col_idx, oc_hat, g, o, o_res, lse);
  } else {
    size_t smb = FineFwdSmem<64>::bytes;
    if ((e = cudaFuncSetAttribute(fine_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_kernel<64><<<grid, 256, smb, st>>>(q, k, v, gate, row_ptr, col_idx, oc_hat, g, o, o_res, lse);
  }
  return cudaGetLastError();
}

}  // namespace vsa2
