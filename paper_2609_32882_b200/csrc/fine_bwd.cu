// Backward of the fine branch (gradient of paper Eq. 12) and of the gated merge (Eq. 14).
//   preprocess: delta = rowsum(dO * O_f), dGate = rowsum(dO * O_c), dO_c_hat[n] = sum_{l in n} gate_l dO_l
//   dQ pass   : query-block stationary, driven by the CSR map
//   dK/dV pass: KV-block stationary, driven by the CSC map (transpose), summing the query heads of a
//               GQA group; no floating-point atomics anywhere.
// With P = exp(S*scale - lse), dP = dO V^T, dS = P * (dP - delta):
//   dQ = dS K * scale,  dK = dS^T Q * scale,  dV = P^T dO.
// The pooling backward of the coarse branch (Eq. 1) is added in the epilogues:
//   dX[l] += dX_c[cube(l)] / count(cube(l)).
#include "wmma_tile.cuh"

namespace vsa2 {

// ------------------------------------------------------------------------------------------
// preprocess: grid (N, Hq, batch), 256 threads
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) bwd_preprocess_kernel(const bf16* __restrict__ d_o, const void* __restrict__ o,
                                                             const bf16* __restrict__ o_res,
                                                             const float* __restrict__ gate,
                                                             const float* __restrict__ oc_hat, Geo g,
                                                             float* __restrict__ delta, float* __restrict__ dgate,
                                                             float* __restrict__ d_oc_hat) {
  // HBM-bound: one pass over dO and O (and the bf16 residual of O).  Four threads per token row; thread qd of a row
  // takes the 16-byte chunks qd, qd + 4, ... of the row, so the four threads of a row read 64 contiguous bytes per load
  // instruction, and all loads of a thread are issued before the first use.
  constexpr int LD = D + 1;            // odd row pitch: the staging stores below hit 32 different banks per warp
  __shared__ float gdo[64 * LD];       // gate_l * dO_l
  __shared__ float ocs[D];
  const int i = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const size_t bhq = (size_t)b * g.Hq + hq;
  const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && gate != nullptr;
  const int r = threadIdx.x >> 2, qd = threadIdx.x & 3;
  constexpr int NCH = D / 32;          // 16-byte chunks (8 channels) per thread
  int nt, nh, nw;
  cube_coords(g, i, nt, nh, nw);
  const int l = cube_token(g, nt, nh, nw, r);
  if (coarse)
    for (int d = threadIdx.x; d < D; d += blockDim.x) ocs[d] = oc_hat[(bhq * g.N + i) * D + d];
  float s_oo = 0.f, s_oc = 0.f;
  const float gt = (coarse && l >= 0) ? gate[bhq * g.L + l] : 0.f;
  uint4 dv[NCH], ob[NCH], rb[NCH];
  float4 of[NCH][2];
  if (l >= 0) {
    const size_t base = (bhq * g.L + l) * D;
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
      const int d0 = (4 * k + qd) * 8;
      dv[k] = __ldg(reinterpret_cast<const uint4*>(d_o + base + d0));
      if (g.out_f32) {
        of[k][0] = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(o) + base + d0));
        of[k][1] = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(o) + base + d0 + 4));
      } else {
        ob[k] = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(o) + base + d0));
        if (o_res != nullptr) rb[k] = __ldg(reinterpret_cast<const uint4*>(o_res + base + d0));
      }
    }
  }
  __syncthreads();                     // ocs visible
  if (l >= 0) {
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
      const int d0 = (4 * k + qd) * 8;
      const __nv_bfloat162* d2 = reinterpret_cast<const __nv_bfloat162*>(&dv[k]);
      float ov[8];
      if (g.out_f32) {
        ov[0] = of[k][0].x; ov[1] = of[k][0].y; ov[2] = of[k][0].z; ov[3] = of[k][0].w;
        ov[4] = of[k][1].x; ov[5] = of[k][1].y; ov[6] = of[k][1].z; ov[7] = of[k][1].w;
      } else {
        const __nv_bfloat162* o2 = reinterpret_cast<const __nv_bfloat162*>(&ob[k]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(o2[e]);
          ov[2 * e] = f.x; ov[2 * e + 1] = f.y;
        }
        if (o_res != nullptr) {
          const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(&rb[k]);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(r2[e]);
            ov[2 * e] += f.x; ov[2 * e + 1] += f.y;
          }
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 dd = __bfloat1622float2(d2[e]);
        const int d = d0 + 2 * e;
        s_oo = fmaf(dd.x, ov[2 * e], s_oo);
        s_oo = fmaf(dd.y, ov[2 * e + 1], s_oo);
        if (coarse) {
          s_oc = fmaf(dd.x, ocs[d], s_oc);
          s_oc = fmaf(dd.y, ocs[d + 1], s_oc);
          gdo[r * LD + d] = gt * dd.x;
          gdo[r * LD + d + 1] = gt * dd.y;
        }
      }
    }
  } else if (coarse) {
#pragma unroll
    for (int k = 0; k < NCH; ++k)
#pragma unroll
      for (int e = 0; e < 8; ++e) gdo[r * LD + (4 * k + qd) * 8 + e] = 0.f;
  }
  s_oo += __shfl_xor_sync(0xffffffffu, s_oo, 1);
  s_oo += __shfl_xor_sync(0xffffffffu, s_oo, 2);
  s_oc += __shfl_xor_sync(0xffffffffu, s_oc, 1);
  s_oc += __shfl_xor_sync(0xffffffffu, s_oc, 2);
  if (qd == 0 && l >= 0) {
    delta[bhq * g.L + l] = s_oo - gt * s_oc;     // rowsum(dO * (O - gate*O_c)) = rowsum(dO * O_f)
    if (dgate != nullptr) dgate[bhq * g.L + l] = s_oc;
  }
  if (coarse) {
    __syncthreads();
    // column sums over the 64 tokens: two threads per channel, 32 tokens each
    const int d = threadIdx.x % D, part = threadIdx.x / D;
    constexpr int PARTS = 256 / D;     // 2 (D = 128) or 4 (D = 64)
    float acc = 0.f;
#pragma unroll 8
    for (int p = part * (64 / PARTS); p < (part + 1) * (64 / PARTS); ++p) acc += gdo[p * LD + d];
    __syncthreads();
    gdo[part * LD + d] = acc;
    __syncthreads();
    if (threadIdx.x < D) {
      float tot = 0.f;
#pragma unroll
      for (int q = 0; q < PARTS; ++q) tot += gdo[q * LD + threadIdx.x];
      d_oc_hat[(bhq * g.N + i) * D + threadIdx.x] = tot;
    }
  }
}

cudaError_t launch_bwd_preprocess(const Geo& g, const bf16* d_o, const void* o, const bf16* o_res, const float* gate,
                                  const float* oc_hat, float* delta, float* dgate, float* d_oc_hat, cudaStream_t st) {
  dim3 grid(g.N, g.Hq, g.batch);
  if (g.D == 128) bwd_preprocess_kernel<128><<<grid, 256, 0, st>>>(d_o, o, o_res, gate, oc_hat, g, delta, dgate, d_oc_hat);
  else bwd_preprocess_kernel<64><<<grid, 256, 0, st>>>(d_o, o, o_res, gate, oc_hat, g, delta, dgate, d_oc_hat);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// dQ pass: grid (N, Hq, batch), 256 threads
// ------------------------------------------------------------------------------------------
template <int D>
struct BwdSmem {
  static constexpr int LDX = D + 8;
  static constexpr int LDS = 64 + 4;
  static constexpr int LDP = 64 + 8;
  static constexpr int LDO = D + 4;
  static constexpr size_t tile = 64 * LDX * sizeof(bf16);
  static constexpr size_t sc = 64 * LDS * sizeof(float);
  static constexpr size_t pb = 64 * LDP * sizeof(bf16);
  static constexpr size_t acc = 64 * LDO * sizeof(float);
  static constexpr size_t dq_bytes = 4 * tile + 2 * sc + pb + acc + 2 * 64 * sizeof(float) + 64;
  static constexpr size_t dkv_bytes = 4 * tile + 2 * sc + 2 * pb + 2 * acc + 2 * 64 * sizeof(float) + 128;
};

template <int D>
__global__ void __launch_bounds__(256) fine_bwd_dq_kernel(const bf16* __restrict__ q, const bf16* __restrict__ k,
                                                          const bf16* __restrict__ v, const bf16* __restrict__ d_o,
                                                          const float* __restrict__ lse, const float* __restrict__ delta,
                                                          const int* __restrict__ row_ptr, const int* __restrict__ col_idx,
                                                          const float* __restrict__ dqc, Geo g, void* __restrict__ dq) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  using SM = BwdSmem<D>;
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);
  bf16* dOs = Qs + 64 * SM::LDX;
  bf16* Ks = dOs + 64 * SM::LDX;
  bf16* Vs = Ks + 64 * SM::LDX;
  float* S = reinterpret_cast<float*>(Vs + 64 * SM::LDX);
  float* dP = S + 64 * SM::LDS;
  bf16* dS = reinterpret_cast<bf16*>(dP + 64 * SM::LDS);
  float* A = reinterpret_cast<float*>(dS + 64 * SM::LDP);
  float* row_lse = A + 64 * SM::LDO;
  float* row_delta = row_lse + 64;
  unsigned char* kvalid = reinterpret_cast<unsigned char*>(row_delta + 64);

  const int i = blockIdx.x, hq = blockIdx.y, b = blockIdx.z, hk = hq / g.rep;
  const size_t bhq = (size_t)b * g.Hq + hq, bhk = (size_t)b * g.Hkv + hk;
  const bf16* kh = k + bhk * g.L * D;
  const bf16* vh = v + bhk * g.L * D;
  const int* cols = col_idx + bhq * g.nnz_cap;
  const int beg = row_ptr[bhq * (g.N + 1) + i], end = row_ptr[bhq * (g.N + 1) + i + 1];
  int nt, nh, nw;
  cube_coords(g, i, nt, nh, nw);

  load_cube_tile<D>(Qs, SM::LDX, q + bhq * g.L * D, g, i);
  load_cube_tile<D>(dOs, SM::LDX, d_o + bhq * g.L * D, g, i);
  for (int e = threadIdx.x; e < 64 * SM::LDO; e += blockDim.x) A[e] = 0.f;
  if (threadIdx.x < 64) {
    int l = cube_token(g, nt, nh, nw, threadIdx.x);
    row_lse[threadIdx.x] = l >= 0 ? lse[bhq * g.L + l] : INFINITY;   // +inf => P = 0 for padding rows
    row_delta[threadIdx.x] = l >= 0 ? delta[bhq * g.L + l] : 0.f;
  }
  for (int it = beg; it < end; ++it) {
    const int j = cols[it];
    __syncthreads();
    load_cube_tile<D>(Ks, SM::LDX, kh, g, j);
    load_cube_tile<D>(Vs, SM::LDX, vh, g, j);
    if (threadIdx.x < 64) {
      int jt, jh, jw;
      cube_coords(g, j, jt, jh, jw);
      kvalid[threadIdx.x] = cube_token(g, jt, jh, jw, threadIdx.x) >= 0;
    }
    __syncthreads();
    tile_gemm<64, 64, D, false, true, false>(Qs, SM::LDX, Ks, SM::LDX, S, SM::LDS);
    tile_gemm<64, 64, D, false, true, false>(dOs, SM::LDX, Vs, SM::LDX, dP, SM::LDS);
    __syncthreads();
    for (int e = threadIdx.x; e < 64 * 64; e += blockDim.x) {
      int r = e >> 6, c = e & 63;
      float p = kvalid[c] ? __expf(S[r * SM::LDS + c] * g.scale - row_lse[r]) : 0.f;
      float ds = p * (dP[r * SM::LDS + c] - row_delta[r]) * g.scale;
      dS[r * SM::LDP + c] = __float2bfloat16_rn(ds);
    }
    __syncthreads();
    tile_gemm<64, D, 64, false, false, true>(dS, SM::LDP, Ks, SM::LDX, A, SM::LDO);
  }
  __syncthreads();
  const int r = threadIdx.x >> 2, qd = threadIdx.x & 3;
  constexpr int OC = D / 4;
  const int l = cube_token(g, nt, nh, nw, r);
  if (l >= 0) {
    const bool coarse = dqc != nullptr;
    const float inv_cnt = 1.f / (float)cube_count(g, i);
    const float* qc_g = coarse ? dqc + (bhq * g.N + i) * D : nullptr;
    const size_t obase = (bhq * g.L + l) * D;
    for (int c = 0; c < OC; ++c) {
      int d = qd * OC + c;
      float val = A[r * SM::LDO + d];
      if (coarse) val = fmaf(qc_g[d], inv_cnt, val);
      store_out(dq, obase + d, val, g.out_f32);
    }
  }
}

// ------------------------------------------------------------------------------------------
// dK/dV pass: grid (N, Hkv, batch), 256 threads
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) fine_bwd_dkv_kernel(const bf16* __restrict__ q, const bf16* __restrict__ k,
                                                           const bf16* __restrict__ v, const bf16* __restrict__ d_o,
                                                           const float* __restrict__ lse, const float* __restrict__ delta,
                                                           const int* __restrict__ col_ptr, const int* __restrict__ row_idx,
                                                           const float* __restrict__ dkc, const float* __restrict__ dvc,
                                                           Geo g, void* __restrict__ dk, void* __restrict__ dv) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  using SM = BwdSmem<D>;
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);
  bf16* Vs = Ks + 64 * SM::LDX;
  bf16* Qs = Vs + 64 * SM::LDX;
  bf16* dOs = Qs + 64 * SM::LDX;
  float* S = reinterpret_cast<float*>(dOs + 64 * SM::LDX);
  float* dP = S + 64 * SM::LDS;
  bf16* P = reinterpret_cast<bf16*>(dP + 64 * SM::LDS);
  bf16* dS = P + 64 * SM::LDP;
  float* AK = reinterpret_cast<float*>(dS + 64 * SM::LDP);
  float* AV = AK + 64 * SM::LDO;
  float* row_lse = AV + 64 * SM::LDO;
  float* row_delta = row_lse + 64;
  unsigned char* kvalid = reinterpret_cast<unsigned char*>(row_delta + 64);

  const int j = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const size_t bhk = (size_t)b * g.Hkv + hk;
  int jt, jh, jw;
  cube_coords(g, j, jt, jh, jw);
  load_cube_tile<D>(Ks, SM::LDX, k + bhk * g.L * D, g, j);
  load_cube_tile<D>(Vs, SM::LDX, v + bhk * g.L * D, g, j);
  for (int e = threadIdx.x; e < 64 * SM::LDO; e += blockDim.x) { AK[e] = 0.f; AV[e] = 0.f; }
  if (threadIdx.x < 64) kvalid[threadIdx.x] = cube_token(g, jt, jh, jw, threadIdx.x) >= 0;

  for (int hh = 0; hh < g.rep; ++hh) {
    const int hq = hk * g.rep + hh;
    const size_t bhq = (size_t)b * g.Hq + hq;
    const int* rows = row_idx + bhq * g.nnz_cap;
    const int beg = col_ptr[bhq * (g.N + 1) + j], end = col_ptr[bhq * (g.N + 1) + j + 1];
    for (int it = beg; it < end; ++it) {
      const int i = rows[it];
      __syncthreads();
      load_cube_tile<D>(Qs, SM::LDX, q + bhq * g.L * D, g, i);
      load_cube_tile<D>(dOs, SM::LDX, d_o + bhq * g.L * D, g, i);
      if (threadIdx.x < 64) {
        int it_, ih_, iw_;
        cube_coords(g, i, it_, ih_, iw_);
        int l = cube_token(g, it_, ih_, iw_, threadIdx.x);
        row_lse[threadIdx.x] = l >= 0 ? lse[bhq * g.L + l] : INFINITY;
        row_delta[threadIdx.x] = l >= 0 ? delta[bhq * g.L + l] : 0.f;
      }
      __syncthreads();
      tile_gemm<64, 64, D, false, true, false>(Qs, SM::LDX, Ks, SM::LDX, S, SM::LDS);
      tile_gemm<64, 64, D, false, true, false>(dOs, SM::LDX, Vs, SM::LDX, dP, SM::LDS);
      __syncthreads();
      for (int e = threadIdx.x; e < 64 * 64; e += blockDim.x) {
        int r = e >> 6, c = e & 63;
        float p = kvalid[c] ? __expf(S[r * SM::LDS + c] * g.scale - row_lse[r]) : 0.f;
        float ds = p * (dP[r * SM::LDS + c] - row_delta[r]) * g.scale;
        P[r * SM::LDP + c] = __float2bfloat16_rn(p);
        dS[r * SM::LDP + c] = __float2bfloat16_rn(ds);
      }
      __syncthreads();
      tile_gemm<64, D, 64, true, false, true>(P, SM::LDP, dOs, SM::LDX, AV, SM::LDO);    // dV += P^T dO
      tile_gemm<64, D, 64, true, false, true>(dS, SM::LDP, Qs, SM::LDX, AK, SM::LDO);    // dK += dS^T Q
    }
  }
  __syncthreads();
  const int r = threadIdx.x >> 2, qd = threadIdx.x & 3;
  constexpr int OC = D / 4;
  const int l = cube_token(g, jt, jh, jw, r);
  if (l >= 0) {
    const bool coarse = dkc != nullptr;
    const float inv_cnt = 1.f / (float)cube_count(g, j);
    const size_t obase = (bhk * g.L + l) * D;
    for (int c = 0; c < OC; ++c) {
      int d = qd * OC + c;
      float vk = AK[r * SM::LDO + d], vv = AV[r * SM::LDO + d];
      if (coarse) {
        float ck = 0.f, cv = 0.f;
        for (int hh = 0; hh < g.rep; ++hh) {
          size_t cidx = (((size_t)b * g.Hq + hk * g.rep + hh) * g.N + j) * D + d;
          ck += dkc[cidx];
          cv += dvc[cidx];
        }
        vk = fmaf(ck, inv_cnt, vk);
        vv = fmaf(cv, inv_cnt, vv);
      }
      store_out(dk, obase + d, vk, g.out_f32);
      store_out(dv, obase + d, vv, g.out_f32);
    }
  }
}

cudaError_t launch_fine_bwd_dq(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                               const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                               const float* dqc, void* dq, cudaStream_t st) {
  dim3 grid(g.N, g.Hq, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    size_t smb = BwdSmem<128>::dq_bytes;
    if ((e = cudaFuncSetAttribute(fine_bwd_dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_bwd_dq_kernel<128><<<grid, 256, smb, st>>>(q, k, v, d_o, lse, delta, row_ptr, col_idx, dqc, g, dq);
  } else {
    size_t smb = BwdSmem<64>::dq_bytes;
    if ((e = cudaFuncSetAttribute(fine_bwd_dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_bwd_dq_kernel<64><<<grid, 256, smb, st>>>(q, k, v, d_o, lse, delta, row_ptr, col_idx, dqc, g, dq);
  }
  return cudaGetLastError();
}

cudaError_t launch_fine_bwd_dkv(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                const float* lse, const float* delta, const int* col_ptr, const int* row_idx,
                                const float* dkc, const float* dvc, void* dk, void* dv, cudaStream_t st) {
  dim3 grid(g.N, g.Hkv, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    size_t smb = BwdSmem<128>::dkv_bytes;
    if ((e = cudaFuncSetAttribute(fine_bwd_dkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_bwd_dkv_kernel<128><<<grid, 256, smb, st>>>(q, k, v, d_o, lse, delta, col_ptr, row_idx, dkc, dvc, g, dk, dv);
  } else {
    size_t smb = BwdSmem<64>::dkv_bytes;
    if ((e = cudaFuncSetAttribute(fine_bwd_dkv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_bwd_dkv_kernel<64><<<grid, 256, smb, st>>>(q, k, v, d_o, lse, delta, col_ptr, row_idx, dkc, dvc, g, dk, dv);
  }
  return cudaGetLastError();
}

}  // namespace vsa2
