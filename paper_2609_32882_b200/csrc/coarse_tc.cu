// Coarse branch on the pooled tokens (paper Eq. 2-3) and its backward with TF32 tensor-core tiles.
// The pooled tensors are fp32 means of 64 tokens; the products run as TF32 (10-bit mantissa) with fp32
// accumulation, softmax statistics in fp32.  Dense attention over N cubes: 1/B^2 of the dense FLOPs.
// Operands are rounded to TF32 once, when they are written to shared memory (tile loads, P and dS), so the
// fragment loads need no conversion; the k loop is the outer one so that the output tiles of a warp share
// the fragment of their common operand and their accumulation chains interleave.
#include <mma.h>

#include "common.cuh"

namespace vsa2 {

using namespace nvcuda;

constexpr int kCT = 64;    // rows per tile (queries and keys)
constexpr int kCoarseThreads = 512;   // 16 warps: one score tile, D/64 output tiles each

template <int D>
struct CoarseTc {
  static constexpr int LDX = D + 4;     // fp32 operand tiles
  static constexpr int LDS = kCT + 4;   // fp32 score tiles
  static constexpr size_t tile = (size_t)kCT * LDX * sizeof(float);
  static constexpr size_t score = (size_t)kCT * LDS * sizeof(float);
  static constexpr size_t fwd_bytes = 4 * tile + score + 3 * kCT * sizeof(float);          // Q, K, V, O, S
  static constexpr size_t bwd_bytes = 4 * tile + 2 * score + 4 * kCT * sizeof(float);      // 4 operand tiles, S, dP
};

typedef wmma::fragment<wmma::matrix_a, 16, 16, 8, wmma::precision::tf32, wmma::row_major> FragA;
typedef wmma::fragment<wmma::matrix_a, 16, 16, 8, wmma::precision::tf32, wmma::col_major> FragAT;
typedef wmma::fragment<wmma::matrix_b, 16, 16, 8, wmma::precision::tf32, wmma::row_major> FragB;
typedef wmma::fragment<wmma::matrix_b, 16, 16, 8, wmma::precision::tf32, wmma::col_major> FragBT;
typedef wmma::fragment<wmma::accumulator, 16, 16, 8, float> FragC;

__device__ __forceinline__ float tf32(float x) { return wmma::__float_to_tf32(x); }

// C[64 x 64] = A[64 x D] * B[64 x D]^T  (both row-major in shared memory, already TF32), 16 warps, one output tile
// each; the contraction is split into two halves with their own accumulators so that two dependent chains interleave
template <int D>
__device__ __forceinline__ void scores_64x64(const float* A, const float* B, float* C) {
  constexpr int LDX = D + 4, LDS = kCT + 4;
  const int warp = threadIdx.x >> 5;
  const int tm = warp >> 2, tn = warp & 3;
  FragC acc0, acc1;
  wmma::fill_fragment(acc0, 0.f);
  wmma::fill_fragment(acc1, 0.f);
#pragma unroll 4
  for (int k = 0; k < D / 2; k += 8) {
    FragA a0, a1;
    FragBT b0, b1;
    wmma::load_matrix_sync(a0, A + tm * 16 * LDX + k, LDX);
    wmma::load_matrix_sync(b0, B + tn * 16 * LDX + k, LDX);
    wmma::load_matrix_sync(a1, A + tm * 16 * LDX + D / 2 + k, LDX);
    wmma::load_matrix_sync(b1, B + tn * 16 * LDX + D / 2 + k, LDX);
    wmma::mma_sync(acc0, a0, b0, acc0);
    wmma::mma_sync(acc1, a1, b1, acc1);
  }
#pragma unroll
  for (int i = 0; i < acc0.num_elements; ++i) acc0.x[i] += acc1.x[i];
  wmma::store_matrix_sync(C + tm * 16 * LDS + tn * 16, acc0, LDS, wmma::mem_row_major);
}

// acc tiles: this warp owns the D/64 consecutive output tiles (tm, tn0 .. tn0 + D/64 - 1) of a [64 x D] result, which
// share the W fragment.   TRANS_W = false: out += W[64 x 64] * X[64 x D];   TRANS_W = true: out += W^T * X
template <int D, bool TRANS_W>
__device__ __forceinline__ void accumulate_64xD(FragC (&acc)[D / 64], const float* W, const float* X) {
  constexpr int LDX = D + 4, LDS = kCT + 4, TN = D / 16, PER = D / 64;
  const int warp = threadIdx.x >> 5;
  const int tm = (warp * PER) / TN, tn0 = (warp * PER) % TN;
#pragma unroll
  for (int k = 0; k < kCT; k += 8) {
    FragA a;
    FragAT at;
    if constexpr (TRANS_W) wmma::load_matrix_sync(at, W + k * LDS + tm * 16, LDS);
    else wmma::load_matrix_sync(a, W + tm * 16 * LDS + k, LDS);
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      FragB b;
      wmma::load_matrix_sync(b, X + k * LDX + (tn0 + i) * 16, LDX);
      if constexpr (TRANS_W) wmma::mma_sync(acc[i], at, b, acc[i]);
      else wmma::mma_sync(acc[i], a, b, acc[i]);
    }
  }
}

template <int D>
__device__ __forceinline__ void load_tile(float* dst, const float* src, int row0, int limit) {
  constexpr int LDX = D + 4, CH = D / 4;
  for (int e = threadIdx.x; e < kCT * CH; e += blockDim.x) {
    const int r = e / CH, c = e % CH;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < limit) v = __ldg(reinterpret_cast<const float4*>(src + (size_t)(row0 + r) * D + c * 4));
    *reinterpret_cast<float4*>(dst + r * LDX + c * 4) = make_float4(tf32(v.x), tf32(v.y), tf32(v.z), tf32(v.w));
  }
}

// ---------------------------------------------------------------------------------------------- forward
// grid (ceil(N/64), Hq, batch), 512 threads
template <int D>
__global__ void __launch_bounds__(kCoarseThreads) coarse_fwd_tc_kernel(const float* __restrict__ qc, const float* __restrict__ kc,
                                                            const float* __restrict__ vc, Geo g,
                                                            float* __restrict__ oc_hat, float* __restrict__ lse_c) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  using C = CoarseTc<D>;
  float* Qs = reinterpret_cast<float*>(smem_raw);
  float* Ks = Qs + kCT * C::LDX;
  float* Vs = Ks + kCT * C::LDX;
  float* Os = Vs + kCT * C::LDX;
  float* S = Os + kCT * C::LDX;
  float* row_m = S + kCT * C::LDS;
  float* row_l = row_m + kCT;
  const int hq = blockIdx.y, b = blockIdx.z, hk = hq / g.rep;
  const int i0 = blockIdx.x * kCT;
  const size_t qoff = (size_t)(b * g.Hq + hq) * g.N * D, koff = (size_t)(b * g.Hkv + hk) * g.N * D;
  load_tile<D>(Qs, qc + qoff, i0, g.N);
  for (int e = threadIdx.x; e < kCT * C::LDX; e += blockDim.x) Os[e] = 0.f;
  if (threadIdx.x < kCT) { row_m[threadIdx.x] = -INFINITY; row_l[threadIdx.x] = 0.f; }
  const int r = threadIdx.x >> 3, qd = threadIdx.x & 7;   // 8 threads per row, 8 columns / D/8 channels each
  for (int j0 = 0; j0 < g.N; j0 += kCT) {
    __syncthreads();
    load_tile<D>(Ks, kc + koff, j0, g.N);
    load_tile<D>(Vs, vc + koff, j0, g.N);
    __syncthreads();
    scores_64x64<D>(Qs, Ks, S);
    __syncthreads();
    {
      float x[8];
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int col = qd * 8 + c;
        x[c] = (j0 + col < g.N) ? S[r * C::LDS + col] * g.scale : -INFINITY;
        mx = fmaxf(mx, x[c]);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      const float m_old = row_m[r], m_new = fmaxf(m_old, mx);
      float ps = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float p = __expf(x[c] - m_new);
        S[r * C::LDS + qd * 8 + c] = tf32(p);
        ps += p;
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      ps += __shfl_xor_sync(0xffffffffu, ps, 4);
      const float alpha = __expf(m_old - m_new);
      for (int c = 0; c < D / 8; ++c) Os[r * C::LDX + qd * (D / 8) + c] *= alpha;
      __syncwarp();
      if (qd == 0) { row_m[r] = m_new; row_l[r] = row_l[r] * alpha + ps; }
    }
    __syncthreads();
    {
      // O += P V with the accumulators round-tripping through shared memory (rows were just rescaled there)
      constexpr int TN = D / 16, PER = D / 64;
      const int warp = threadIdx.x >> 5;
      const int tm = (warp * PER) / TN, tn0 = (warp * PER) % TN;
      FragC acc[PER];
#pragma unroll
      for (int i = 0; i < PER; ++i)
        wmma::load_matrix_sync(acc[i], Os + tm * 16 * C::LDX + (tn0 + i) * 16, C::LDX, wmma::mem_row_major);
      accumulate_64xD<D, false>(acc, S, Vs);
#pragma unroll
      for (int i = 0; i < PER; ++i)
        wmma::store_matrix_sync(Os + tm * 16 * C::LDX + (tn0 + i) * 16, acc[i], C::LDX, wmma::mem_row_major);
    }
  }
  __syncthreads();
  const int i = i0 + r;
  if (i < g.N) {
    const float inv = 1.f / row_l[r];
    for (int c = 0; c < D / 8; ++c) {
      const int d = qd * (D / 8) + c;
      oc_hat[qoff + (size_t)i * D + d] = Os[r * C::LDX + d] * inv;
    }
    if (qd == 0) lse_c[(size_t)(b * g.Hq + hq) * g.N + i] = row_m[r] + __logf(row_l[r]);
  }
}

// ---------------------------------------------------------------------------------------------- backward
// ROWS = true : 64 query cubes stationary; streams key tiles; writes dQ_c and delta_c.
// ROWS = false: 64 key cubes stationary; streams query tiles; writes dK_c, dV_c (per query head).
// dS = P * (dP - delta_c) * scale, P = exp(S*scale - lse_c), dP = dO_c_hat V_c^T, delta_c = rowsum(dO_c_hat * O_c_hat).
template <int D, bool ROWS>
__global__ void __launch_bounds__(kCoarseThreads) coarse_bwd_tc_kernel(const float* __restrict__ qc, const float* __restrict__ kc,
                                                            const float* __restrict__ vc, const float* __restrict__ oc_hat,
                                                            const float* __restrict__ lse_c, const float* __restrict__ d_oc,
                                                            Geo g, float* __restrict__ delta_c, float* __restrict__ out0,
                                                            float* __restrict__ out1) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  using C = CoarseTc<D>;
  float* X0 = reinterpret_cast<float*>(smem_raw);   // stationary operand of the score product (Q or K)
  float* X1 = X0 + kCT * C::LDX;                    // stationary operand of the dP product (dO_c or V)
  float* Y0 = X1 + kCT * C::LDX;                    // streamed operand of the score product (K or Q)
  float* Y1 = Y0 + kCT * C::LDX;                    // streamed operand of the dP product (V or dO_c)
  float* S = Y1 + kCT * C::LDX;                     // scores -> P   [query][key]
  float* dP = S + kCT * C::LDS;                     // dP -> dS      [query][key]
  float* q_lse = dP + kCT * C::LDS;                 // per query row of the current (query) tile
  float* q_delta = q_lse + kCT;
  const int hq = blockIdx.y, b = blockIdx.z, hk = hq / g.rep;
  const int s0 = blockIdx.x * kCT;
  const size_t qoff = (size_t)(b * g.Hq + hq) * g.N * D, koff = (size_t)(b * g.Hkv + hk) * g.N * D;
  const size_t roff = (size_t)(b * g.Hq + hq) * g.N;
  const int r = threadIdx.x >> 3, qd = threadIdx.x & 7;
  if (ROWS) {
    load_tile<D>(X0, qc + qoff, s0, g.N);
    load_tile<D>(X1, d_oc + qoff, s0, g.N);
    __syncthreads();
    // delta_c of the stationary query rows
    float acc = 0.f;
    const int i = s0 + r;
    if (i < g.N)
      for (int c = 0; c < D / 8; ++c) {
        const int d = qd * (D / 8) + c;
        acc = fmaf(X1[r * C::LDX + d], __ldg(oc_hat + qoff + (size_t)i * D + d), acc);
      }
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    if (qd == 0) {
      q_delta[r] = acc;
      q_lse[r] = i < g.N ? lse_c[roff + i] : INFINITY;
      if (i < g.N) delta_c[roff + i] = acc;
    }
  } else {
    load_tile<D>(X0, kc + koff, s0, g.N);
    load_tile<D>(X1, vc + koff, s0, g.N);
  }
  FragC acc0[D / 64], acc1[D / 64];
#pragma unroll
  for (int i = 0; i < D / 64; ++i) { wmma::fill_fragment(acc0[i], 0.f); wmma::fill_fragment(acc1[i], 0.f); }

  for (int j0 = 0; j0 < g.N; j0 += kCT) {
    __syncthreads();
    if (ROWS) {
      load_tile<D>(Y0, kc + koff, j0, g.N);
      load_tile<D>(Y1, vc + koff, j0, g.N);
    } else {
      load_tile<D>(Y0, qc + qoff, j0, g.N);
      load_tile<D>(Y1, d_oc + qoff, j0, g.N);
      if (threadIdx.x < kCT) {
        const int i = j0 + threadIdx.x;
        q_lse[threadIdx.x] = i < g.N ? lse_c[roff + i] : INFINITY;
        q_delta[threadIdx.x] = i < g.N ? delta_c[roff + i] : 0.f;
      }
    }
    __syncthreads();
    // S[query][key], dP[query][key]
    if (ROWS) {
      scores_64x64<D>(X0, Y0, S);
      scores_64x64<D>(X1, Y1, dP);
    } else {
      scores_64x64<D>(Y0, X0, S);
      scores_64x64<D>(Y1, X1, dP);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < kCT * kCT; e += blockDim.x) {
      const int qi = e >> 6, ki = e & 63;
      const bool ok = ROWS ? (j0 + ki < g.N) : (s0 + ki < g.N);     // the key must exist (missing queries carry lse = +inf)
      const float p = ok ? __expf(S[qi * C::LDS + ki] * g.scale - q_lse[qi]) : 0.f;
      const float ds = p * (dP[qi * C::LDS + ki] - q_delta[qi]) * g.scale;
      S[qi * C::LDS + ki] = tf32(p);
      dP[qi * C::LDS + ki] = tf32(ds);
    }
    __syncthreads();
    if (ROWS) {
      accumulate_64xD<D, false>(acc0, dP, Y0);        // dQ_c += dS K_c
    } else {
      accumulate_64xD<D, true>(acc0, dP, Y0);         // dK_c += dS^T Q_c
      accumulate_64xD<D, true>(acc1, S, Y1);          // dV_c += P^T dO_c_hat
    }
  }
  // accumulators -> shared memory (operand tiles are idle) -> global
  __syncthreads();
  {
    constexpr int TN = D / 16, PER = D / 64;
    const int warp = threadIdx.x >> 5;
    const int tm = (warp * PER) / TN, tn0 = (warp * PER) % TN;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      wmma::store_matrix_sync(Y0 + tm * 16 * C::LDX + (tn0 + i) * 16, acc0[i], C::LDX, wmma::mem_row_major);
      if (!ROWS) wmma::store_matrix_sync(Y1 + tm * 16 * C::LDX + (tn0 + i) * 16, acc1[i], C::LDX, wmma::mem_row_major);
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < kCT * (D / 4); e += blockDim.x) {
    const int rr = e / (D / 4), c = e % (D / 4);
    const int i = s0 + rr;
    if (i >= g.N) continue;
    *reinterpret_cast<float4*>(out0 + qoff + (size_t)i * D + c * 4) = *reinterpret_cast<const float4*>(Y0 + rr * C::LDX + c * 4);
    if (!ROWS)
      *reinterpret_cast<float4*>(out1 + qoff + (size_t)i * D + c * 4) = *reinterpret_cast<const float4*>(Y1 + rr * C::LDX + c * 4);
  }
}

cudaError_t launch_coarse_fwd_tc(const Geo& g, const float* qc, const float* kc, const float* vc, float* oc_hat,
                                 float* lse_c, cudaStream_t st) {
  dim3 grid((g.N + kCT - 1) / kCT, g.Hq, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    const size_t smb = CoarseTc<128>::fwd_bytes;
    if ((e = cudaFuncSetAttribute(coarse_fwd_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    coarse_fwd_tc_kernel<128><<<grid, kCoarseThreads, smb, st>>>(qc, kc, vc, g, oc_hat, lse_c);
  } else {
    const size_t smb = CoarseTc<64>::fwd_bytes;
    if ((e = cudaFuncSetAttribute(coarse_fwd_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    coarse_fwd_tc_kernel<64><<<grid, kCoarseThreads, smb, st>>>(qc, kc, vc, g, oc_hat, lse_c);
  }
  return cudaGetLastError();
}

template <int D>
static cudaError_t coarse_bwd_tc_t(const Geo& g, const float* qc, const float* kc, const float* vc, const float* oc_hat,
                                   const float* lse_c, const float* d_oc, float* delta_c, float* dqc, float* dkc,
                                   float* dvc, cudaStream_t st) {
  dim3 grid((g.N + kCT - 1) / kCT, g.Hq, g.batch);
  const size_t smb = CoarseTc<D>::bwd_bytes;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(coarse_bwd_tc_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
  if ((e = cudaFuncSetAttribute(coarse_bwd_tc_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
  coarse_bwd_tc_kernel<D, true><<<grid, kCoarseThreads, smb, st>>>(qc, kc, vc, oc_hat, lse_c, d_oc, g, delta_c, dqc, nullptr);
  coarse_bwd_tc_kernel<D, false><<<grid, kCoarseThreads, smb, st>>>(qc, kc, vc, oc_hat, lse_c, d_oc, g, delta_c, dkc, dvc);
  return cudaGetLastError();
}

cudaError_t launch_coarse_bwd_tc(const Geo& g, const float* qc, const float* kc, const float* vc, const float* oc_hat,
                                 const float* lse_c, const float* d_oc_hat, float* delta_c, float* dqc, float* dkc,
                                 float* dvc, cudaStream_t st) {
  if (g.D == 128) return coarse_bwd_tc_t<128>(g, qc, kc, vc, oc_hat, lse_c, d_oc_hat, delta_c, dqc, dkc, dvc, st);
  return coarse_bwd_tc_t<64>(g, qc, kc, vc, oc_hat, lse_c, d_oc_hat, delta_c, dqc, dkc, dvc, st);
}

}  // namespace vsa2
