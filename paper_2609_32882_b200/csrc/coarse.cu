// Coarse branch on the pooled tokens (paper Eq. 2-3): P_c = softmax(Q_c K_c^T * scale),
// O_c_hat = P_c V_c, and its backward.  Dense attention over N cubes in fp32; 1/B^2 of the
// dense FLOPs (appendix "Sparsity Computation").
#include "common.cuh"

namespace vsa2 {

constexpr int kCR = 16;   // stationary rows per CTA
constexpr int kCT = 64;   // streamed rows per tile

template <int D>
struct CoarseSmem {
  static constexpr int LDT = D + 1;
  // a0, a1: [16][D]; t0, t1: [64][D+1]; w0, w1: [16][64]
  static constexpr size_t floats = 2 * kCR * D + 2 * kCT * LDT + 2 * kCR * kCT + 4 * kCR + 2 * kCT;
  static constexpr size_t bytes = floats * sizeof(float);
};

// out[r][j] = sum_d a[r][d] * t[j][d]   (16 x 64 dots of length D), 256 threads
template <int D>
__device__ __forceinline__ void dots16x64(const float* a, const float* t, float* out) {
  constexpr int LDT = D + 1;
  const int j = threadIdx.x & 63, r0 = (threadIdx.x >> 6) * 4;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
  for (int d = 0; d < D; ++d) {
    float tv = t[j * LDT + d];
#pragma unroll
    for (int r = 0; r < 4; ++r) acc[r] = fmaf(a[(r0 + r) * D + d], tv, acc[r]);
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) out[(r0 + r) * kCT + j] = acc[r];
}

// acc[r] += sum_j w[r0+r][j] * t[j][d]  for this thread's column d and its rows
template <int D>
__device__ __forceinline__ void accum16(float (&acc)[kCR * D / 256], const float* w, const float* t) {
  constexpr int LDT = D + 1, RPT = kCR * D / 256;
  const int d = threadIdx.x % D, r0 = (threadIdx.x / D) * RPT;
#pragma unroll 4
  for (int j = 0; j < kCT; ++j) {
    float tv = t[j * LDT + d];
#pragma unroll
    for (int r = 0; r < RPT; ++r) acc[r] = fmaf(w[(r0 + r) * kCT + j], tv, acc[r]);
  }
}

template <int D>
__device__ __forceinline__ void load_rows(float* dst, int ld, const float* src, int row0, int nrows, int limit) {
  for (int e = threadIdx.x; e < nrows * D; e += blockDim.x) {
    int r = e / D, d = e % D;
    dst[r * ld + d] = (row0 + r < limit) ? __ldg(src + (size_t)(row0 + r) * D + d) : 0.f;
  }
}

// grid (ceil(N/16), Hq, batch), 256 threads.  Online softmax over key tiles of 64 cubes.
template <int D>
__global__ void __launch_bounds__(256) coarse_fwd_kernel(const float* __restrict__ qc, const float* __restrict__ kc,
                                                         const float* __restrict__ vc, Geo g,
                                                         float* __restrict__ oc_hat, float* __restrict__ lse_c) {
  extern __shared__ __align__(16) float sm[];
  using SM = CoarseSmem<D>;
  float* qs = sm;                       // [16][D]
  float* ks = qs + 2 * kCR * D;         // [64][D+1]
  float* vs = ks + kCT * SM::LDT;       // [64][D+1]
  float* s = vs + kCT * SM::LDT;        // [16][64]
  float* row_m = s + 2 * kCR * kCT;     // [16]
  float* row_l = row_m + kCR;           // [16]
  float* row_a = row_l + kCR;           // [16]
  constexpr int RPT = kCR * D / 256;
  const int hq = blockIdx.y, b = blockIdx.z, hk = hq / g.rep;
  const int i0 = blockIdx.x * kCR;
  const size_t qoff = (size_t)(b * g.Hq + hq) * g.N * D, koff = (size_t)(b * g.Hkv + hk) * g.N * D;
  load_rows<D>(qs, D, qc + qoff, i0, kCR, g.N);
  if (threadIdx.x < kCR) { row_m[threadIdx.x] = -INFINITY; row_l[threadIdx.x] = 0.f; }
  float acc[RPT];
#pragma unroll
  for (int r = 0; r < RPT; ++r) acc[r] = 0.f;
  const int r0 = (threadIdx.x / D) * RPT;
  for (int j0 = 0; j0 < g.N; j0 += kCT) {
    __syncthreads();
    load_rows<D>(ks, SM::LDT, kc + koff, j0, kCT, g.N);
    load_rows<D>(vs, SM::LDT, vc + koff, j0, kCT, g.N);
    __syncthreads();
    dots16x64<D>(qs, ks, s);
    __syncthreads();
    // softmax bookkeeping: warp w owns rows 2w, 2w+1; each lane two columns
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rr = 0; rr < 2; ++rr) {
      int r = warp * 2 + rr;
      float x0 = (j0 + lane < g.N) ? s[r * kCT + lane] * g.scale : -INFINITY;
      float x1 = (j0 + lane + 32 < g.N) ? s[r * kCT + lane + 32] * g.scale : -INFINITY;
      float mx = fmaxf(x0, x1);
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float m_old = row_m[r], m_new = fmaxf(m_old, mx);
      float p0 = expf(x0 - m_new), p1 = expf(x1 - m_new);
      float ps = p0 + p1;
      for (int o = 16; o; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      s[r * kCT + lane] = p0;
      s[r * kCT + lane + 32] = p1;
      __syncwarp();
      if (lane == 0) {
        float a = expf(m_old - m_new);
        row_a[r] = a;
        row_l[r] = row_l[r] * a + ps;
        row_m[r] = m_new;
      }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RPT; ++r) acc[r] *= row_a[r0 + r];
    accum16<D>(acc, s, vs);
  }
  __syncthreads();
  const int d = threadIdx.x % D;
#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    int i = i0 + r0 + r;
    if (i < g.N) oc_hat[qoff + (size_t)i * D + d] = acc[r] / row_l[r0 + r];
  }
  if (threadIdx.x < kCR && i0 + threadIdx.x < g.N)
    lse_c[(size_t)(b * g.Hq + hq) * g.N + i0 + threadIdx.x] = row_m[threadIdx.x] + logf(row_l[threadIdx.x]);
}

// Backward of the coarse attention, one stationary side per launch.
//   ROWS = true : stationary = 16 query cubes; streams key cubes; writes dQ_c and delta_c.
//   ROWS = false: stationary = 16 key cubes; streams query cubes; writes dK_c, dV_c (per query head).
// dS = P * (dP - delta_c), P = exp(S*scale - lse_c), dP = dO_c_hat V_c^T, delta_c = rowsum(dO_c_hat * O_c_hat).
template <int D, bool ROWS>
__global__ void __launch_bounds__(256) coarse_bwd_kernel(const float* __restrict__ qc, const float* __restrict__ kc,
                                                         const float* __restrict__ vc, const float* __restrict__ oc_hat,
                                                         const float* __restrict__ lse_c, const float* __restrict__ d_oc,
                                                         Geo g, float* __restrict__ delta_c, float* __restrict__ out0,
                                                         float* __restrict__ out1) {
  extern __shared__ __align__(16) float sm[];
  using SM = CoarseSmem<D>;
  float* a0 = sm;                        // stationary operand for the score dots  [16][D]
  float* a1 = a0 + kCR * D;              // stationary operand for the dP dots     [16][D]
  float* t0 = a1 + kCR * D;              // streamed tile for the score dots       [64][D+1]
  float* t1 = t0 + kCT * SM::LDT;        // streamed tile for the dP dots          [64][D+1]
  float* w0 = t1 + kCT * SM::LDT;        // P  (or dS)                             [16][64]
  float* w1 = w0 + kCR * kCT;            // dS                                     [16][64]
  float* st_lse = w1 + kCR * kCT;        // [16] per stationary row
  float* st_delta = st_lse + kCR;        // [16]
  float* tl_lse = st_delta + 3 * kCR;    // [64] per streamed row
  float* tl_delta = tl_lse + kCT;        // [64]
  constexpr int RPT = kCR * D / 256;
  const int hq = blockIdx.y, b = blockIdx.z, hk = hq / g.rep;
  const int s0 = blockIdx.x * kCR;
  const size_t qoff = (size_t)(b * g.Hq + hq) * g.N * D, koff = (size_t)(b * g.Hkv + hk) * g.N * D;
  const size_t roff = (size_t)(b * g.Hq + hq) * g.N;
  if (ROWS) {
    load_rows<D>(a0, D, qc + qoff, s0, kCR, g.N);
    load_rows<D>(a1, D, d_oc + qoff, s0, kCR, g.N);
    __syncthreads();
    // delta_c of the stationary rows: warp w rows 2w, 2w+1
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int rr = 0; rr < 2; ++rr) {
      int r = warp * 2 + rr, i = s0 + r;
      float acc = 0.f;
      if (i < g.N)
        for (int d = lane; d < D; d += 32) acc += a1[r * D + d] * __ldg(oc_hat + qoff + (size_t)i * D + d);
      for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (lane == 0) {
        st_delta[r] = acc;
        st_lse[r] = i < g.N ? lse_c[roff + i] : 0.f;
        if (i < g.N) delta_c[roff + i] = acc;
      }
    }
  } else {
    load_rows<D>(a0, D, kc + koff, s0, kCR, g.N);
    load_rows<D>(a1, D, vc + koff, s0, kCR, g.N);
  }
  float acc0[RPT], acc1[RPT];
#pragma unroll
  for (int r = 0; r < RPT; ++r) { acc0[r] = 0.f; acc1[r] = 0.f; }
  for (int j0 = 0; j0 < g.N; j0 += kCT) {
    __syncthreads();
    if (ROWS) {
      load_rows<D>(t0, SM::LDT, kc + koff, j0, kCT, g.N);
      load_rows<D>(t1, SM::LDT, vc + koff, j0, kCT, g.N);
    } else {
      load_rows<D>(t0, SM::LDT, qc + qoff, j0, kCT, g.N);
      load_rows<D>(t1, SM::LDT, d_oc + qoff, j0, kCT, g.N);
      if (threadIdx.x < kCT) {
        int i = j0 + threadIdx.x;
        tl_lse[threadIdx.x] = i < g.N ? lse_c[roff + i] : 0.f;
        tl_delta[threadIdx.x] = i < g.N ? delta_c[roff + i] : 0.f;
      }
    }
    __syncthreads();
    dots16x64<D>(a0, t0, w0);   // scores (stationary x streamed)
    dots16x64<D>(a1, t1, w1);   // dP
    __syncthreads();
    for (int e = threadIdx.x; e < kCR * kCT; e += blockDim.x) {
      int r = e / kCT, c = e % kCT;
      bool ok = (s0 + r < g.N) && (j0 + c < g.N);
      float lse = ROWS ? st_lse[r] : tl_lse[c];
      float dl = ROWS ? st_delta[r] : tl_delta[c];
      float p = ok ? expf(w0[e] * g.scale - lse) : 0.f;
      float ds = p * (w1[e] - dl) * g.scale;
      w0[e] = p;
      w1[e] = ds;
    }
    __syncthreads();
    if (ROWS) {
      accum16<D>(acc0, w1, t0);            // dQ_c += dS K_c
    } else {
      accum16<D>(acc0, w1, t0);            // dK_c += dS^T Q_c
      accum16<D>(acc1, w0, t1);            // dV_c += P^T dO_c_hat
    }
  }
  const int d = threadIdx.x % D, r0 = (threadIdx.x / D) * RPT;
#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    int i = s0 + r0 + r;
    if (i < g.N) {
      out0[qoff + (size_t)i * D + d] = acc0[r];
      if (!ROWS) out1[qoff + (size_t)i * D + d] = acc1[r];
    }
  }
}

cudaError_t launch_coarse_fwd(const Geo& g, const float* qc, const float* kc, const float* vc, float* oc_hat,
                              float* lse_c, cudaStream_t st) {
  dim3 grid((g.N + kCR - 1) / kCR, g.Hq, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    size_t smb = CoarseSmem<128>::bytes;
    if ((e = cudaFuncSetAttribute(coarse_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    coarse_fwd_kernel<128><<<grid, 256, smb, st>>>(qc, kc, vc, g, oc_hat, lse_c);
  } else {
    size_t smb = CoarseSmem<64>::bytes;
    if ((e = cudaFuncSetAttribute(coarse_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    coarse_fwd_kernel<64><<<grid, 256, smb, st>>>(qc, kc, vc, g, oc_hat, lse_c);
  }
  return cudaGetLastError();
}

// dqc, dkc, dvc [B,Hq,N,D] (dkc, dvc per QUERY head; the group sum happens where they are consumed);
// delta_c [B,Hq,N] is scratch supplied by the caller.
template <int D>
static cudaError_t coarse_bwd_t(const Geo& g, const float* qc, const float* kc, const float* vc, const float* oc_hat,
                                const float* lse_c, const float* d_oc, float* delta_c, float* dqc, float* dkc,
                                float* dvc, cudaStream_t st) {
  dim3 grid((g.N + kCR - 1) / kCR, g.Hq, g.batch);
  size_t smb = CoarseSmem<D>::bytes;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(coarse_bwd_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
  if ((e = cudaFuncSetAttribute(coarse_bwd_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
  coarse_bwd_kernel<D, true><<<grid, 256, smb, st>>>(qc, kc, vc, oc_hat, lse_c, d_oc, g, delta_c, dqc, nullptr);
  coarse_bwd_kernel<D, false><<<grid, 256, smb, st>>>(qc, kc, vc, oc_hat, lse_c, d_oc, g, delta_c, dkc, dvc);
  return cudaGetLastError();
}

cudaError_t launch_coarse_bwd(const Geo& g, const float* qc, const float* kc, const float* vc, const float* oc_hat,
                              const float* lse_c, const float* d_oc_hat, float* delta_c, float* dqc, float* dkc,
                              float* dvc, cudaStream_t st) {
  if (g.D == 128) return coarse_bwd_t<128>(g, qc, kc, vc, oc_hat, lse_c, d_oc_hat, delta_c, dqc, dkc, dvc, st);
  return coarse_bwd_t<64>(g, qc, kc, vc, oc_hat, lse_c, d_oc_hat, delta_c, dqc, dkc, dvc, st);
}

}  // namespace vsa2
