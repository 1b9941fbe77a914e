// Forward of the coarse branch (paper Eq. 2-3): dense attention over the N pooled tokens of a head, TF32 products with
// fp32 accumulation and fp32 softmax statistics.  The operands are fp32 means of 64 (or 128) tokens and the output feeds
// dGate = sum_d dO * O_c in the backward, which needs better than bf16 operand precision (see the note in api.cu), so
// this small problem (1/B^2 of the dense FLOPs) stays on mma.sync TF32 instead of the bf16 tcgen05 path.
//
// One warp owns 16 query rows for the whole key loop: its Q fragments, the running maximum / sum of its rows and its
// 16 x D output accumulators live in registers; a CTA of four warps (64 query rows) shares key / value tiles of 32 pooled
// tokens, double-buffered with cp.async; P goes from the score accumulators to the A operand of the second product through
// a warp-private strip of shared memory (the TF32 fragment layouts of C and A differ).  Two CTAs fit an SM.
#include "common.cuh"

namespace vsa2 {

namespace {

constexpr int kCfRows = 64;      // query rows per CTA (16 per warp)
constexpr int kCfKeys = 32;      // keys per tile
constexpr int kCfThreads = 128;

template <int D>
struct CoarseFwdSmem {
  static constexpr int LDK = D + 4;     // pitch = 4 mod 32 floats: the B fragments of Q K^T read 32 different banks
  static constexpr int LDV = D + 8;     // pitch = 8 mod 32 floats: the B fragments of P V read 32 different banks
  static constexpr int LDP = kCfKeys + 4;
  static constexpr size_t k_tile = (size_t)kCfKeys * LDK * sizeof(float);
  static constexpr size_t v_tile = (size_t)kCfKeys * LDV * sizeof(float);
  static constexpr size_t p_strip = (size_t)16 * LDP * sizeof(float);
  static constexpr size_t bytes = 2 * (k_tile + v_tile) + 4 * p_strip;
};

__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// rows j0 .. j0 + 31 of K_c and V_c (rows beyond the last pooled token repeat it; their scores are masked)
template <int D>
__device__ __forceinline__ void issue_tile(float* ks, float* vs, const float* kc, const float* vc, int j0, int N) {
  using S = CoarseFwdSmem<D>;
  constexpr int CH = D / 4;                       // 16-byte chunks per row
  for (int e = threadIdx.x; e < kCfKeys * CH; e += kCfThreads) {
    const int r = e / CH, c = e % CH;
    const int row = min(j0 + r, N - 1);
    cp_async16(ks + r * S::LDK + c * 4, kc + (size_t)row * D + c * 4);
    cp_async16(vs + r * S::LDV + c * 4, vc + (size_t)row * D + c * 4);
  }
}

// grid (ceil(N / 64), Hq, batch), 128 threads
template <int D>
__global__ void __launch_bounds__(kCfThreads, 2)
coarse_fwd_mma_kernel(const float* __restrict__ qc, const float* __restrict__ kc, const float* __restrict__ vc, Geo g,
                      float* __restrict__ oc_hat, float* __restrict__ lse_c) {
  using S = CoarseFwdSmem<D>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* kbuf = reinterpret_cast<float*>(smem_raw);                       // [2][32][LDK]
  float* vbuf = kbuf + 2 * kCfKeys * S::LDK;                              // [2][32][LDV]
  float* pbuf = vbuf + 2 * kCfKeys * S::LDV;                              // [4 warps][16][LDP]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gq = lane >> 2, tq = lane & 3;                                // fragment coordinates of this lane
  const int hq = blockIdx.y, b = blockIdx.z, hk = hq / g.rep;
  const int N = g.N;
  const size_t qoff = (size_t)(b * g.Hq + hq) * N * D, koff = (size_t)(b * g.Hkv + hk) * N * D;
  const float* kbase = kc + koff;
  const float* vbase = vc + koff;
  const int row_lo = blockIdx.x * kCfRows + warp * 16 + gq, row_hi = row_lo + 8;   // this lane's two query rows
  const float sl2 = g.scale * 1.4426950408889634f;                        // scores in log2 units

  issue_tile<D>(kbuf, vbuf, kbase, vbase, 0, N);
  cp_async_commit();

  // Q fragments of the warp's 16 rows, all D / 8 contraction steps, converted once
  uint32_t qf[D / 8][4];
  {
    const float* q_lo = qc + qoff + (size_t)min(row_lo, N - 1) * D;
    const float* q_hi = qc + qoff + (size_t)min(row_hi, N - 1) * D;
#pragma unroll
    for (int ks = 0; ks < D / 8; ++ks) {
      qf[ks][0] = to_tf32(__ldg(q_lo + ks * 8 + tq));
      qf[ks][1] = to_tf32(__ldg(q_hi + ks * 8 + tq));
      qf[ks][2] = to_tf32(__ldg(q_lo + ks * 8 + tq + 4));
      qf[ks][3] = to_tf32(__ldg(q_hi + ks * 8 + tq + 4));
    }
  }
  float o[D / 8][4];
#pragma unroll
  for (int n = 0; n < D / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;       // running maximum (log2 units) and sum
  float* pw = pbuf + warp * 16 * S::LDP;

  const int n_tiles = (N + kCfKeys - 1) / kCfKeys;
  for (int t = 0; t < n_tiles; ++t) {
    const int j0 = t * kCfKeys;
    const float* ks_ = kbuf + (t & 1) * kCfKeys * S::LDK;
    const float* vs_ = vbuf + (t & 1) * kCfKeys * S::LDV;
    if (t + 1 < n_tiles) {
      issue_tile<D>(kbuf + ((t + 1) & 1) * kCfKeys * S::LDK, vbuf + ((t + 1) & 1) * kCfKeys * S::LDV, kbase, vbase,
                    j0 + kCfKeys, N);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();                         // tile t has landed for every thread

    // S[16, 32] = Q K^T
    float s[kCfKeys / 8][4];
#pragma unroll
    for (int n = 0; n < kCfKeys / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 8; ++ks) {
#pragma unroll
      for (int n = 0; n < kCfKeys / 8; ++n) {
        const float* kp = ks_ + (n * 8 + gq) * S::LDK + ks * 8 + tq;
        mma_tf32(s[n], qf[ks], to_tf32(kp[0]), to_tf32(kp[4]));
      }
    }
    // online softmax of the two rows of this lane (columns 2 tq, 2 tq + 1 of every 8-key group; the quad shares a row)
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int n = 0; n < kCfKeys / 8; ++n) {
      const int col = j0 + n * 8 + 2 * tq;
      s[n][0] = col < N ? s[n][0] * sl2 : -INFINITY;
      s[n][1] = col + 1 < N ? s[n][1] * sl2 : -INFINITY;
      s[n][2] = col < N ? s[n][2] * sl2 : -INFINITY;
      s[n][3] = col + 1 < N ? s[n][3] * sl2 : -INFINITY;
      mx_lo = fmaxf(mx_lo, fmaxf(s[n][0], s[n][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[n][2], s[n][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);   // finite: every tile holds a valid key
    const float a_lo = exp2f(m_lo - mn_lo), a_hi = exp2f(m_hi - mn_hi);
    float ps_lo = 0.f, ps_hi = 0.f;
#pragma unroll
    for (int n = 0; n < kCfKeys / 8; ++n) {
      const float p0 = exp2f(s[n][0] - mn_lo), p1 = exp2f(s[n][1] - mn_lo);
      const float p2 = exp2f(s[n][2] - mn_hi), p3 = exp2f(s[n][3] - mn_hi);
      ps_lo += p0 + p1;
      ps_hi += p2 + p3;
      *reinterpret_cast<float2*>(pw + gq * S::LDP + n * 8 + 2 * tq) = make_float2(p0, p1);
      *reinterpret_cast<float2*>(pw + (gq + 8) * S::LDP + n * 8 + 2 * tq) = make_float2(p2, p3);
    }
    ps_lo += __shfl_xor_sync(0xffffffffu, ps_lo, 1);
    ps_lo += __shfl_xor_sync(0xffffffffu, ps_lo, 2);
    ps_hi += __shfl_xor_sync(0xffffffffu, ps_hi, 1);
    ps_hi += __shfl_xor_sync(0xffffffffu, ps_hi, 2);
    l_lo = l_lo * a_lo + ps_lo;
    l_hi = l_hi * a_hi + ps_hi;
    m_lo = mn_lo;
    m_hi = mn_hi;
#pragma unroll
    for (int n = 0; n < D / 8; ++n) {
      o[n][0] *= a_lo; o[n][1] *= a_lo;
      o[n][2] *= a_hi; o[n][3] *= a_hi;
    }
    __syncwarp();                            // the strip of P is complete

    // O[16, D] += P V
#pragma unroll
    for (int ks = 0; ks < kCfKeys / 8; ++ks) {
      uint32_t pf[4];
      pf[0] = to_tf32(pw[gq * S::LDP + ks * 8 + tq]);
      pf[1] = to_tf32(pw[(gq + 8) * S::LDP + ks * 8 + tq]);
      pf[2] = to_tf32(pw[gq * S::LDP + ks * 8 + tq + 4]);
      pf[3] = to_tf32(pw[(gq + 8) * S::LDP + ks * 8 + tq + 4]);
#pragma unroll
      for (int n = 0; n < D / 8; ++n) {
        const float* vp = vs_ + (ks * 8 + tq) * S::LDV + n * 8 + gq;
        mma_tf32(o[n], pf, to_tf32(vp[0]), to_tf32(vp[4 * S::LDV]));
      }
    }
    __syncthreads();                         // everyone is done with tile t before its buffer is refilled
  }

  const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
  if (row_lo < N) {
    float* dst = oc_hat + qoff + (size_t)row_lo * D;
#pragma unroll
    for (int n = 0; n < D / 8; ++n)
      *reinterpret_cast<float2*>(dst + n * 8 + 2 * tq) = make_float2(o[n][0] * inv_lo, o[n][1] * inv_lo);
    if (tq == 0) lse_c[(size_t)(b * g.Hq + hq) * N + row_lo] = (m_lo + log2f(l_lo)) * 0.6931471805599453f;
  }
  if (row_hi < N) {
    float* dst = oc_hat + qoff + (size_t)row_hi * D;
#pragma unroll
    for (int n = 0; n < D / 8; ++n)
      *reinterpret_cast<float2*>(dst + n * 8 + 2 * tq) = make_float2(o[n][2] * inv_hi, o[n][3] * inv_hi);
    if (tq == 0) lse_c[(size_t)(b * g.Hq + hq) * N + row_hi] = (m_hi + log2f(l_hi)) * 0.6931471805599453f;
  }
}

}  // namespace

cudaError_t launch_coarse_fwd_mma(const Geo& g, const float* qc, const float* kc, const float* vc, float* oc_hat,
                                  float* lse_c, cudaStream_t st) {
  dim3 grid((g.N + kCfRows - 1) / kCfRows, g.Hq, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    const size_t smb = CoarseFwdSmem<128>::bytes;
    if ((e = cudaFuncSetAttribute(coarse_fwd_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    coarse_fwd_mma_kernel<128><<<grid, kCfThreads, smb, st>>>(qc, kc, vc, g, oc_hat, lse_c);
  } else {
    const size_t smb = CoarseFwdSmem<64>::bytes;
    if ((e = cudaFuncSetAttribute(coarse_fwd_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    coarse_fwd_mma_kernel<64><<<grid, kCfThreads, smb, st>>>(qc, kc, vc, g, oc_hat, lse_c);
  }
  return cudaGetLastError();
}

}  // namespace vsa2
