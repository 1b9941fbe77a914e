// Router block scores (paper Eq. 6-7): P_r = MeanPool_{GxG}(softmax(Q_r K_r^T * scale)).
// Two passes over the pooled keys, as in the paper's kernel description (Sec. 2.2 "Kernel
// Implementation"): pass 1 accumulates the row log-sum-exp, pass 2 recomputes the scores,
// applies the softmax and pools G x G sub-blocks on chip, so P^_r never reaches memory.
#include "wmma_tile.cuh"

namespace vsa2 {

constexpr int kRT = 128;   // router rows (and keys) per tile

// Shared memory: Qs [128][D+8] bf16, Ks [128][D+8] bf16, S [128][132] fp32.
template <int D>
struct RouterSmem {
  static constexpr int LDQ = D + 8;
  static constexpr int LDS = kRT + 4;
  static constexpr size_t bytes = 2 * (size_t)kRT * LDQ * sizeof(bf16) + (size_t)kRT * LDS * sizeof(float);
};

// grid (ceil(N*G/128), Hq, batch), 256 threads.
// PASS 1: lse_r[b,hq,row] = log sum_{valid keys} exp(s*scale).   PASS 2: writes P_r.
template <int D, int PASS>
__global__ void __launch_bounds__(256) router_kernel(const bf16* __restrict__ qr, const bf16* __restrict__ kr, Geo g,
                                                     float* __restrict__ lse_r, float* __restrict__ pr) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  using SM = RouterSmem<D>;
  bf16* Qs = reinterpret_cast<bf16*>(smem_raw);
  bf16* Ks = Qs + kRT * SM::LDQ;
  float* S = reinterpret_cast<float*>(Ks + kRT * SM::LDQ);
  __shared__ unsigned char kvalid[kRT];
  __shared__ unsigned char qvalid[kRT];
  __shared__ float row_lse[kRT];

  const int hq = blockIdx.y, b = blockIdx.z;
  const int hk = hq / g.rep;
  const int rows_total = g.N * g.G;
  const int row0 = blockIdx.x * kRT;
  const bf16* qbase = qr + ((size_t)(b * g.Hq + hq) * rows_total) * D;
  const bf16* kbase = kr + ((size_t)(b * g.Hkv + hk) * rows_total) * D;
  float* lse_base = lse_r + (size_t)(b * g.Hq + hq) * rows_total;
  constexpr int CH = D / 8;

  for (int c = threadIdx.x; c < kRT * CH; c += blockDim.x) {
    int r = c / CH, ch = c % CH;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row0 + r < rows_total) v = __ldg(reinterpret_cast<const uint4*>(qbase + (size_t)(row0 + r) * D + ch * 8));
    *reinterpret_cast<uint4*>(Qs + r * SM::LDQ + ch * 8) = v;
  }
  if (threadIdx.x < kRT) {
    int r = row0 + threadIdx.x;
    bool ok = r < rows_total && subcube_count(g, r / g.G, r % g.G) > 0;
    qvalid[threadIdx.x] = ok;
    if (PASS == 2) row_lse[threadIdx.x] = ok ? lse_base[r] : 0.f;
  }
  // pass-1 running statistics: thread t owns row t/2, column half t%2
  float m_run = -INFINITY, l_run = 0.f;
  const int my_row = threadIdx.x >> 1, my_half = threadIdx.x & 1;

  for (int k0 = 0; k0 < rows_total; k0 += kRT) {
    __syncthreads();
    for (int c = threadIdx.x; c < kRT * CH; c += blockDim.x) {
      int r = c / CH, ch = c % CH;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (k0 + r < rows_total) v = __ldg(reinterpret_cast<const uint4*>(kbase + (size_t)(k0 + r) * D + ch * 8));
      *reinterpret_cast<uint4*>(Ks + r * SM::LDQ + ch * 8) = v;
    }
    if (threadIdx.x < kRT) {
      int r = k0 + threadIdx.x;
      kvalid[threadIdx.x] = r < rows_total && subcube_count(g, r / g.G, r % g.G) > 0;
    }
    __syncthreads();
    tile_gemm<kRT, kRT, D, false, true, false>(Qs, SM::LDQ, Ks, SM::LDQ, S, SM::LDS);
    __syncthreads();
    if (PASS == 1) {
      const float* srow = S + my_row * SM::LDS + my_half * 64;
      float mx = -INFINITY;
      for (int c = 0; c < 64; ++c)
        if (kvalid[my_half * 64 + c]) mx = fmaxf(mx, srow[c] * g.scale);
      if (mx > -INFINITY) {
        float m_new = fmaxf(m_run, mx);
        float acc = 0.f;
        for (int c = 0; c < 64; ++c)
          if (kvalid[my_half * 64 + c]) acc += __expf(srow[c] * g.scale - m_new);
        l_run = l_run * __expf(m_run - m_new) + acc;
        m_run = m_new;
      }
    } else {
      // exp in place, then pool: each thread sums G x G entries of one (query cube, key cube) pair
      for (int e = threadIdx.x; e < kRT * kRT; e += blockDim.x) {
        int r = e / kRT, c = e % kRT;
        float p = 0.f;
        if (qvalid[r] && kvalid[c]) p = __expf(S[r * SM::LDS + c] * g.scale - row_lse[r]);
        S[r * SM::LDS + c] = p;
      }
      __syncthreads();
      const int TC = kRT / g.G;     // cubes per tile side
      for (int e = threadIdx.x; e < TC * TC; e += blockDim.x) {
        int ci = e / TC, cj = e % TC;
        int qi = row0 / g.G + ci, kj = k0 / g.G + cj;
        if (qi >= g.N || kj >= g.N) continue;
        float acc = 0.f;
        int gi = 0;
        for (int a = 0; a < g.G; ++a) {
          gi += qvalid[ci * g.G + a];
          const float* srow = S + (ci * g.G + a) * SM::LDS + cj * g.G;
          for (int c = 0; c < g.G; ++c) acc += srow[c];
        }
        pr[((size_t)(b * g.Hq + hq) * g.N + qi) * g.N + kj] = gi > 0 ? acc / ((float)gi * (float)g.G) : 0.f;
      }
    }
  }
  if (PASS == 1) {
    // merge the two column halves of a row (adjacent lanes)
    float m_o = __shfl_xor_sync(0xffffffffu, m_run, 1);
    float l_o = __shfl_xor_sync(0xffffffffu, l_run, 1);
    float m = fmaxf(m_run, m_o);
    float l = 0.f;
    if (m > -INFINITY) l = l_run * __expf(m_run - m) + l_o * __expf(m_o - m);
    if (my_half == 0 && row0 + my_row < rows_total) lse_base[row0 + my_row] = (l > 0.f) ? m + __logf(l) : 0.f;
  }
}

cudaError_t launch_router_scores(const Geo& g, const bf16* qr, const bf16* kr, float* lse_r, float* pr,
                                 cudaStream_t st) {
  const int rows_total = g.N * g.G;
  dim3 grid((rows_total + kRT - 1) / kRT, g.Hq, g.batch);
  cudaError_t e;
  if (g.D == 128) {
    size_t sm = RouterSmem<128>::bytes;
    if ((e = cudaFuncSetAttribute(router_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm))) return e;
    if ((e = cudaFuncSetAttribute(router_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm))) return e;
    {
      ProfScope ps(VSA2_KERNEL_ROUTER_LSE, st, 1);
      router_kernel<128, 1><<<grid, 256, sm, st>>>(qr, kr, g, lse_r, pr);
    }
    ProfScope ps(VSA2_KERNEL_ROUTER_POOL, st, 1);
    router_kernel<128, 2><<<grid, 256, sm, st>>>(qr, kr, g, lse_r, pr);
  } else {
    size_t sm = RouterSmem<64>::bytes;
    if ((e = cudaFuncSetAttribute(router_kernel<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm))) return e;
    if ((e = cudaFuncSetAttribute(router_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm))) return e;
    {
      ProfScope ps(VSA2_KERNEL_ROUTER_LSE, st, 1);
      router_kernel<64, 1><<<grid, 256, sm, st>>>(qr, kr, g, lse_r, pr);
    }
    ProfScope ps(VSA2_KERNEL_ROUTER_POOL, st, 1);
    router_kernel<64, 2><<<grid, 256, sm, st>>>(qr, kr, g, lse_r, pr);
  }
  return cudaGetLastError();
}

}  // namespace vsa2
