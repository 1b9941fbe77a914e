// First step of the backward pass: the per-token quantities of the gated merge (paper Eq. 14) and of the fine softmax
// (Eq. 12) that the dQ and dK/dV passes (fine_bwd_tc.cu) and the coarse backward read:
//   delta = rowsum(dO * O_f), dGate = rowsum(dO * O_c), dO_c_hat[n] = sum_{l in n} gate_l dO_l
// HBM-bound: one pass over dO, O (and the bf16 rounding residual of O).
#include "common.cuh"

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
  // text blocks (i >= Nvid) take no part in the coarse branch or the gate: only delta is formed for them
  const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && gate != nullptr && !block_is_text(g, i);
  const int r = threadIdx.x >> 2, qd = threadIdx.x & 3;
  constexpr int NCH = D / 32;          // 16-byte chunks (8 channels) per thread
  const int l = block_token(g, i, r);
  if (coarse)
    for (int d = threadIdx.x; d < D; d += blockDim.x) ocs[d] = oc_hat[(bhq * g.Nvid + i) * D + d];
  float s_oo = 0.f, s_oc = 0.f;
  const float gt = (coarse && l >= 0) ? gate[bhq * g.L + l] : 0.f;
  uint4 dv[NCH], ob[NCH], rb[NCH];
  float4 of[NCH][2];
  if (l >= 0) {
    const size_t base = (bhq * g.S + l) * D;
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
    delta[bhq * g.S + l] = s_oo - gt * s_oc;     // rowsum(dO * (O - gate*O_c)) = rowsum(dO * O_f)
    if (dgate != nullptr && coarse) dgate[bhq * g.L + l] = s_oc;
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
      d_oc_hat[(bhq * g.Nvid + i) * D + threadIdx.x] = tot;
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

}  // namespace vsa2
