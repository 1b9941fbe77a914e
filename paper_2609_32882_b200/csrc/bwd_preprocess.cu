// First step of the backward pass: the per-token quantities of the gated merge (paper Eq. 14) and of the fine softmax
// (Eq. 12) that the dQ and dK/dV passes (fine_bwd_tc.cu) and the coarse backward read:
//   delta = rowsum(dO * O_f), dGate = rowsum(dO * O_c), dO_c_hat[n] = sum_{l in n} gate_l dO_l
// HBM-bound: one pass over dO, O (and the bf16 rounding residual of O).
#include "common.cuh"

namespace vsa2 {

// One thread per (64-token block, 16-byte channel chunk): it walks the block's tokens four at a time (12 loads in flight),
// keeps its 8 channels of sum_l gate_l dO_l and of O_c in registers, and the D / 8 threads of a block reduce the two row sums
// of a token with shuffles -- no shared memory, and a warp's loads cover whole token rows.
template <int D>
__global__ void __launch_bounds__(128) bwd_preprocess_kernel(const bf16* __restrict__ d_o, const void* __restrict__ o,
                                                             const bf16* __restrict__ o_res,
                                                             const float* __restrict__ gate,
                                                             const float* __restrict__ oc_hat, Geo g,
                                                             float* __restrict__ delta, float* __restrict__ dgate,
                                                             float* __restrict__ d_oc_hat) {
  constexpr int CH = D / 8;            // threads per block = 16-byte chunks of a token row
  constexpr int BLOCKS = 128 / CH;     // 64-token blocks per CTA
  constexpr int TOK = 4;               // tokens in flight per thread
  const int i = blockIdx.x * BLOCKS + threadIdx.x / CH, ch = threadIdx.x % CH, hq = blockIdx.y, b = blockIdx.z;
  if (i >= g.N) return;                // (whole shuffle groups leave together)
  const int lane = threadIdx.x & 31;
  const unsigned group_mask = (CH == 16 ? 0xffffu : 0xffu) << (lane & ~(CH - 1));
  const size_t bhq = (size_t)b * g.Hq + hq;
  // text blocks (i >= Nvid) take no part in the coarse branch or the gate: only delta is formed for them
  const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && gate != nullptr && !block_is_text(g, i);
  float ocv[8], acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) ocv[e] = acc[e] = 0.f;
  if (coarse) {
    const float4* p4 = reinterpret_cast<const float4*>(oc_hat + (bhq * g.Nvid + i) * D + ch * 8);
    const float4 x = __ldg(p4), y = __ldg(p4 + 1);
    ocv[0] = x.x; ocv[1] = x.y; ocv[2] = x.z; ocv[3] = x.w;
    ocv[4] = y.x; ocv[5] = y.y; ocv[6] = y.z; ocv[7] = y.w;
  }
  for (int p0 = 0; p0 < kBlockTokens; p0 += TOK) {
    int l[TOK];
    float gt[TOK];
    uint4 dv[TOK], ob[TOK], rb[TOK];
    float4 of[TOK][2];
#pragma unroll
    for (int u = 0; u < TOK; ++u) {
      l[u] = block_token(g, i, p0 + u);
      gt[u] = 0.f;
      dv[u] = ob[u] = rb[u] = make_uint4(0, 0, 0, 0);
      of[u][0] = of[u][1] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l[u] >= 0) {
        const size_t base = (bhq * g.S + l[u]) * D + ch * 8;
        dv[u] = __ldg(reinterpret_cast<const uint4*>(d_o + base));
        if (g.out_f32) {
          of[u][0] = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(o) + base));
          of[u][1] = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(o) + base + 4));
        } else {
          ob[u] = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(o) + base));
          if (o_res != nullptr) rb[u] = __ldg(reinterpret_cast<const uint4*>(o_res + base));
        }
        if (coarse) gt[u] = __ldg(gate + bhq * g.L + l[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < TOK; ++u) {
      float ov[8], dd[8];
      const __nv_bfloat162* d2 = reinterpret_cast<const __nv_bfloat162*>(&dv[u]);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(d2[e]);
        dd[2 * e] = f.x; dd[2 * e + 1] = f.y;
      }
      if (g.out_f32) {
        ov[0] = of[u][0].x; ov[1] = of[u][0].y; ov[2] = of[u][0].z; ov[3] = of[u][0].w;
        ov[4] = of[u][1].x; ov[5] = of[u][1].y; ov[6] = of[u][1].z; ov[7] = of[u][1].w;
      } else {
        const __nv_bfloat162* o2 = reinterpret_cast<const __nv_bfloat162*>(&ob[u]);
        const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(&rb[u]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(o2[e]), r = __bfloat1622float2(r2[e]);     // (no residual: rb is zero)
          ov[2 * e] = f.x + r.x; ov[2 * e + 1] = f.y + r.y;
        }
      }
      float s_oo = 0.f, s_oc = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        s_oo = fmaf(dd[e], ov[e], s_oo);
        s_oc = fmaf(dd[e], ocv[e], s_oc);
        acc[e] = fmaf(gt[u], dd[e], acc[e]);
      }
#pragma unroll
      for (int off = CH / 2; off >= 1; off >>= 1) {
        s_oo += __shfl_xor_sync(group_mask, s_oo, off);
        s_oc += __shfl_xor_sync(group_mask, s_oc, off);
      }
      if (ch == 0 && l[u] >= 0) {
        delta[bhq * g.S + l[u]] = s_oo - gt[u] * s_oc;     // rowsum(dO * (O - gate*O_c)) = rowsum(dO * O_f)
        if (dgate != nullptr && coarse) dgate[bhq * g.L + l[u]] = s_oc;
      }
    }
  }
  if (coarse) {
    float4* dst = reinterpret_cast<float4*>(d_oc_hat + (bhq * g.Nvid + i) * D + ch * 8);
    dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
}

cudaError_t launch_bwd_preprocess(const Geo& g, const bf16* d_o, const void* o, const bf16* o_res, const float* gate,
                                  const float* oc_hat, float* delta, float* dgate, float* d_oc_hat, cudaStream_t st) {
  const int blocks = 128 / (g.D / 8);
  dim3 grid((g.N + blocks - 1) / blocks, g.Hq, g.batch);
  if (g.D == 128) bwd_preprocess_kernel<128><<<grid, 128, 0, st>>>(d_o, o, o_res, gate, oc_hat, g, delta, dgate, d_oc_hat);
  else bwd_preprocess_kernel<64><<<grid, 128, 0, st>>>(d_o, o, o_res, gate, oc_hat, g, delta, dgate, d_oc_hat);
  return cudaGetLastError();
}

}  // namespace vsa2
