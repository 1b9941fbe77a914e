// Mean pooling of one tensor over cubes (coarse branch, paper Eq. 1) and over router
// sub-cubes (Eq. 5).  HBM-bound: every cube tile is read once with 16-byte loads.
#include "common.cuh"

namespace vsa2 {

// One CTA per (cube, head, batch).  The cube's 64 x D bf16 tile is staged in shared memory as
// fp32; padding positions hold +0.
//   xc [b, h, N, D]   fp32 : sum over valid tokens / count.
//   xr [b, h, N*G, D] bf16 : fp32 sum along w, then h, then t (each left to right), IEEE fp32
//                            division by the valid count, rounded to bf16 (nearest even).
template <int D>
__global__ void __launch_bounds__(256) pool_kernel(const bf16* __restrict__ x, int heads, Geo g,
                                                   bf16* __restrict__ xr, float* __restrict__ xc) {
  __shared__ float tile[kBlockTokens][D];
  const int n = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const size_t bh = (size_t)b * heads + h;
  const bf16* base = x + bh * (size_t)g.S * D;
  int nt, nh, nw;
  cube_coords(g, n, nt, nh, nw);
  constexpr int CH = D / 8;
  for (int c = threadIdx.x; c < kBlockTokens * CH; c += blockDim.x) {
    int p = c / CH, ch = c % CH;
    int l = cube_token(g, nt, nh, nw, p);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (l >= 0) v = __ldg(reinterpret_cast<const uint4*>(base + (size_t)l * D + ch * 8));
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h2[i]);
      tile[p][ch * 8 + 2 * i] = f.x;
      tile[p][ch * 8 + 2 * i + 1] = f.y;
    }
  }
  __syncthreads();
  if (xc != nullptr) {
    const float cnt = (float)cube_count(g, n);
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
      float s = 0.f;
#pragma unroll 8
      for (int p = 0; p < kBlockTokens; ++p) s += tile[p][d];
      xc[(bh * g.N + n) * D + d] = cnt > 0.f ? s / cnt : 0.f;
    }
  }
  if (xr != nullptr) {
    for (int idx = threadIdx.x; idx < g.G * (D / 2); idx += blockDim.x) {
      int gsub = idx / (D / 2), d = (idx % (D / 2)) * 2;
      int gw = gsub % g.Gw;
      int r = gsub / g.Gw;
      int gh = r % g.Gh;
      int gt = r / g.Gh;
      float t0 = 0.f, t1 = 0.f;
      for (int it = 0; it < g.Rt; ++it) {
        float h0 = 0.f, h1 = 0.f;
        for (int ih = 0; ih < g.Rh; ++ih) {
          int p0 = ((gt * g.Rt + it) * g.Bh + (gh * g.Rh + ih)) * g.Bw + gw * g.Rw;
          float w0 = tile[p0][d], w1 = tile[p0][d + 1];
          for (int iw = 1; iw < g.Rw; ++iw) {
            w0 = __fadd_rn(w0, tile[p0 + iw][d]);
            w1 = __fadd_rn(w1, tile[p0 + iw][d + 1]);
          }
          h0 = ih ? __fadd_rn(h0, w0) : w0;
          h1 = ih ? __fadd_rn(h1, w1) : w1;
        }
        t0 = it ? __fadd_rn(t0, h0) : h0;
        t1 = it ? __fadd_rn(t1, h1) : h1;
      }
      int cnt = subcube_count(g, n, gsub);
      float m0 = 0.f, m1 = 0.f;
      if (cnt > 0) {
        m0 = __fdiv_rn(t0, (float)cnt);
        m1 = __fdiv_rn(t1, (float)cnt);
      }
      __nv_bfloat162 o = __floats2bfloat162_rn(m0, m1);
      *reinterpret_cast<__nv_bfloat162*>(xr + ((bh * g.N + n) * g.G + gsub) * D + d) = o;
    }
  }
}

// Cube-major copy of a raster tensor (paper Sec. 2.2 "Permutation") and back.  One CTA per (cube, head, batch):
//   forward: y[b, h, n * B + p, :] = x[b, h, token(n, p), :], zero where position p of cube n lies outside the grid
//   inverse: x[b, h, token(n, p), :] = y[b, h, n * B + p, :] for the positions inside the grid
// The attention kernels never need this copy (they address cubes through tensor maps over the raster layout); it is for
// callers whose surrounding code works in the cube-major layout.
template <int D>
__global__ void __launch_bounds__(256) permute_kernel(const bf16* __restrict__ src, int heads, Geo g, int inverse,
                                                      bf16* __restrict__ dst) {
  const int n = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const size_t bh = (size_t)b * heads + h;
  const int B = g.Bt * g.Bh * g.Bw;
  int nt, nh, nw;
  cube_coords(g, n, nt, nh, nw);
  constexpr int CH = D / 8;
  for (int c = threadIdx.x; c < B * CH; c += blockDim.x) {
    const int p = c / CH, ch = c % CH;
    const int l = cube_token(g, nt, nh, nw, p);
    const size_t raster = (bh * g.S + (size_t)max(l, 0)) * D + ch * 8;
    const size_t cubed = ((bh * g.N + n) * B + p) * (size_t)D + ch * 8;
    if (!inverse) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (l >= 0) v = __ldg(reinterpret_cast<const uint4*>(src + raster));
      *reinterpret_cast<uint4*>(dst + cubed) = v;
    } else if (l >= 0) {
      *reinterpret_cast<uint4*>(dst + raster) = __ldg(reinterpret_cast<const uint4*>(src + cubed));
    }
  }
}

cudaError_t launch_permute(const Geo& g, const bf16* src, int heads, bool inverse, bf16* dst, cudaStream_t st) {
  dim3 grid(g.N, heads, g.batch);
  if (g.D == 128) permute_kernel<128><<<grid, 256, 0, st>>>(src, heads, g, inverse ? 1 : 0, dst);
  else permute_kernel<64><<<grid, 256, 0, st>>>(src, heads, g, inverse ? 1 : 0, dst);
  return cudaGetLastError();
}

cudaError_t launch_pool(const Geo& g, const bf16* x, int heads, bf16* xr, float* xc, cudaStream_t st) {
  dim3 grid(g.N, heads, g.batch);
  if (g.D == 128) pool_kernel<128><<<grid, 256, 0, st>>>(x, heads, g, xr, xc);
  else pool_kernel<64><<<grid, 256, 0, st>>>(x, heads, g, xr, xc);
  return cudaGetLastError();
}

}  // namespace vsa2
