// Mean pooling over cubes (coarse branch, paper Eq. 1) and over router sub-cubes (Eq. 5).
// HBM-bound: every token row is read once with 16-byte loads.
// (one cube decode per thread: this file keeps the reciprocal form of the index divisions, which measured 7 % faster here)
#define VSA2_RECIPROCAL_DIVMOD 1
#include "common.cuh"

namespace vsa2 {

// One thread per (cube, 16-byte channel chunk): it reads the cube's tokens sub-cube by sub-cube (8 loads in flight for the
// 2 x 2 x 2 router pool), so no tile is staged in shared memory and a warp's loads cover whole 256-byte token rows.
//   xr [b, h, N*G, D] bf16 : fp32 sum along w, then h, then t (each left to right; padding positions add +0), IEEE fp32
//                            division by the valid count, rounded to bf16 (nearest even).
//   xc [b, h, N, D]   fp32 : sum of the sub-cube sums / count.
// Up to three tensors per launch (grid.y runs over the heads of all of them).
struct PoolJob {
  const bf16* x;
  bf16* xr;
  float* xc;
  int heads;
};
struct PoolJobs {
  PoolJob job[3];
  int n;
};

__device__ __forceinline__ void add8(float (&acc)[8], const float (&v)[8], bool first) {
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = first ? v[i] : __fadd_rn(acc[i], v[i]);
}
__device__ __forceinline__ void load8(const bf16* base, int t, int h, int w, const Geo& g, int D, float (&f)[8]) {
  uint4 v = make_uint4(0, 0, 0, 0);
  if (t < g.T && h < g.H && w < g.W) v = __ldg(reinterpret_cast<const uint4*>(base + (size_t)((t * g.H + h) * g.W + w) * D));
  const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 x = __bfloat1622float2(h2[i]);
    f[2 * i] = x.x;
    f[2 * i + 1] = x.y;
  }
}

template <int D, bool R222>
__global__ void __launch_bounds__(128) pool_kernel(PoolJobs jobs, Geo g) {
  constexpr int CH = D / 8;            // 16-byte chunks of a token row
  constexpr int CUBES = 128 / CH;      // cubes per CTA
  int h = blockIdx.y;
  PoolJob jb = jobs.job[0];
  if (jobs.n > 1 && h >= jb.heads) {
    h -= jb.heads;
    jb = jobs.job[1];
    if (jobs.n > 2 && h >= jb.heads) {
      h -= jb.heads;
      jb = jobs.job[2];
    }
  }
  const int n = blockIdx.x * CUBES + threadIdx.x / CH, ch = threadIdx.x % CH, b = blockIdx.z;
  if (n >= g.N) return;
  const size_t bh = (size_t)b * jb.heads + h;
  const bf16* base = jb.x + bh * (size_t)g.S * D + ch * 8;
  int nt, nh, nw;
  cube_coords(g, n, nt, nh, nw);
  float tot[8];
  for (int gsub = 0; gsub < g.G; ++gsub) {
    const int gw = gsub % g.Gw, r = gsub / g.Gw, gh = r % g.Gh, gt = r / g.Gh;
    const int t0 = nt * g.Bt + gt * g.Rt, h0 = nh * g.Bh + gh * g.Rh, w0 = nw * g.Bw + gw * g.Rw;
    float ts[8];
    if (R222) {
      float v[8][8];
#pragma unroll
      for (int k = 0; k < 8; ++k) load8(base, t0 + (k >> 2), h0 + ((k >> 1) & 1), w0 + (k & 1), g, D, v[k]);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        ts[i] = __fadd_rn(__fadd_rn(__fadd_rn(v[0][i], v[1][i]), __fadd_rn(v[2][i], v[3][i])),
                          __fadd_rn(__fadd_rn(v[4][i], v[5][i]), __fadd_rn(v[6][i], v[7][i])));
    } else {
      for (int it = 0; it < g.Rt; ++it) {
        float hs[8];
        for (int ih = 0; ih < g.Rh; ++ih) {
          float ws[8];
          for (int iw = 0; iw < g.Rw; ++iw) {
            float v[8];
            load8(base, t0 + it, h0 + ih, w0 + iw, g, D, v);
            add8(ws, v, iw == 0);
          }
          add8(hs, ws, ih == 0);
        }
        add8(ts, hs, it == 0);
      }
    }
    add8(tot, ts, gsub == 0);
    if (jb.xr != nullptr) {
      const int cnt = subcube_count(g, n, gsub);
      uint4 o = make_uint4(0, 0, 0, 0);
      if (cnt > 0) {
        const float c = (float)cnt;
        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) o2[i] = __floats2bfloat162_rn(__fdiv_rn(ts[2 * i], c), __fdiv_rn(ts[2 * i + 1], c));
      }
      *reinterpret_cast<uint4*>(jb.xr + ((bh * g.N + n) * g.G + gsub) * D + ch * 8) = o;
    }
  }
  if (jb.xc != nullptr) {
    const float cnt = (float)cube_count(g, n);
    float* dst = jb.xc + (bh * g.N + n) * D + ch * 8;
    float m[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) m[i] = cnt > 0.f ? tot[i] / cnt : 0.f;
    *reinterpret_cast<float4*>(dst) = make_float4(m[0], m[1], m[2], m[3]);
    *reinterpret_cast<float4*>(dst + 4) = make_float4(m[4], m[5], m[6], m[7]);
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

static cudaError_t launch_pool_jobs(const Geo& g, const PoolJobs& jobs, cudaStream_t st) {
  int heads = 0;
  for (int i = 0; i < jobs.n; ++i) heads += jobs.job[i].heads;
  const int cubes = 128 / (g.D / 8);
  dim3 grid((g.N + cubes - 1) / cubes, heads, g.batch);
  const bool r222 = g.Rt == 2 && g.Rh == 2 && g.Rw == 2;
  if (g.D == 128) {
    if (r222) pool_kernel<128, true><<<grid, 128, 0, st>>>(jobs, g);
    else pool_kernel<128, false><<<grid, 128, 0, st>>>(jobs, g);
  } else {
    if (r222) pool_kernel<64, true><<<grid, 128, 0, st>>>(jobs, g);
    else pool_kernel<64, false><<<grid, 128, 0, st>>>(jobs, g);
  }
  return cudaGetLastError();
}

cudaError_t launch_pool(const Geo& g, const bf16* x, int heads, bf16* xr, float* xc, cudaStream_t st) {
  PoolJobs jobs{};
  jobs.job[0] = PoolJob{x, xr, xc, heads};
  jobs.n = 1;
  return launch_pool_jobs(g, jobs, st);
}

// router means of Q and K (Eq. 5) in one launch
cudaError_t launch_pool_router(const Geo& g, const bf16* q, const bf16* k, bf16* qr, bf16* kr, cudaStream_t st) {
  PoolJobs jobs{};
  jobs.job[0] = PoolJob{q, qr, nullptr, g.Hq};
  jobs.job[1] = PoolJob{k, kr, nullptr, g.Hkv};
  jobs.n = 2;
  return launch_pool_jobs(g, jobs, st);
}

// cube means of Q, K and V (Eq. 1) in one launch
cudaError_t launch_pool_coarse(const Geo& g, const bf16* q, const bf16* k, const bf16* v, float* qc, float* kc, float* vc,
                               cudaStream_t st) {
  PoolJobs jobs{};
  jobs.job[0] = PoolJob{q, nullptr, qc, g.Hq};
  jobs.job[1] = PoolJob{k, nullptr, kc, g.Hkv};
  jobs.job[2] = PoolJob{v, nullptr, vc, g.Hkv};
  jobs.n = 3;
  return launch_pool_jobs(g, jobs, st);
}

}  // namespace vsa2
