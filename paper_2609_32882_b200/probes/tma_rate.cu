// TMA throughput probe: pairs of 16 KB cube tiles into a ring, 148 CTAs, various addressing modes.
#include <cstdio>
#include <cstdlib>
#include <vector>
#include "tmap.cuh"
#include "tc05.cuh"
using namespace vsa2;
constexpr int SLOTS = 6;
constexpr uint32_t SLOT = 32768;
struct Bars { uint64_t full[SLOTS], empty[SLOTS]; int abort_flag; };

__device__ __forceinline__ void bulk_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(tc::smem_u32(dst)), "l"(src), "r"(bytes), "r"(tc::smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(tc::smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(tc::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__global__ void __launch_bounds__(64, 1) probe(const __grid_constant__ CUtensorMap tm5, const __grid_constant__ CUtensorMap tm3,
                                               const unsigned char* base, Geo g, int heads, int mode, int tiles, long long* out) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  Bars* bars = reinterpret_cast<Bars*>(smem + SLOTS * SLOT);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    bars->abort_flag = 0;
    for (int s = 0; s < SLOTS; ++s) { tc::mbar_init(&bars->full[s], 1); tc::mbar_init(&bars->empty[s], 1); }
    tc::fence_barrier_init();
  }
  __syncthreads();
  long long t_start = clock64(), issue_clk = 0;
  if (warp == 0) {
    uint32_t rng = blockIdx.x * 2654435761u + 12345u;
    for (int t = 0; t < tiles; ++t) {
      const uint32_t s = t % SLOTS, par = (t / SLOTS) & 1;
      int ok = 1;
      if (lane == 0) {
        ok = tc::mbar_wait(&bars->empty[s], par ^ 1, &bars->abort_flag);
        if (ok) tc::mbar_expect_tx(&bars->full[s], SLOT);
      }
      if (!__shfl_sync(0xffffffffu, ok, 0)) break;
      rng = rng * 1664525u + 1013904223u;
      const int h = (blockIdx.x + t / 64) % heads;
      // two nearby-but-distinct cubes (like a selected pair)
      const int j0 = (rng >> 8) % g.N, j1 = (j0 + 1 + ((rng >> 4) & 7)) % g.N;
      const long long c0 = clock64();
      if (mode == 0) {            // 5-D raster, 4 lanes
        if (lane < 4) {
          const int j = (lane & 1) ? j1 : j0, hh = lane >> 1;
          int jt, jh, jw; cube_coords(g, j, jt, jh, jw);
          tc::tma_load_5d(smem + s * SLOT + (2 * hh + (lane & 1)) * 8192, &tm5, &bars->full[s], hh * 64, jw * g.Bw, jh * g.Bh, jt * g.Bt, h);
        }
      } else if (mode == 1) {     // 5-D raster, lane 0 issues all four
        if (lane == 0) {
          for (int q = 0; q < 4; ++q) {
            const int j = (q & 1) ? j1 : j0, hh = q >> 1;
            int jt, jh, jw; cube_coords(g, j, jt, jh, jw);
            tc::tma_load_5d(smem + s * SLOT + (2 * hh + (q & 1)) * 8192, &tm5, &bars->full[s], hh * 64, jw * g.Bw, jh * g.Bh, jt * g.Bt, h);
          }
        }
      } else if (mode == 2) {     // 3-D cube-major [BH*N][64][128], 4 lanes
        if (lane < 4) {
          const int j = (lane & 1) ? j1 : j0, hh = lane >> 1;
          tma_load_3d(smem + s * SLOT + (2 * hh + (lane & 1)) * 8192, &tm3, &bars->full[s], hh * 64, 0, h * g.N + j);
        }
      } else if (mode == 3) {     // 1-D bulk copies of 16 KB (pre-swizzled image), 2 lanes
        if (lane < 2) {
          const int j = lane ? j1 : j0;
          bulk_1d(smem + s * SLOT + lane * 16384, base + ((size_t)h * g.N + j) * 16384, 16384, &bars->full[s]);
        }
      } else if (mode == 4) {     // 1-D bulk copies of 8 KB, 4 lanes
        if (lane < 4) {
          const int j = (lane & 1) ? j1 : j0, hh = lane >> 1;
          bulk_1d(smem + s * SLOT + lane * 8192, base + ((size_t)h * g.N + j) * 16384 + hh * 8192, 8192, &bars->full[s]);
        }
      }
      __syncwarp();
      issue_clk += clock64() - c0;
    }
  } else if (lane == 0) {
    for (int t = 0; t < tiles; ++t) {
      const uint32_t s = t % SLOTS, par = (t / SLOTS) & 1;
      if (!tc::mbar_wait(&bars->full[s], par, &bars->abort_flag)) break;
      tc::mbar_arrive(&bars->empty[s]);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) { out[2 * blockIdx.x] = clock64() - t_start; }
  if (threadIdx.x == 0) out[2 * blockIdx.x + 1] = issue_clk;
}

int main(int argc, char** argv) {
  Geo g{};
  g.batch = 1; g.Hq = g.Hkv = 4; g.rep = 1; g.D = 128; g.T = 21; g.H = 45; g.W = 80; g.L = g.T * g.H * g.W;
  g.Bt = g.Bh = g.Bw = 4; g.Nt = 6; g.Nh = 12; g.Nw = 20; g.N = 1440;
  const int heads = argc > 1 ? atoi(argv[1]) : 4;
  g.Hq = g.Hkv = heads;
  const size_t bytes = (size_t)heads * g.N * 16384;   // >= raster size (padded)
  unsigned char* d; cudaMalloc(&d, bytes); cudaMemset(d, 0, bytes);
  CUtensorMap tm5, tm3;
  if (!make_cube_tmap(&tm5, d, g, heads)) { printf("tmap5 failed\n"); return 1; }
  {
    EncodeTiledFn fn = encode_tiled_fn();
    cuuint64_t dims[3] = {128, 64, (cuuint64_t)heads * g.N};
    cuuint64_t strides[2] = {256, 16384};
    cuuint32_t box[3] = {64, 64, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (fn(&tm3, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, d, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) { printf("tmap3 failed\n"); return 1; }
  }
  long long* out; cudaMalloc(&out, 148 * 2 * sizeof(long long));
  const size_t smb = SLOTS * SLOT + 1024 + 1024;
  cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb);
  const int tiles = 4000;
  const char* names[5] = {"5-D raster, 4 lanes", "5-D raster, 1 lane", "3-D cube-major, 4 lanes", "1-D bulk 2 x 16 KB", "1-D bulk 4 x 8 KB"};
  for (int rep = 0; rep < 2; ++rep)
    for (int mode = 0; mode < 5; ++mode) {
      probe<<<148, 64, smb>>>(tm5, tm3, d, g, heads, mode, tiles, out);
      cudaError_t e = cudaDeviceSynchronize();
      if (e != cudaSuccess) { printf("mode %d: %s\n", mode, cudaGetErrorString(e)); return 1; }
      std::vector<long long> h(296);
      cudaMemcpy(h.data(), out, 296 * sizeof(long long), cudaMemcpyDeviceToHost);
      double tot = 0, iss = 0;
      for (int i = 0; i < 148; ++i) { tot += h[2 * i]; iss += h[2 * i + 1]; }
      if (rep) printf("%-26s heads %d: %7.1f clk per 32 KB pair per SM (issue %6.1f clk)  -> %.2f TB/s aggregate at 1.965 GHz\n", names[mode], heads,
             tot / 148 / tiles, iss / 148 / tiles, 32768.0 * 148 / (tot / 148 / tiles) * 1.965e9 / 1e12);
    }
  return 0;
}
