// probe: raw tcgen05 throughput of the instruction mix used by the attention kernels
#include <cstdio>
#include <cuda_runtime.h>
#include "tc05.cuh"
using namespace vsa2;
__global__ void __launch_bounds__(128, 1) rate_kernel(int iters, int mode, long long* cycles) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  __shared__ __align__(8) uint64_t bar;
  __shared__ __align__(8) uint64_t bar2[3];
  __shared__ __align__(8) uint64_t bar_done;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  for (int i = threadIdx.x; i < 160 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u;
  if (threadIdx.x == 0) { abort_flag = 0; tc::mbar_init(&bar, 1); for (int i = 0; i < 3; ++i) tc::mbar_init(&bar2[i], 1); tc::mbar_init(&bar_done, 1); tc::fence_barrier_init(); tc::mbar_arrive(&bar_done); }
  if (threadIdx.x < 32) { tc::tmem_alloc(&tmem_base_s, 512); tc::tmem_relinquish(); }
  tc::fence_proxy_async_smem();
  tc::tc_fence_before(); __syncthreads(); tc::tc_fence_after();
  uint32_t tb = tmem_base_s;
  if (threadIdx.x == 0) {
    uint32_t base = tc::smem_u32(smem);
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
      if (mode == 0 || mode == 2) {   // S-type: M128 N64 K-major x K-major, 8 k-steps
        uint32_t id = tc::idesc_bf16(128, 64, false, false);
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t a = base + (ks / 4) * 16384 + (ks % 4) * 32, b = base + 65536 + (ks / 4) * 8192 + (ks % 4) * 32;
          tc::mma_ss(tb + (it & 1) * 64, tc::smem_desc_sw128(a, 16, 1024), tc::smem_desc_sw128(b, 16, 1024), id, ks > 0);
        }
      }
      if (mode == 1 || mode == 2) {   // PV-type: M128 N64 MN-major x MN-major
        uint32_t id = tc::idesc_bf16(128, 64, true, true);
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t a = base + 32768 + (ks / 4) * 8192 + (ks % 4) * 2048, b = base + 98304 + ks * 2048;
          tc::mma_ss(tb + 128, tc::smem_desc_sw128(a, 16384, 1024), tc::smem_desc_sw128(b, 0, 1024), id, true);
        }
      }
      if (mode == 3) {                // N=128 K-major (router-like): M128 N128
        uint32_t id = tc::idesc_bf16(128, 128, false, false);
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t a = base + (ks / 4) * 16384 + (ks % 4) * 32, b = base + 65536 + (ks / 4) * 16384 + (ks % 4) * 32;
          tc::mma_ss(tb + (it & 1) * 128, tc::smem_desc_sw128(a, 16, 1024), tc::smem_desc_sw128(b, 16, 1024), id, ks > 0);
        }
      }
      if (mode >= 5 && mode <= 7) {   // M=64 variants, K-major: N = 64, 128, 256
        int n = mode == 5 ? 64 : mode == 6 ? 128 : 256;
        uint32_t id = tc::idesc_bf16(64, n, false, false);
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t a = base + (ks / 4) * 16384 + (ks % 4) * 32, b = base + 65536 + (ks / 4) * 32768 + (ks % 4) * 32;
          tc::mma_ss(tb + (it & 1) * 256, tc::smem_desc_sw128(a, 16, 1024), tc::smem_desc_sw128(b, 16, 1024), id, ks > 0);
        }
      }
      if (mode >= 8) {                // S-type 8 instr + sync ops: 8: +1 commit, 9: +3 commits, 10: +1 commit + 3 satisfied waits, 11: + wait for own commit each iter
        uint32_t id = tc::idesc_bf16(128, 64, false, false);
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t a = base + (ks / 4) * 16384 + (ks % 4) * 32, b = base + 65536 + (ks / 4) * 8192 + (ks % 4) * 32;
          tc::mma_ss(tb + (it & 1) * 64, tc::smem_desc_sw128(a, 16, 1024), tc::smem_desc_sw128(b, 16, 1024), id, ks > 0);
        }
        tc::mma_commit(&bar2[0]);
        if (mode == 9) { tc::mma_commit(&bar2[1]); tc::mma_commit(&bar2[2]); }
        if (mode == 10) { for (int w = 0; w < 3; ++w) tc::mbar_wait(&bar_done, 0, &abort_flag); }
        if (mode == 11) { tc::mbar_wait(&bar2[0], it & 1, &abort_flag); }
      }
      if (mode == 4) {                // N=256 K-major
        uint32_t id = tc::idesc_bf16(128, 256, false, false);
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t a = base + (ks / 4) * 16384 + (ks % 4) * 32, b = base + 65536 + (ks / 4) * 32768 + (ks % 4) * 32;
          tc::mma_ss(tb + (it & 1) * 256, tc::smem_desc_sw128(a, 16, 1024), tc::smem_desc_sw128(b, 16, 1024), id, ks > 0);
        }
      }
    }
    tc::mma_commit(&bar);
    tc::mbar_wait(&bar, 0, &abort_flag);
    long long t1 = clock64();
    cycles[blockIdx.x] = t1 - t0;
  }
  tc::tc_fence_before(); __syncthreads();
  if (threadIdx.x < 32) tc::tmem_dealloc(tb, 512);
}
int main() {
  long long* d; cudaMalloc(&d, 148 * 8);
  cudaFuncSetAttribute(rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  const char* names[] = {"S-type M128 N64 K-major (8 instr)", "PV-type M128 N64 MN-major (8 instr)", "S+PV (16 instr)", "M128 N128 K-major (8 instr)", "M128 N256 K-major (8 instr)", "M64 N64", "M64 N128", "M64 N256", "S8 + 1 commit", "S8 + 3 commits", "S8 + commit + 3 satisfied waits", "S8 + commit + wait own commit"};
  for (int grid : {148}) for (int mode : {0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11}) {
    int iters = 2000;
    rate_kernel<<<grid, 128, 200 * 1024>>>(10, mode, d); cudaDeviceSynchronize();
    rate_kernel<<<grid, 128, 200 * 1024>>>(iters, mode, d);
    cudaError_t e = cudaDeviceSynchronize();
    long long c[148]; cudaMemcpy(c, d, grid * 8, cudaMemcpyDeviceToHost);
    double flop = (mode == 2 ? 16 : 8) * 2.0 * ((mode >= 5 && mode <= 7) ? 64 : 128) * 16 * (mode == 3 || mode == 6 ? 128 : (mode == 4 || mode == 7) ? 256 : 64);
    printf("grid %3d %-40s err=%d cycles/iter %.1f  flop/clk/SM %.0f\n", grid, names[mode], (int)e, (double)c[0] / iters, flop * iters / c[0]);
  }
  return 0;
}
