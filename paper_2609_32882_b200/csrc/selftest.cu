// Self-test of the tensor-core building blocks exactly as the attention kernels use them:
// cube tiles fetched by 5-D TMA into 128-byte-swizzled shared memory, one K-major x K-major product
// (S^T = K_pair Q^T) and one MN-major x MN-major product (O^T = V_pair^T P^T) with accumulators in
// tensor memory.  One CTA; results go back to global memory for a host-side comparison.
#include "common.cuh"
#include "tc05.cuh"
#include "tmap.cuh"

namespace vsa2 {

template <int D>
__global__ void __launch_bounds__(128) selftest_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                       const __grid_constant__ CUtensorMap tm_k,
                                                       const __grid_constant__ CUtensorMap tm_v, Geo g, int cq, int ca,
                                                       int cb, const bf16* __restrict__ pt_in, float* __restrict__ st_out,
                                                       float* __restrict__ ot_out, uint4* __restrict__ dump,
                                                       int* __restrict__ status) {
  constexpr int DH = D / 64;                 // 64-channel halves
  constexpr uint32_t SLAB = 64 * 128;        // one cube, 64 channels: 8 KB
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);   // swizzle atoms need 1 KB alignment
  unsigned char* kslot = smem;                        // [half][A | B] slabs
  unsigned char* qtile = kslot + 2 * DH * SLAB;       // [half] slabs
  unsigned char* vslot = qtile + DH * SLAB;           // [A half0 .. | B half0 ..] slabs
  unsigned char* ptile = vslot + 2 * DH * SLAB;       // P^T: 128 rows of 128 bytes
  __shared__ __align__(8) uint64_t bar_full, bar_s, bar_o;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    abort_flag = 0;
    tc::mbar_init(&bar_full, 1);
    tc::mbar_init(&bar_s, 1);
    tc::mbar_init(&bar_o, 1);
    tc::fence_barrier_init();
  }
  if (warp == 0) {
    tc::tmem_alloc(&tmem_base_s, 128);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  // P^T rows into the swizzled MN-major layout: 16-byte chunk c of row r lands at chunk (c ^ (r & 7))
  {
    const uint4* src = reinterpret_cast<const uint4*>(pt_in + (size_t)tid * 64);
#pragma unroll
    for (int c = 0; c < 8; ++c)
      *reinterpret_cast<uint4*>(ptile + tid * 128 + ((c ^ (tid & 7)) << 4)) = src[c];
  }
  tc::fence_proxy_async_smem();
  __syncthreads();

  int cqt, cqh, cqw, cat, cah, caw, cbt, cbh, cbw;
  cube_coords(g, cq, cqt, cqh, cqw);
  cube_coords(g, ca, cat, cah, caw);
  cube_coords(g, cb, cbt, cbh, cbw);
  if (tid == 0) {
    tc::mbar_expect_tx(&bar_full, 5 * DH * SLAB);
    for (int h = 0; h < DH; ++h) {
      tc::tma_load_5d(kslot + (2 * h + 0) * SLAB, &tm_k, &bar_full, h * 64, caw * g.Bw, cah * g.Bh, cat * g.Bt, 0);
      tc::tma_load_5d(kslot + (2 * h + 1) * SLAB, &tm_k, &bar_full, h * 64, cbw * g.Bw, cbh * g.Bh, cbt * g.Bt, 0);
      tc::tma_load_5d(qtile + h * SLAB, &tm_q, &bar_full, h * 64, cqw * g.Bw, cqh * g.Bh, cqt * g.Bt, 0);
      tc::tma_load_5d(vslot + (0 * DH + h) * SLAB, &tm_v, &bar_full, h * 64, caw * g.Bw, cah * g.Bh, cat * g.Bt, 0);
      tc::tma_load_5d(vslot + (1 * DH + h) * SLAB, &tm_v, &bar_full, h * 64, cbw * g.Bw, cbh * g.Bh, cbt * g.Bt, 0);
    }
    if (tc::mbar_wait(&bar_full, 0, &abort_flag)) {
      tc::tc_fence_after();
      // S^T[128 kv, 64 q] = K_pair[128, D] * Q[64, D]^T   (both operands K-major)
      constexpr uint32_t idesc_s = tc::idesc_bf16(128, 64, false, false);
      for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t a = tc::smem_u32(kslot) + (ks / 4) * 2 * SLAB + (ks % 4) * 32;
        uint32_t b = tc::smem_u32(qtile) + (ks / 4) * SLAB + (ks % 4) * 32;
        tc::mma_ss(tmem_base, tc::smem_desc_sw128(a, 16, 1024), tc::smem_desc_sw128(b, 16, 1024), idesc_s, ks > 0);
      }
      tc::mma_commit(&bar_s);
      // O^T[128 d, 64 q] = V_pair^T[128 d, 128 kv] * P^T[128 kv, 64 q]   (both operands MN-major)
      constexpr uint32_t idesc_o = tc::idesc_bf16(128, 64, true, true);
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t a = tc::smem_u32(vslot) + (ks / 4) * DH * SLAB + (ks % 4) * 2048;
        uint32_t b = tc::smem_u32(ptile) + ks * 2048;
        tc::mma_ss(tmem_base + 64, tc::smem_desc_sw128(a, DH == 2 ? SLAB : 0, 1024), tc::smem_desc_sw128(b, 0, 1024),
                   idesc_o, ks > 0);
      }
      tc::mma_commit(&bar_o);
    }
  }
  __syncthreads();
  bool ok = tc::mbar_wait(&bar_s, 0, &abort_flag) && tc::mbar_wait(&bar_o, 0, &abort_flag);
  tc::tc_fence_after();
  if (ok) {
    uint32_t r[32];
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
    for (int c0 = 0; c0 < 128; c0 += 32) {
      tc::tmem_ld32(lane_addr + c0, r);
      tc::tmem_ld_wait();
      float* dst = (c0 < 64 ? st_out : ot_out) + (size_t)tid * 64 + (c0 & 63);
      for (int c = 0; c < 32; ++c) dst[c] = __uint_as_float(r[c]);
    }
    for (int e = tid; e < 2 * DH * (int)SLAB / 16; e += blockDim.x) dump[e] = reinterpret_cast<const uint4*>(kslot)[e];
  } else if (tid == 0) {
    atomicExch(status, VSA2_ERR_DEVICE_TIMEOUT);
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem_base, 128);
}

// The give-up path of the attention kernels in isolation: a CTA allocates tensor memory, one role waits on an mbarrier
// that no role ever arrives at, with a limit of `limit_us` microseconds instead of the kernels' 2 s; the wait runs out,
// the role raises the CTA's abort flag, every thread leaves through the common exit, the status word receives
// VSA2_ERR_DEVICE_TIMEOUT and the tensor memory is released.  Nothing faults or hangs; the context stays usable.
__global__ void __launch_bounds__(128) selftest_timeout_kernel(unsigned limit_us, int* __restrict__ status,
                                                               unsigned long long* __restrict__ waited_ns) {
  __shared__ __align__(8) uint64_t never, other;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    abort_flag = 0;
    tc::mbar_init(&never, 1);
    tc::mbar_init(&other, 1);
    tc::fence_barrier_init();
  }
  if (warp == 0) {
    tc::tmem_alloc(&tmem_base_s, 128);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  if (tid == 32) {
    // the role whose producer never shows up
    const unsigned long long t0 = tc::global_timer_ns();
    const bool ok = tc::mbar_wait_ns(&never, 0, &abort_flag, (unsigned long long)limit_us * 1000ull);
    if (waited_ns != nullptr) *waited_ns = tc::global_timer_ns() - t0;
    if (ok) atomicExch(status, VSA2_ERR_INVALID_ARG);      // cannot happen: nothing arrives on that barrier
  } else if (tid == 64) {
    // a second role parked on another barrier: it must leave as soon as the first one has given up (shared abort flag),
    // long before its own 2 s limit
    tc::mbar_wait(&other, 0, &abort_flag);
  }
  tc::tc_fence_before();
  __syncthreads();
  if (abort_flag && tid == 0) atomicExch(status, VSA2_ERR_DEVICE_TIMEOUT);
  if (warp == 0) tc::tmem_dealloc(tmem_base, 128);
}

}  // namespace vsa2

using namespace vsa2;

// Host-only check of the index division the kernels use (common.cuh: q = floor(n * ceil(2^32 / d) / 2^32)): every n up to
// n_max for every divisor d_min .. d_exhaustive, and for the larger divisors up to d_max every multiple of d and its two
// neighbours.  Returns the number of wrong quotients.
extern "C" int64_t vsa2_selftest_divmod(int32_t n_max, int32_t d_min, int32_t d_exhaustive, int32_t d_max) {
  int64_t bad = 0;
  for (int d = d_min < 1 ? 1 : d_min; d <= d_max; ++d) {
    const unsigned m = div_magic(d);
    if (d <= d_exhaustive) {
      for (int n = 0; n <= n_max; ++n) bad += mulhi_div(n, m) != n / d;
    } else {
      for (long long k = 0; k * d <= n_max; ++k)
        for (int e = -1; e <= 1; ++e) {
          const long long n = k * d + e;
          if (n >= 0 && n <= n_max) bad += mulhi_div((int)n, m) != (int)(n / d);
        }
    }
  }
  return bad;
}

extern "C" int vsa2_selftest_timeout(uint32_t limit_us, int32_t* status, uint64_t* waited_ns, void* cuda_stream) {
  if (status == nullptr || limit_us == 0 || limit_us > 100000u) return VSA2_ERR_INVALID_ARG;
  selftest_timeout_kernel<<<1, 128, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      limit_us, status, reinterpret_cast<unsigned long long*>(waited_ns));
  return cudaGetLastError() == cudaSuccess ? VSA2_OK : VSA2_ERR_CUDA;
}

extern "C" int vsa2_selftest_umma(const vsa2_params* p, const void* q, const void* k, const void* v, int32_t cube_q,
                                  int32_t cube_a, int32_t cube_b, const void* p_t, float* s_t_out, float* o_t_out,
                                  void* k_tile_dump, int32_t* status, void* cuda_stream) {
  vsa2_sizes sz;
  int rc = vsa2_query_sizes(p, &sz);
  if (rc != VSA2_OK) return rc;
  if (sz.block_tokens != kBlockTokens) return VSA2_ERR_UNSUPPORTED;      // the self-test addresses 64-token tiles
  if (!q || !k || !v || !p_t || !s_t_out || !o_t_out || !k_tile_dump || !status) return VSA2_ERR_INVALID_ARG;
  Geo g = {};
  g.batch = p->batch; g.Hq = p->heads_q; g.Hkv = p->heads_kv; g.rep = g.Hq / g.Hkv; g.D = p->head_dim;
  g.T = p->grid_t; g.H = p->grid_h; g.W = p->grid_w; g.L = (int)sz.seq_len;
  g.Bt = p->cube_t; g.Bh = p->cube_h; g.Bw = p->cube_w;
  g.Nt = (g.T + g.Bt - 1) / g.Bt; g.Nh = (g.H + g.Bh - 1) / g.Bh; g.Nw = (g.W + g.Bw - 1) / g.Bw; g.N = sz.n_cubes;
  g.Nvid = g.N; g.Lt = 0; g.S = g.L;
  geo_set_magics(g);
  if (cube_q < 0 || cube_q >= g.N || cube_a < 0 || cube_a >= g.N || cube_b < 0 || cube_b >= g.N) return VSA2_ERR_INVALID_ARG;
  CUtensorMap tq, tk, tv;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv))
    return VSA2_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int DH = g.D / 64;
  size_t smem = (size_t)(2 * DH + DH + 2 * DH) * 8192 + 16384 + 1024;
  cudaError_t e;
  if (g.D == 128) {
    if ((e = cudaFuncSetAttribute(selftest_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return VSA2_ERR_CUDA;
    selftest_kernel<128><<<1, 128, smem, st>>>(tq, tk, tv, g, cube_q, cube_a, cube_b, reinterpret_cast<const bf16*>(p_t),
                                               s_t_out, o_t_out, reinterpret_cast<uint4*>(k_tile_dump), status);
  } else {
    if ((e = cudaFuncSetAttribute(selftest_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem))) return VSA2_ERR_CUDA;
    selftest_kernel<64><<<1, 128, smem, st>>>(tq, tk, tv, g, cube_q, cube_a, cube_b, reinterpret_cast<const bf16*>(p_t),
                                              s_t_out, o_t_out, reinterpret_cast<uint4*>(k_tile_dump), status);
  }
  return cudaGetLastError() == cudaSuccess ? VSA2_OK : VSA2_ERR_CUDA;
}
