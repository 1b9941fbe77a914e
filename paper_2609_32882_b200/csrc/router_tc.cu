// Router block scores (paper Eq. 6-7) on the Blackwell tensor cores, two passes as in the paper's kernel
// description (Sec. 2.2 "Kernel Implementation"): pass 1 accumulates the row log-sum-exp of
// Q_r K_r^T * scale, pass 2 recomputes the scores, applies the softmax and pools G x G sub-blocks on chip.
//
// A CTA owns 128 consecutive pooled queries (128/G query cubes) of one head and streams the head's pooled
// keys in tiles of 128 through a TMA ring; S [128 q, 128 keys] lands in tensor memory (four buffers).
// Four compute threads own each query row, 32 key columns of every tile each (a single warp per scheduler keeps
// the exponential unit only half busy); pass 1 merges their running (max, sum) pairs once per item.  The G
// rows of a query cube sit in G adjacent lanes: their pooled sums are combined with warp shuffles.
// Both passes are bound by the exponential unit (one ex2 per score), not by the tensor pipe.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kRtParts = 4;        // compute threads per pooled query row (each owns 128 / kRtParts key columns of a tile)
constexpr int kRtThreads = 64 + 128 * kRtParts;    // TMA warp, MMA warp, 4 * kRtParts compute warps
constexpr int kRtSlots = 4;
constexpr int kRtTile = 128;
constexpr int kRtBufs = 4;         // score tiles in tensor memory (4 x 128 columns = all of it)

template <int D>
struct RouterTc {
  static constexpr int DH = D / 64;
  static constexpr uint32_t HALF = kRtTile * 128;          // 128 rows x 64 channels
  static constexpr uint32_t TILE = DH * HALF;
  static constexpr uint32_t OFF_Q = kRtSlots * TILE;
  static constexpr uint32_t OFF_MISC = OFF_Q + TILE;
  static constexpr uint32_t MISC_BYTES = 4096;
  static size_t smem_bytes(int valid_words) { return OFF_MISC + MISC_BYTES + (size_t)valid_words * 4 + 1024; }
};

struct RouterMisc {
  uint64_t q_full, q_empty;
  uint64_t k_full[kRtSlots], k_empty[kRtSlots];
  uint64_t s_full[kRtBufs], s_free[kRtBufs];
  uint64_t part_ready, part_free;   // pass 1: hand-over of part_stats
  uint32_t tmem_base;
  int abort_flag;
  float2 part_stats[kRtParts - 1][128];   // pass 1: (running max, running sum) of the threads of parts 1 .. kRtParts-1
};

// tensor map over pooled operands [BH, N*G, D] bf16: box = 64 channels x 128 rows x 1
inline bool make_pooled_tmap(CUtensorMap* out, const void* base, int D, int rows_per_head, int heads_total) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows_per_head, (cuuint64_t)heads_total};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)rows_per_head * D * 2};
  cuuint32_t box[3] = {64, kRtTile, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(tc::smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(tc::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// PASS 1 writes lse2[b, hq, row] = log2 sum_{valid keys} 2^(s * scale * log2 e);  PASS 2 writes P_r.
template <int D, int PASS, int G>
__global__ void __launch_bounds__(kRtThreads, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, Geo g,
                 float* __restrict__ lse2, float* __restrict__ pr, StatusBlock* status) {
  using C = RouterTc<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = smem + C::OFF_Q;
  RouterMisc* misc = reinterpret_cast<RouterMisc*>(smem + C::OFF_MISC);
  uint32_t* valid_bits = reinterpret_cast<uint32_t*>(smem + C::OFF_MISC + C::MISC_BYTES);   // one bit per pooled token

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NG = g.N * g.G;
  const int row_tiles = (NG + kRtTile - 1) / kRtTile;
  const int total_items = g.batch * g.Hq * row_tiles;
  const int valid_words = (row_tiles * kRtTile) / 32;
  const float c2 = g.scale * 1.4426950408889634f;

  // validity of every pooled token of the sequence (a sub-cube that is padding only is invalid)
  for (int w = tid; w < valid_words; w += blockDim.x) {
    uint32_t bits = 0u;
    for (int bit = 0; bit < 32; ++bit) {
      const int r = w * 32 + bit;
      if (r < NG && subcube_count(g, r / g.G, r % g.G) > 0) bits |= 1u << bit;
    }
    valid_bits[w] = bits;
  }
  if (tid == 0) {
    misc->abort_flag = 0;
    tc::mbar_init(&misc->q_full, 1);
    tc::mbar_init(&misc->q_empty, 1);
    for (int s = 0; s < kRtSlots; ++s) {
      tc::mbar_init(&misc->k_full[s], 1);
      tc::mbar_init(&misc->k_empty[s], 1);
    }
    for (int s = 0; s < kRtBufs; ++s) {
      tc::mbar_init(&misc->s_full[s], 1);
      tc::mbar_init(&misc->s_free[s], 128 * kRtParts);
    }
    tc::mbar_init(&misc->part_ready, 128 * (kRtParts - 1));
    tc::mbar_init(&misc->part_free, 128);
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
  }
  if (warp == 1) {
    tc::tmem_alloc(&misc->tmem_base, 128 * kRtBufs);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t seq = 0, n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++n_items) {
        const int rt = item % row_tiles, bhq = item / row_tiles;
        const int b = bhq / g.Hq, hq = bhq % g.Hq, bhk = b * g.Hkv + hq / g.rep;
        VSA2_WAIT(&misc->q_empty, (n_items & 1) ^ 1);
        tc::mbar_expect_tx(&misc->q_full, C::TILE);
        for (int h = 0; h < C::DH; ++h) tma_load_3d(q_tile + h * C::HALF, &tm_q, &misc->q_full, h * 64, rt * kRtTile, bhq);
        for (int kt = 0; kt < row_tiles; ++kt, ++seq) {
          const uint32_t slot = seq % kRtSlots, par = (seq / kRtSlots) & 1;
          VSA2_WAIT(&misc->k_empty[slot], par ^ 1);
          tc::mbar_expect_tx(&misc->k_full[slot], C::TILE);
          for (int h = 0; h < C::DH; ++h)
            tma_load_3d(smem + slot * C::TILE + h * C::HALF, &tm_k, &misc->k_full[slot], h * 64, kt * kRtTile, bhk);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = tc::idesc_bf16(128, 128, false, false);
      const uint32_t q_addr = tc::smem_u32(q_tile), slot0 = tc::smem_u32(smem);
      uint32_t seq = 0, n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++n_items) {
        VSA2_WAIT(&misc->q_full, n_items & 1);
        for (int kt = 0; kt < row_tiles; ++kt, ++seq) {
          const uint32_t slot = seq % kRtSlots, buf = seq % kRtBufs;
          VSA2_WAIT(&misc->k_full[slot], (seq / kRtSlots) & 1);
          VSA2_WAIT(&misc->s_free[buf], ((seq / kRtBufs) & 1) ^ 1);
          tc::tc_fence_after();
          const uint32_t k_addr = slot0 + slot * C::TILE;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t aa = q_addr + (ks / 4) * C::HALF + (ks % 4) * 32;
            const uint32_t bb = k_addr + (ks / 4) * C::HALF + (ks % 4) * 32;
            tc::mma_ss(tmem_base + buf * 128, tc::smem_desc_sw128(aa, 16, 1024), tc::smem_desc_sw128(bb, 16, 1024), idesc,
                       ks > 0);
          }
          tc::mma_commit(&misc->s_full[buf]);
          tc::mma_commit(&misc->k_empty[slot]);
          if (kt == row_tiles - 1) tc::mma_commit(&misc->q_empty);
        }
      }
    }
  } else {
    const int quad = warp & 3;                   // tensor-memory lane quadrant of this warp
    const int part = (warp - 2) >> 2;            // which 128 / kRtParts key columns of every tile
    const int row = (quad << 5) | lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t seq = 0, n_items = 0;
    for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++n_items) {
      const int rt = item % row_tiles, bhq = item / row_tiles;
      const int r = rt * kRtTile + row;                          // pooled query index inside the head
      const bool q_valid = (valid_bits[r >> 5] >> (r & 31)) & 1u;
      float m_run = -INFINITY, l_run = 0.f;
      float my_lse2 = 0.f, inv_norm = 0.f;
      if (PASS == 2) {
        my_lse2 = q_valid ? lse2[(size_t)bhq * NG + r] : INFINITY;          // +inf => p = 0 for padding rows
        const uint32_t vb = __ballot_sync(0xffffffffu, q_valid);
        const int gi = __popc((vb >> (lane & ~(G - 1))) & ((G == 32) ? 0xffffffffu : ((1u << G) - 1u)));
        inv_norm = gi > 0 ? 1.f / ((float)gi * (float)G) : 0.f;
      }
      const int qi = r / G;                                       // query cube of this row
      for (int kt = 0; kt < row_tiles; ++kt, ++seq) {
        const uint32_t buf = seq % kRtBufs;
        VSA2_WAIT(&misc->s_full[buf], (seq / kRtBufs) & 1);
        tc::tc_fence_after();
#pragma unroll
        for (int ch = part * (4 / kRtParts); ch < (part + 1) * (4 / kRtParts); ++ch) {
          uint32_t s[32];
          tc::tmem_ld32(lane_addr + buf * 128 + ch * 32, s);
          tc::tmem_ld_wait();
          const uint32_t kbits = valid_bits[kt * 4 + ch];
          if (PASS == 1) {
            // the maximum is taken over the raw scores (the scale is positive) and the scale folded into the exponent's
            // multiply-add: four instructions per score instead of five (both passes are issue- and exponential-bound)
            float cmax = -INFINITY;
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              if (kbits != 0xffffffffu && !((kbits >> c) & 1u)) s[c] = 0xff800000u;      // -inf
              cmax = fmaxf(cmax, __uint_as_float(s[c]));
            }
            if (cmax > -INFINITY) {
              const float m_new = fmaxf(m_run, cmax * c2);
              float acc = 0.f;
#pragma unroll
              for (int c = 0; c < 32; ++c) acc += ex2_approx(fmaf(__uint_as_float(s[c]), c2, -m_new));
              l_run = l_run * ex2_approx(m_run - m_new) + acc;
              m_run = m_new;
            }
          } else {
            // softmax, then G x G pooling: G columns in registers, G rows across adjacent lanes
            float p[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              p[c] = ex2_approx(fmaf(__uint_as_float(s[c]), c2, -my_lse2));
              if (kbits != 0xffffffffu) p[c] = ((kbits >> c) & 1u) ? p[c] : 0.f;
            }
            // Column sums of the 32 / G key cubes of the chunk, then the sum over the G rows of the query cube, which sit in
            // G adjacent lanes: a butterfly that halves the values a lane carries at every step (4 shuffles instead of
            // 3 per key cube; the passes are bound by instruction issue) and leaves each total in one lane.
            static_assert(G == 8 || G == 16, "router pooling layout");
            float tv[32 / G];
#pragma unroll
            for (int cc = 0; cc < 32 / G; ++cc) {
              float tot = 0.f;
#pragma unroll
              for (int c = 0; c < G; ++c) tot += p[cc * G + c];
              tv[cc] = tot;
            }
            float t;
            int cc_mine;
            if constexpr (G == 8) {
              const bool hi4 = lane & 4, hi2 = lane & 2;
              const float k0 = hi4 ? tv[2] : tv[0], k1 = hi4 ? tv[3] : tv[1];
              const float s0 = hi4 ? tv[0] : tv[2], s1 = hi4 ? tv[1] : tv[3];
              const float u0 = k0 + __shfl_xor_sync(0xffffffffu, s0, 4), u1 = k1 + __shfl_xor_sync(0xffffffffu, s1, 4);
              t = (hi2 ? u1 : u0) + __shfl_xor_sync(0xffffffffu, hi2 ? u0 : u1, 2);
              t += __shfl_xor_sync(0xffffffffu, t, 1);
              cc_mine = (hi4 ? 2 : 0) + (hi2 ? 1 : 0);
            } else {
              const bool hi8 = lane & 8;
              t = (hi8 ? tv[1] : tv[0]) + __shfl_xor_sync(0xffffffffu, hi8 ? tv[0] : tv[1], 8);
              t += __shfl_xor_sync(0xffffffffu, t, 4);
              t += __shfl_xor_sync(0xffffffffu, t, 2);
              t += __shfl_xor_sync(0xffffffffu, t, 1);
              cc_mine = hi8 ? 1 : 0;
            }
            const int kj = (kt * kRtTile + ch * 32) / G + cc_mine;
            const bool owner = G == 8 ? !(lane & 1) : !(lane & 7);
            if (owner && qi < g.N && kj < g.N) pr[((size_t)bhq * g.N + qi) * g.N + kj] = t * inv_norm;
          }
        }
        tc::tc_fence_before();
        tc::mbar_arrive(&misc->s_free[buf]);
      }
      if (PASS == 1) {
        // merge the two column halves of the row
        if (part > 0) {
          VSA2_WAIT(&misc->part_free, (n_items & 1) ^ 1);
          misc->part_stats[part - 1][row] = make_float2(m_run, l_run);
          tc::mbar_arrive(&misc->part_ready);
        } else {
          VSA2_WAIT(&misc->part_ready, n_items & 1);
          float2 o[kRtParts - 1];
          float m_new = m_run;
#pragma unroll
          for (int pp = 0; pp < kRtParts - 1; ++pp) {
            o[pp] = misc->part_stats[pp][row];
            m_new = fmaxf(m_new, o[pp].x);
          }
          tc::mbar_arrive(&misc->part_free);
          if (m_new > -INFINITY) {
            l_run *= ex2_approx(m_run - m_new);
#pragma unroll
            for (int pp = 0; pp < kRtParts - 1; ++pp) l_run += o[pp].y * ex2_approx(o[pp].x - m_new);
          }
          if (r < NG) lse2[(size_t)bhq * NG + r] = (l_run > 0.f) ? m_new + __log2f(l_run) : 0.f;
        }
      }
    }
  }

done:
  tc::tc_fence_before();
  __syncthreads();
  if (misc->abort_flag) {
    if (tid == 0) {
      atomicExch(&status->status, VSA2_ERR_DEVICE_TIMEOUT);
      const unsigned long long t0 = tc::global_timer_ns();
      while (tc::global_timer_ns() - t0 < 200000ull) {
      }
    }
    __syncthreads();
  }
  if (warp == 1) tc::tmem_dealloc(tmem_base, 128 * kRtBufs);
}

bool router_tc_supported(const Geo& g) { return g.G == 8 || g.G == 16; }

cudaError_t launch_router_scores_tc(const Geo& g, const bf16* qr, const bf16* kr, float* lse_r, float* pr,
                                    StatusBlock* status, cudaStream_t st) {
  const int NG = g.N * g.G;
  CUtensorMap tq, tk;
  if (!make_pooled_tmap(&tq, qr, g.D, NG, g.batch * g.Hq) || !make_pooled_tmap(&tk, kr, g.D, NG, g.batch * g.Hkv))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int row_tiles = (NG + kRtTile - 1) / kRtTile;
  const int total = g.batch * g.Hq * row_tiles;
  const int grid = total < sms ? total : sms;
  const int valid_words = row_tiles * kRtTile / 32;
#define VSA2_ROUTER_LAUNCH(DD, GG)                                                                                     \
  do {                                                                                                               \
    const size_t smb = RouterTc<DD>::smem_bytes(valid_words);                                                        \
    if (smb > 227 * 1024) return cudaErrorInvalidValue;                                                              \
    if ((e = cudaFuncSetAttribute(router_tc_kernel<DD, 1, GG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e; \
    if ((e = cudaFuncSetAttribute(router_tc_kernel<DD, 2, GG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e; \
    {                                                                                                                \
      ProfScope ps(VSA2_KERNEL_ROUTER_LSE, st, 1);                                                                   \
      router_tc_kernel<DD, 1, GG><<<grid, kRtThreads, smb, st>>>(tq, tk, g, lse_r, pr, status);                          \
    }                                                                                                                \
    {                                                                                                                \
      ProfScope ps(VSA2_KERNEL_ROUTER_POOL, st, 1);                                                                  \
      router_tc_kernel<DD, 2, GG><<<grid, kRtThreads, smb, st>>>(tq, tk, g, lse_r, pr, status);                          \
    }                                                                                                                \
  } while (0)
  if (g.D == 128 && g.G == 8) VSA2_ROUTER_LAUNCH(128, 8);
  else if (g.D == 128 && g.G == 16) VSA2_ROUTER_LAUNCH(128, 16);
  else if (g.D == 64 && g.G == 8) VSA2_ROUTER_LAUNCH(64, 8);
  else if (g.D == 64 && g.G == 16) VSA2_ROUTER_LAUNCH(64, 16);
  else return cudaErrorInvalidValue;
#undef VSA2_ROUTER_LAUNCH
  return cudaGetLastError();
}

}  // namespace vsa2
