// Backward of the fine branch (gradient of paper Eq. 12) on the Blackwell tensor cores.
//
// With P = exp(S*scale - lse), dP = dO V^T and dS = P * (dP - delta) * scale:
//   dQ = dS K,   dK = dS^T Q,   dV = P^T dO.
// As in the forward kernel every product is taken in the orientation that fills the 128 rows of a tcgen05
// MMA, with 64-token cube tiles fetched by 5-D TMA and used both K-major and MN-major from the same
// shared-memory image:
//
//   dQ pass (query block stationary, CSR map), two selected KV blocks stacked per tile:
//     S^T  [128 kv, 64 q] = K_pair Q^T          dP^T [128 kv, 64 q] = V_pair dO^T
//     dS^T = P^T * (dP^T - delta_q) * scale     (one thread per key row; lse, delta broadcast per column)
//     dQ^T [D, 64 q]     += K_pair^T dS^T
//
//   dK/dV pass (KV block stationary, CSC map = transposed map), two query blocks stacked per tile, the
//   query heads of a GQA group concatenated:
//     S    [128 q, 64 kv] = Q_pair K^T          dP   [128 q, 64 kv] = dO_pair V^T
//     P, dS                                      (one thread per query row; lse, delta are per-thread scalars)
//     dV^T [D, 64 kv]    += dO_pair^T P          dK^T [D, 64 kv]    += Q_pair^T dS
//
// Accumulators stay in tensor memory for the whole list of a block, so every output element is written
// once, by one thread, in a fixed order: no floating-point atomics, bitwise reproducible.
// The pooling backward of the coarse branch (Eq. 1) is added in the epilogues.
#include "fine_bwd_tc.cuh"

namespace vsa2 {

// ================================================================================================
// dQ pass
// ================================================================================================
struct DqArgs {
  int* item_counter;    // global, zero before the launch
  const float* lse;
  const float* delta;
  const int* row_ptr;
  const int* col_idx;
  const float* dqc;     // [B, Hq, N, D] or null
  void* dq;
  StatusBlock* status;
};

// Roles: warp 0 = TMA producer of the K pairs (ring A; a slot is held until the dQ^T product of its tile is done) and of
// the stationary Q and dO tiles, warp 1 = TMA producer of the V pairs (ring B), warp 2 = issuer of S^T, warp 3 = issuer
// of dP^T, warp 12 = issuer of dQ^T += K_pair^T dS^T, warps 4..11 = elementwise stage + epilogue (each half of the query
// columns): P is formed from S^T while dP^T is still being computed.
// SPLIT: dS^T is handed to the dQ^T product as [bf16(dS^T) | bf16(dS^T - bf16(dS^T))] (one N = 128 product into two
// accumulator halves that the epilogue adds), which removes the bf16 rounding of dS from dQ; the two operand buffers
// then hold one tile (hi, lo) instead of two tiles.
template <int D, bool SPLIT>
__global__ void __launch_bounds__(kDqThreads, 1)
fine_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                      const __grid_constant__ CUtensorMap tm_qt, const __grid_constant__ CUtensorMap tm_kt,
                      const __grid_constant__ CUtensorMap tm_vt, const __grid_constant__ CUtensorMap tm_dot, Geo g,
                      DqArgs a) {
  using C = BwdTc<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = smem + C::OFF_ST0;
  unsigned char* do_tile = smem + C::OFF_ST1;
  unsigned char* ds_tile = smem + C::OFF_P;      // two buffers
  BwdMisc* misc = reinterpret_cast<BwdMisc*>(smem + C::OFF_MISC);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hq * g.N;
  const float c2 = g.scale * 1.4426950408889634f;

  if (tid == 0) {
    bwd_init_barriers(misc);
    item_queue_init(&misc->items, 2 + 3 + 256);     // lane 0 of the producers, three issuers, the elementwise threads
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
    tc::prefetch_tmap(&tm_do);
  }
  if (warp == 2) {
    tc::tmem_alloc(&misc->tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  // tensor-memory columns: S^T buffers 0, 64; dP^T buffers 128, 192; dQ^T 256 (SPLIT: its low-order part at 320)

  if (warp < 2) {
    // ------------------------------------------------------------------ TMA producers
    const int which = warp;                               // 0: K pairs (ring A) + Q, dO tiles; 1: V pairs (ring B)
    const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
    const CUtensorMap* tm_text = which == 0 ? &tm_kt : &tm_vt;
    const int my_blk = lane & 1;
    uint32_t tg = 0, n_items = 0, published = 0;
    for (uint32_t seq = 0;; ++seq) {
      // warp 0, lane 0 is the CTA's scheduler
      int item = 0;
      if (lane == 0) {
        if (which == 0 && !item_publish_ahead(&misc->items, seq, published, a.item_counter, total_items, &misc->abort_flag)) item = -2;
        else item = item_get(&misc->items, seq, &misc->abort_flag);
      }
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item == -2) goto done;
      if (item < 0) break;
      int i, bhq;
      item_block(g, item, bhq, i);
      const int b = bhq / g.Hq, hq = bhq % g.Hq, bhk = b * g.Hkv + hq / g.rep;
      const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
      const int k = end - beg;
      if (k == 0) continue;
      const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
      if (which == 0) {
        int c1, c2, c3;
        block_box(g, i, c1, c2, c3);
        const bool qtext = block_is_text(g, i);
        int ok = 1;
        if (lane == 0) {
          ok = tc::mbar_wait(&misc->st_empty, (n_items & 1) ^ 1, &misc->abort_flag);
          if (ok) tc::mbar_expect_tx(&misc->st_full, 2 * C::TILE);
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
        if (lane < 2 * C::DH) {
          const int h = lane >> 1;
          if (lane & 1) tc::tma_load_5d(do_tile + h * kSlab, qtext ? &tm_dot : &tm_do, &misc->st_full, h * 64, c1, c2, c3, bhq);
          else tc::tma_load_5d(q_tile + h * kSlab, qtext ? &tm_qt : &tm_q, &misc->st_full, h * 64, c1, c2, c3, bhq);
        }
      }
      ++n_items;
      const int nt = (k + 1) >> 1;
      int j = cols[(my_blk == 1 && k > 1) ? 1 : 0];
      for (int t = 0; t < nt; ++t, ++tg) {
        int c1, c2, c3;
        block_box(g, j, c1, c2, c3);
        const CUtensorMap* tm_j = block_is_text(g, j) ? tm_text : tm;
        const unsigned ef0 = block_edge_flags(g, j);
        if (t + 1 < nt) j = cols[(my_blk == 1 && 2 * t + 3 < k) ? 2 * t + 3 : 2 * t + 2];
        if (which == 0) {
          const unsigned ef1 = __shfl_sync(0xffffffffu, ef0, 1);
          VSA2_RING_LOAD(misc->a_full, misc->a_empty, kRingA, smem, tm_j, tg, c3, c2, c1, bhk,
                         { misc->edge[slot_][0] = (unsigned char)ef0; misc->edge[slot_][1] = (unsigned char)ef1; }, mbar_wait);
        } else {
          VSA2_RING_LOAD(misc->b_full, misc->b_empty, kRingB, smem + C::OFF_RING_B, tm_j, tg, c3, c2, c1, bhk, {}, mbar_wait);
        }
      }
    }
  } else if (warp == 2 || warp == 3) {
    // ------------------------------------------------------------------ issuers of S^T = K_pair Q^T (warp 2) and
    // dP^T = V_pair dO^T (warp 3).  The whole warp runs the loop and one elected lane issues: a converged warp keeps the
    // descriptors in uniform registers, and a tcgen05.mma then issues every ~74 cycles instead of ~117 from a lone lane.
    {
      const bool is_s = warp == 2;
      const uint32_t b_addr = tc::smem_u32(is_s ? q_tile : do_tile), base = tc::smem_u32(smem);
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        int i, bhq;
        item_block(g, item, bhq, i);
        const int k = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - a.row_ptr[(size_t)bhq * (g.N + 1) + i];
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->st_full, n_items & 1);
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t sb = tg & 1, pb = (tg >> 1) & 1;
          if (is_s) {
            const uint32_t sa = tg % kRingA, pa = (tg / kRingA) & 1;
            VSA2_WAIT(&misc->a_full[sa], pa);
            VSA2_WAIT(&misc->s_free[sb], pb ^ 1);
            tc::tc_fence_after();
            if (tc::elect_one()) {
              mma_pair_kmajor<D>(tmem_base + sb * 64, base + sa * C::SLOT, b_addr);
              tc::mma_commit(&misc->s_full[sb]);
              if (t == nt - 1) tc::mma_commit(&misc->st_empty);
            }
          } else {
            VSA2_WAIT(&misc->b_full[sb], pb);
            VSA2_WAIT(&misc->dp_free[sb], pb ^ 1);
            tc::tc_fence_after();
            if (tc::elect_one()) {
              mma_pair_kmajor<D>(tmem_base + 128 + sb * 64, base + C::OFF_RING_B + sb * C::SLOT, b_addr);
              tc::mma_commit(&misc->dp_full[sb]);
              tc::mma_commit(&misc->b_empty[sb]);
              if (t == nt - 1) tc::mma_commit(&misc->st_empty);
            }
          }
          __syncwarp();
        }
        ++n_items;
      }
    }
  } else if (warp == 12) {
    // ------------------------------------------------------------------ issuer of dQ^T += K_pair^T dS^T
    {
      const uint32_t ds_addr = tc::smem_u32(ds_tile), base = tc::smem_u32(smem);
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        int i, bhq;
        item_block(g, item, bhq, i);
        const int k = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - a.row_ptr[(size_t)bhq * (g.N + 1) + i];
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t sd = SPLIT ? 0u : (tg & 1), pd = SPLIT ? (tg & 1) : ((tg >> 1) & 1), sa = tg % kRingA;
          VSA2_WAIT(&misc->ds_ready[sd], pd);
          tc::tc_fence_after();
          if (tc::elect_one()) {
            if constexpr (SPLIT) mma_pairT_mnmajor_n128<D>(tmem_base + 256, base + sa * C::SLOT, ds_addr, C::PBYTES, t > 0);
            else mma_pairT_mnmajor<D>(tmem_base + 256, base + sa * C::SLOT, ds_addr + sd * C::PBYTES, t > 0);
            tc::mma_commit(&misc->a_empty[sa]);
            tc::mma_commit(&misc->ds_free[sd]);
            if (t == nt - 1) tc::mma_commit(&misc->o_full);
          }
          __syncwarp();
        }
        ++n_items;
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------------------------------------------ elementwise stage + epilogue (256 threads):
    // warps 4..7 take query columns 0..31 of every tile, warps 8..11 columns 32..63
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;            // which 32 query columns
    const int row = (quad << 5) | lane;          // key row of the tile (S^T, dP^T) / channel (dQ^T)
    const int sm_tid = tid - 128;                // 0..255
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    CubePos cpos;
    cpos.init(g, row & 63);
    const int blk = row >> 6;
    uint32_t tg = 0, n_items = 0;
    for (uint32_t n_all = 0;; ++n_all) {
      VSA2_NEXT_ITEM(item, n_all);
      int i, bhq;
      item_block(g, item, bhq, i);
      const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
      const int k = end - beg;
      const int tb = n_all & 1;
      const uint32_t e_sync0 = n_all * (g.out_f32 ? 1u : 3u);     // index of this item's first group sync
      if (sm_tid < 64) {
        const int l = block_token(g, i, sm_tid);
        misc->tok[tb][sm_tid] = l;
        misc->stats[tb * 64 + sm_tid] = l >= 0 ? a.lse[(size_t)bhq * g.S + l] * 1.4426950408889634f : INFINITY;
        misc->stats[128 + tb * 64 + sm_tid] = l >= 0 ? a.delta[(size_t)bhq * g.S + l] : 0.f;
      }
      const float coarse_d = (a.dqc != nullptr && row < D && !block_is_text(g, i))
                                 ? a.dqc[((size_t)bhq * g.Nvid + i) * D + row] / (float)cube_count(g, i) : 0.f;
      VSA2_GROUP_SYNC_AT(&misc->e_sync, e_sync0);
      if (k > 0) {
        const int nt = (k + 1) >> 1;
        const float4* lse4 = reinterpret_cast<const float4*>(misc->stats + tb * 64) + half * 8;
        const float4* del4 = reinterpret_cast<const float4*>(misc->stats + 128 + tb * 64) + half * 8;
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t s = tg & 1, par = (tg >> 1) & 1;
          const bool dup = (blk == 1) && (2 * t + 1 >= k);
          uint32_t packed[16], packed_lo[SPLIT ? 16 : 1];
          {
            uint32_t sv[32];      // S^T, then P^T
            VSA2_WAIT(&misc->s_full[s], par);
            tc::tc_fence_after();
            // (the K slot of the tile, and with it its edge flags, stays until the tile's dQ^T product is done)
            const bool valid = !dup && cpos.valid(misc->edge[tg % kRingA][blk], g);
            tc::tmem_ld32(lane_addr + s * 64 + half * 32, sv);
            tc::tmem_ld_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&misc->s_free[s]);
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              const float4 ls = lse4[c4];
              sv[4 * c4 + 0] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(sv[4 * c4 + 0]), c2, -ls.x)));
              sv[4 * c4 + 1] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(sv[4 * c4 + 1]), c2, -ls.y)));
              sv[4 * c4 + 2] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(sv[4 * c4 + 2]), c2, -ls.z)));
              sv[4 * c4 + 3] = __float_as_uint(ex2_approx(fmaf(__uint_as_float(sv[4 * c4 + 3]), c2, -ls.w)));
            }
            uint32_t dp[32];
            VSA2_WAIT(&misc->dp_full[s], par);
            tc::tc_fence_after();
            tc::tmem_ld32(lane_addr + 128 + s * 64 + half * 32, dp);
            tc::tmem_ld_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&misc->dp_free[s]);
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              const float4 dl = del4[c4];
              const float d0 = __uint_as_float(sv[4 * c4 + 0]) * (__uint_as_float(dp[4 * c4 + 0]) - dl.x);
              const float d1 = __uint_as_float(sv[4 * c4 + 1]) * (__uint_as_float(dp[4 * c4 + 1]) - dl.y);
              const float d2 = __uint_as_float(sv[4 * c4 + 2]) * (__uint_as_float(dp[4 * c4 + 2]) - dl.z);
              const float d3 = __uint_as_float(sv[4 * c4 + 3]) * (__uint_as_float(dp[4 * c4 + 3]) - dl.w);
              if constexpr (SPLIT) {
                uint32_t h0, l0, h1, l1;
                split_bf16x2(d0, d1, h0, l0);
                split_bf16x2(d2, d3, h1, l1);
                packed[2 * c4] = valid ? h0 : 0u;
                packed[2 * c4 + 1] = valid ? h1 : 0u;
                packed_lo[2 * c4] = valid ? l0 : 0u;
                packed_lo[2 * c4 + 1] = valid ? l1 : 0u;
              } else {
                packed[2 * c4] = valid ? pack_bf16x2(d0, d1) : 0u;
                packed[2 * c4 + 1] = valid ? pack_bf16x2(d2, d3) : 0u;
              }
            }
          }
          const uint32_t sd = SPLIT ? 0u : s;
          VSA2_WAIT(&misc->ds_free[sd], SPLIT ? ((tg & 1) ^ 1) : (par ^ 1));
          {
            unsigned char* prow = ds_tile + sd * C::PBYTES + row * 128;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              *reinterpret_cast<uint4*>(prow + (((half * 4 + ch) ^ (row & 7)) << 4)) =
                  make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
              if constexpr (SPLIT)
                *reinterpret_cast<uint4*>(prow + C::PBYTES + (((half * 4 + ch) ^ (row & 7)) << 4)) =
                    make_uint4(packed_lo[4 * ch], packed_lo[4 * ch + 1], packed_lo[4 * ch + 2], packed_lo[4 * ch + 3]);
            }
          }
          tc::fence_proxy_async_smem();
          tc::mbar_arrive(&misc->ds_ready[sd]);
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
      }
      // epilogue: dQ[l, d] = scale * dQ^T[d, q] + dQ_c[i, d] / count(i) (dS goes to its product without the softmax scale);
      // this thread owns 32 query columns of channel `row`
      {
        uint32_t o0[32];
        if (k > 0) {
          tc::tmem_ld32(lane_addr + 256 + half * 32, o0);
          tc::tmem_ld_wait();
          if constexpr (SPLIT) {
            uint32_t o1[32];
            tc::tmem_ld32(lane_addr + 320 + half * 32, o1);
            tc::tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; ++c) o0[c] = __float_as_uint(__uint_as_float(o0[c]) + __uint_as_float(o1[c]));
          }
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) o0[c] = 0u;
        }
        if (g.out_f32) {
          if (row < D) {
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int l = misc->tok[tb][half * 32 + c];
              if (l < 0) continue;
              store_out(a.dq, ((size_t)bhq * g.S + l) * D + row, fmaf(__uint_as_float(o0[c]), g.scale, coarse_d), 1);
            }
          }
        } else {
          // bf16: transpose through shared memory (the dS^T buffers are idle now), then 16-byte stores
          bf16* st = reinterpret_cast<bf16*>(ds_tile);                  // [64 q][D]
          if (row < D) {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              st[(half * 32 + c) * D + row] = __float2bfloat16_rn(fmaf(__uint_as_float(o0[c]), g.scale, coarse_d));
          }
          VSA2_GROUP_SYNC_AT(&misc->e_sync, e_sync0 + 1);
          constexpr int CH = D / 8;
          for (int e = sm_tid; e < 64 * CH; e += 256) {
            const int qi = e / CH, ch = e % CH;
            const int l = misc->tok[tb][qi];
            if (l < 0) continue;
            *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.dq) + ((size_t)bhq * g.S + l) * D + ch * 8) =
                *reinterpret_cast<const uint4*>(st + qi * D + ch * 8);
          }
          VSA2_GROUP_SYNC_AT(&misc->e_sync, e_sync0 + 2);
        }
      }
      if (k > 0) ++n_items;
    }
  }

done:
  tc::tc_fence_before();
  __syncthreads();
  if (misc->abort_flag) {
    if (tid == 0) {
      atomicExch(&a.status->status, VSA2_ERR_DEVICE_TIMEOUT);
      const unsigned long long t0 = tc::global_timer_ns();
      while (tc::global_timer_ns() - t0 < 200000ull) {
      }
    }
    __syncthreads();
  }
  if (warp == 2) tc::tmem_dealloc(tmem_base, 512);
}

// ================================================================================================
// launcher
// ================================================================================================
cudaError_t launch_fine_bwd_dq_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                  const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                                  const float* dqc, void* dq, StatusBlock* status, cudaStream_t st) {
  CUtensorMap tq, tk, tv, tdo, tqt, tkt, tvt, tdot;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_cube_tmap(&tdo, d_o, g, g.Hq) || !make_text_tmap(&tqt, q, g, g.Hq) || !make_text_tmap(&tkt, k, g, g.Hkv) ||
      !make_text_tmap(&tvt, v, g, g.Hkv) || !make_text_tmap(&tdot, d_o, g, g.Hq))
    return cudaErrorInvalidValue;
  int sms = 0;
  cudaError_t e;
  if ((e = bwd_sm_count(&sms)) != cudaSuccess) return e;
  DqArgs a{&status->pad[2], lse, delta, row_ptr, col_idx, dqc, dq, status};
  const int total = g.batch * g.Hq * g.N;
  const int grid = total < sms ? total : sms;
  const bool split = !(g.flags & VSA2_FLAG_FAST_BWD);
#define VSA2_LAUNCH_DQ(DD, SP)                                                                                                   \
  do {                                                                                                                           \
    if ((e = cudaFuncSetAttribute(fine_bwd_dq_tc_kernel<DD, SP>, cudaFuncAttributeMaxDynamicSharedMemorySize,                    \
                                  (int)BwdTc<DD>::smem_bytes)))                                                                  \
      return e;                                                                                                                  \
    fine_bwd_dq_tc_kernel<DD, SP><<<grid, kDqThreads, BwdTc<DD>::smem_bytes, st>>>(tq, tk, tv, tdo, tqt, tkt, tvt, tdot, g, a);                       \
  } while (0)
  if (g.D == 128) {
    if (split) VSA2_LAUNCH_DQ(128, true);
    else VSA2_LAUNCH_DQ(128, false);
  } else {
    if (split) VSA2_LAUNCH_DQ(64, true);
    else VSA2_LAUNCH_DQ(64, false);
  }
#undef VSA2_LAUNCH_DQ
  return cudaGetLastError();
}

}  // namespace vsa2
