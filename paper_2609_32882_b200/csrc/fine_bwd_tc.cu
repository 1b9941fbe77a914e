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
  // fp16 form and its fallback: `range_flag` (zero at first) is set when a value left the fp16 range.  when = 0: the launch
  // always runs; 1: it runs if the flag is clear (and sets it if a dS saturates); 2: it runs only if the flag is set.
  int* range_flag;
  int when;
};

// Copies of two bf16 tensors in fp16 (8 elements per thread and step).  Every finite bf16 below 65520 in magnitude has an
// exact fp16 image down to 2^-24 granularity (fp16 keeps more mantissa bits), so products of the copies equal the products
// of the originals; a finite value beyond that range sets `range_flag` and the caller's fp16 kernels stand back.
__global__ void __launch_bounds__(256) cast_bf16_to_f16_kernel(const uint4* __restrict__ xa, uint4* __restrict__ ya, size_t na,
                                                               const uint4* __restrict__ xb, uint4* __restrict__ yb, size_t nb,
                                                               int* range_flag) {
  const size_t stride = (size_t)gridDim.x * blockDim.x, n = na + nb;
  bool bad = false;
  constexpr int U = 4;      // 16-byte loads in flight per thread (a pure streaming kernel)
  for (size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < n; i0 += U * stride) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t i = i0 + u * stride;
      v[u] = i < n ? (i < na ? __ldg(xa + i) : __ldg(xb + (i - na))) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const size_t i = i0 + u * stride;
      if (i >= n) break;
      const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
      uint32_t r[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t m0 = w[e] & 0x7fffu, m1 = (w[e] >> 16) & 0x7fffu;     // magnitudes as bf16 bit patterns (0x4780 = 65536)
        bad |= (m0 >= 0x4780u && m0 < 0x7f80u) || (m1 >= 0x4780u && m1 < 0x7f80u);
        const __half2 h = __floats2half2_rn(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xffff0000u));
        r[e] = *reinterpret_cast<const uint32_t*>(&h);
      }
      const uint4 o = make_uint4(r[0], r[1], r[2], r[3]);
      if (i < na) ya[i] = o;
      else yb[i - na] = o;
    }
  }
  if (bad) atomicExch(range_flag, 1);
}

// Roles: warp 0 = TMA producer of the K pairs (ring A; a slot is held until the dQ^T product of its tile is done) and of
// the stationary Q and dO tiles, warp 1 = TMA producer of the V pairs (ring B), warp 2 = issuer of S^T, warp 3 = issuer
// of dP^T, warp 12 = issuer of dQ^T += K_pair^T dS^T, warps 4..11 = elementwise stage + epilogue (each half of the query
// columns): P is formed from S^T while dP^T is still being computed.
// SPLIT: dS^T is handed to the dQ^T product as [bf16(dS^T) | bf16(dS^T - bf16(dS^T))] (one N = 128 product into two
// accumulator halves that the epilogue adds), which removes the bf16 rounding of dS from dQ; the two operand buffers
// then hold one tile (hi, lo) instead of two tiles.
// F16 (without SPLIT): the maps of Q and K point at fp16 copies of the tensors and dS^T is rounded to fp16, so S^T and the
// dQ^T product are fp16 x fp16 instructions (dP^T stays bf16 x bf16: V and dO are not copied).  S^T comes out as with the
// bf16 originals (the copies are exact), dS keeps 11 significant bits instead of 8, which is what the pair form is for, at
// the cost of the plain form.
template <int D, bool SPLIT, bool F16>
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
  if (a.when != 0 && ((*a.range_flag != 0) != (a.when == 2))) return;     // (the flag is final before this launch starts)

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
              mma_pair_kmajor<D, F16>(tmem_base + sb * 64, base + sa * C::SLOT, b_addr);
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
            // (F16: the second block of an odd list's last tile repeats the first and stays out of the product; the other
            //  forms zero its dS rows instead)
            else mma_pairT_mnmajor<D, F16>(tmem_base + 256, base + sa * C::SLOT, ds_addr + sd * C::PBYTES, t > 0,
                                           (F16 && t == nt - 1 && (k & 1)) ? 4 : 8);
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
              } else if constexpr (F16) {
                // No validity mask in this form: a key row without a token (a position of an edge cube outside the grid, a row
                // behind the last text token) is a zero row of the K tile and adds nothing to dQ^T whatever its dS, and the
                // repeated block of an odd list's last tile is left out by the issuer.  (A dS beyond the fp16 range, such a
                // row's included, becomes an infinity, which the epilogue finds in the accumulator.)
                packed[2 * c4] = pack_f16x2(d0, d1);
                packed[2 * c4 + 1] = pack_f16x2(d2, d3);
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
          // F16: a dS that left the fp16 range went into the product as an infinity and has made every channel of its query
          // column non-finite: the result of this launch is not to be used, the fallback launch redoes it
          if constexpr (F16) {
            if (row < D && any_non_finite32(o0)) atomicExch(a.range_flag, 1);
          }
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
// `q16`, `k16`: null, or scratch for fp16 copies of Q and K (as many elements as the tensors).  With them the default pass
// (no precision flag) is: the copy, the fp16 form of the kernel, and a launch of the pair form that does nothing unless the
// range flag came up (a finite |Q|, |K| >= 65520 or a |dS| >= 65504: the pair form then computes dQ as before).
cudaError_t launch_fine_bwd_dq_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                  const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                                  const float* dqc, void* dq, StatusBlock* status, cudaStream_t st, void* q16, void* k16) {
  const bool f16 = fine_bwd_dq_uses_f16(g) && q16 != nullptr && k16 != nullptr;
  const bf16* qa = f16 ? reinterpret_cast<const bf16*>(q16) : q;      // (same element size and layout: the maps only move bytes)
  const bf16* ka = f16 ? reinterpret_cast<const bf16*>(k16) : k;
  CUtensorMap tq, tk, tv, tdo, tqt, tkt, tvt, tdot, tq0, tk0, tqt0, tkt0;
  if (!make_cube_tmap(&tq, qa, g, g.Hq) || !make_cube_tmap(&tk, ka, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_cube_tmap(&tdo, d_o, g, g.Hq) || !make_text_tmap(&tqt, qa, g, g.Hq) || !make_text_tmap(&tkt, ka, g, g.Hkv) ||
      !make_text_tmap(&tvt, v, g, g.Hkv) || !make_text_tmap(&tdot, d_o, g, g.Hq))
    return cudaErrorInvalidValue;
  if (f16 && (!make_cube_tmap(&tq0, q, g, g.Hq) || !make_cube_tmap(&tk0, k, g, g.Hkv) || !make_text_tmap(&tqt0, q, g, g.Hq) ||
              !make_text_tmap(&tkt0, k, g, g.Hkv)))
    return cudaErrorInvalidValue;
  int sms = 0;
  cudaError_t e;
  if ((e = bwd_sm_count(&sms)) != cudaSuccess) return e;
  int* flag = &status->pad[kRangeFlagSlot];
  DqArgs a{&status->pad[2], lse, delta, row_ptr, col_idx, dqc, dq, status, flag, 0};
  const int total = g.batch * g.Hq * g.N;
  const int grid = total < sms ? total : sms;
  const bool split = !(g.flags & VSA2_FLAG_FAST_BWD);
#define VSA2_LAUNCH_DQ(DD, SP, F, TQ, TK, TQT, TKT)                                                                              \
  do {                                                                                                                           \
    if ((e = cudaFuncSetAttribute(fine_bwd_dq_tc_kernel<DD, SP, F>, cudaFuncAttributeMaxDynamicSharedMemorySize,                 \
                                  (int)BwdTc<DD>::smem_bytes)))                                                                  \
      return e;                                                                                                                  \
    fine_bwd_dq_tc_kernel<DD, SP, F><<<grid, kDqThreads, BwdTc<DD>::smem_bytes, st>>>(TQ, TK, tv, tdo, TQT, TKT, tvt, tdot, g, a); \
  } while (0)
  if (f16) {
    if ((e = launch_cast_bf16_to_f16(q, q16, (size_t)g.batch * g.Hq * g.S * g.D, k, k16, (size_t)g.batch * g.Hkv * g.S * g.D, flag,
                                     st)) != cudaSuccess)
      return e;
    a.when = 1;
    if (g.D == 128) VSA2_LAUNCH_DQ(128, false, true, tq, tk, tqt, tkt);
    else VSA2_LAUNCH_DQ(64, false, true, tq, tk, tqt, tkt);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    a.when = 2;
    a.item_counter = &status->pad[kRangeFlagSlot + 1];     // (its own counter: the fp16 launch has used the other)
    if (g.D == 128) VSA2_LAUNCH_DQ(128, true, false, tq0, tk0, tqt0, tkt0);
    else VSA2_LAUNCH_DQ(64, true, false, tq0, tk0, tqt0, tkt0);
    return cudaGetLastError();
  }
  if (g.D == 128) {
    if (split) VSA2_LAUNCH_DQ(128, true, false, tq, tk, tqt, tkt);
    else VSA2_LAUNCH_DQ(128, false, false, tq, tk, tqt, tkt);
  } else {
    if (split) VSA2_LAUNCH_DQ(64, true, false, tq, tk, tqt, tkt);
    else VSA2_LAUNCH_DQ(64, false, false, tq, tk, tqt, tkt);
  }
#undef VSA2_LAUNCH_DQ
  return cudaGetLastError();
}

cudaError_t launch_cast_bf16_to_f16(const bf16* a, void* a16, size_t na, const bf16* b, void* b16, size_t nb, int* range_flag,
                                    cudaStream_t st) {
  int sms = 0;
  cudaError_t e;
  if ((e = bwd_sm_count(&sms)) != cudaSuccess) return e;
  if ((na | nb) & 7) return cudaErrorInvalidValue;
  cast_bf16_to_f16_kernel<<<sms * 16, 256, 0, st>>>(reinterpret_cast<const uint4*>(a), reinterpret_cast<uint4*>(a16), na / 8,
                                                     reinterpret_cast<const uint4*>(b), reinterpret_cast<uint4*>(b16), nb / 8,
                                                     range_flag);
  return cudaGetLastError();
}

// whether the dQ pass of this problem takes its fp16 form when it is given the scratch for the copies
bool fine_bwd_dq_uses_f16(const Geo& g) { return !(g.flags & (VSA2_FLAG_FAST_BWD | VSA2_FLAG_PRECISE_BWD)); }

}  // namespace vsa2
