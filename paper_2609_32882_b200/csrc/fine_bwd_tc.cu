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
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kBwdThreads = 192;
constexpr int kBwdSlots = 4;

template <int D>
struct BwdTc {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLOT = 2 * DH * kSlab;   // a pair of cube tiles, [half][A | B]
  static constexpr uint32_t TILE = DH * kSlab;       // one cube tile, [half]
  static constexpr uint32_t PBYTES = 128 * 128;      // 128 rows x 64 bf16
  static constexpr uint32_t OFF_ST0 = kBwdSlots * SLOT;        // stationary tile 0 (Q or K)
  static constexpr uint32_t OFF_ST1 = OFF_ST0 + TILE;          // stationary tile 1 (dO or V)
  static constexpr uint32_t OFF_P = OFF_ST1 + TILE;            // two 16 KB operand buffers
  static constexpr uint32_t OFF_MISC = OFF_P + 2 * PBYTES;
  static constexpr size_t smem_bytes = OFF_MISC + 4096 + 1024;
};

struct BwdMisc {
  uint64_t st_full, st_empty, o_full, o_empty;
  uint64_t ring_full[kBwdSlots], ring_empty[kBwdSlots];
  uint64_t sdp_full[2], ds_ready[2], ds_free[2];
  uint32_t tmem_base;
  int abort_flag;
  float lse2[2][64];     // dQ pass: per query column, lse * log2(e) (+inf for padding), by item parity
  float delta[2][64];
  int tok[2][64];
};

// ================================================================================================
// dQ pass
// ================================================================================================
struct DqArgs {
  const float* lse;
  const float* delta;
  const int* row_ptr;
  const int* col_idx;
  const float* dqc;     // [B, Hq, N, D] or null
  void* dq;
  StatusBlock* status;
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
fine_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, Geo g,
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
    misc->abort_flag = 0;
    tc::mbar_init(&misc->st_full, 1);
    tc::mbar_init(&misc->st_empty, 1);
    tc::mbar_init(&misc->o_full, 1);
    tc::mbar_init(&misc->o_empty, 128);
    for (int s = 0; s < kBwdSlots; ++s) {
      tc::mbar_init(&misc->ring_full[s], 1);
      tc::mbar_init(&misc->ring_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->sdp_full[s], 1);
      tc::mbar_init(&misc->ds_ready[s], 128);
      tc::mbar_init(&misc->ds_free[s], 1);
    }
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
    tc::prefetch_tmap(&tm_do);
  }
  if (warp == 1) {
    tc::tmem_alloc(&misc->tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  // tensor-memory columns: S^T buffers 0, 64; dP^T buffers 128, 192; dQ^T 256

  if (warp == 0) {
    if (lane == 0) {
      uint32_t seq = 0, n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const int i = item % g.N, bhq = item / g.N;
        const int b = bhq / g.Hq, hq = bhq % g.Hq, bhk = b * g.Hkv + hq / g.rep;
        const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
        const int k = end - beg;
        if (k == 0) continue;
        const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
        int it_, ih_, iw_;
        cube_coords(g, i, it_, ih_, iw_);
        VSA2_WAIT(&misc->st_empty, (n_items & 1) ^ 1);
        tc::mbar_expect_tx(&misc->st_full, 2 * C::TILE);
        for (int h = 0; h < C::DH; ++h) {
          tc::tma_load_5d(q_tile + h * kSlab, &tm_q, &misc->st_full, h * 64, iw_ * g.Bw, ih_ * g.Bh, it_ * g.Bt, bhq);
          tc::tma_load_5d(do_tile + h * kSlab, &tm_do, &misc->st_full, h * 64, iw_ * g.Bw, ih_ * g.Bh, it_ * g.Bt, bhq);
        }
        ++n_items;
        const int nt = (k + 1) >> 1;
        for (int t = 0; t < nt; ++t) {
          const int ja = cols[2 * t], jb = (2 * t + 1 < k) ? cols[2 * t + 1] : ja;
          int at, ah, aw, bt, bh_, bw;
          cube_coords(g, ja, at, ah, aw);
          cube_coords(g, jb, bt, bh_, bw);
          for (int which = 0; which < 2; ++which, ++seq) {   // K pair, then V pair
            const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
            const uint32_t slot = seq % kBwdSlots, par = (seq / kBwdSlots) & 1;
            unsigned char* dst = smem + slot * C::SLOT;
            VSA2_WAIT(&misc->ring_empty[slot], par ^ 1);
            tc::mbar_expect_tx(&misc->ring_full[slot], C::SLOT);
            for (int h = 0; h < C::DH; ++h) {
              tc::tma_load_5d(dst + (2 * h + 0) * kSlab, tm, &misc->ring_full[slot], h * 64, aw * g.Bw, ah * g.Bh, at * g.Bt, bhk);
              tc::tma_load_5d(dst + (2 * h + 1) * kSlab, tm, &misc->ring_full[slot], h * 64, bw * g.Bw, bh_ * g.Bh, bt * g.Bt, bhk);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t q_addr = tc::smem_u32(q_tile), do_addr = tc::smem_u32(do_tile), ds_addr = tc::smem_u32(ds_tile);
      const uint32_t slot0 = tc::smem_u32(smem);
      uint32_t seq0 = 0, tt = 0, n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const int i = item % g.N, bhq = item / g.N;
        const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
        const int k = end - beg;
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->st_full, n_items & 1);
        tc::tc_fence_after();
        for (int t = 0; t <= nt; ++t) {
          if (t < nt) {
            const uint32_t sk = seq0 + 2 * t, sv = sk + 1;
            const uint32_t slot_k = sk % kBwdSlots, slot_v = sv % kBwdSlots, buf = (tt + t) & 1;
            VSA2_WAIT(&misc->ring_full[slot_k], (sk / kBwdSlots) & 1);
            VSA2_WAIT(&misc->ring_full[slot_v], (sv / kBwdSlots) & 1);
            tc::tc_fence_after();
            mma_pair_kmajor<D>(tmem_base + buf * 64, slot0 + slot_k * C::SLOT, q_addr);
            mma_pair_kmajor<D>(tmem_base + 128 + buf * 64, slot0 + slot_v * C::SLOT, do_addr);
            tc::mma_commit(&misc->sdp_full[buf]);
            tc::mma_commit(&misc->ring_empty[slot_v]);
            if (t == nt - 1) tc::mma_commit(&misc->st_empty);
          }
          if (t >= 1) {
            const uint32_t tp = tt + t - 1, buf = tp & 1;
            const uint32_t sk = seq0 + 2 * (t - 1), slot_k = sk % kBwdSlots;
            VSA2_WAIT(&misc->ds_ready[buf], (tp >> 1) & 1);
            if (t == 1) VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);
            tc::tc_fence_after();
            mma_pairT_mnmajor<D>(tmem_base + 256, slot0 + slot_k * C::SLOT, ds_addr + buf * C::PBYTES, t > 1);
            tc::mma_commit(&misc->ring_empty[slot_k]);
            tc::mma_commit(&misc->ds_free[buf]);
            if (t == nt) tc::mma_commit(&misc->o_full);
          }
        }
        seq0 += 2 * nt;
        tt += nt;
        ++n_items;
      }
    }
  } else {
    const int quad = warp & 3;
    const int row = (quad << 5) | lane;
    const int sm_tid = tid - 64;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t tt = 0, n_items = 0, n_all = 0;
    for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++n_all) {
      const int i = item % g.N, bhq = item / g.N;
      const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
      const int k = end - beg;
      const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
      const int tb = n_all & 1;
      if (sm_tid < 64) {
        int it_, ih_, iw_;
        cube_coords(g, i, it_, ih_, iw_);
        const int l = cube_token(g, it_, ih_, iw_, sm_tid);
        misc->tok[tb][sm_tid] = l;
        misc->lse2[tb][sm_tid] = l >= 0 ? a.lse[(size_t)bhq * g.L + l] * 1.4426950408889634f : INFINITY;
        misc->delta[tb][sm_tid] = l >= 0 ? a.delta[(size_t)bhq * g.L + l] : 0.f;
      }
      const float coarse_d = (a.dqc != nullptr && row < D)
                                 ? a.dqc[((size_t)bhq * g.N + i) * D + row] / (float)cube_count(g, i) : 0.f;
      tc::named_bar_sync(1, 128);
      if (k > 0) {
        const int nt = (k + 1) >> 1;
        for (int t = 0; t < nt; ++t, ++tt) {
          const uint32_t buf = tt & 1, use = (tt >> 1) & 1;
          const int blk = row >> 6;
          const bool dup = (blk == 1) && (2 * t + 1 >= k);
          const int j = cols[dup ? 2 * t : 2 * t + blk];
          const bool valid = !dup && pos_valid(g, j, row & 63);
          VSA2_WAIT(&misc->sdp_full[buf], use);
          tc::tc_fence_after();
          uint32_t packed[32];
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t s[32], dp[32];
            tc::tmem_ld32(lane_addr + buf * 64 + half * 32, s);
            tc::tmem_ld32(lane_addr + 128 + buf * 64 + half * 32, dp);
            tc::tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              const int q0 = half * 32 + c;
              float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), c2, -misc->lse2[tb][q0]));
              float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), c2, -misc->lse2[tb][q0 + 1]));
              float d0 = p0 * (__uint_as_float(dp[c]) - misc->delta[tb][q0]) * g.scale;
              float d1 = p1 * (__uint_as_float(dp[c + 1]) - misc->delta[tb][q0 + 1]) * g.scale;
              packed[half * 16 + (c >> 1)] = valid ? pack_bf16x2(d0, d1) : 0u;
            }
          }
          VSA2_WAIT(&misc->ds_free[buf], use ^ 1);
          store_row_sw128(ds_tile + buf * C::PBYTES, row, packed);
          tc::fence_proxy_async_smem();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->ds_ready[buf]);
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
      }
      // epilogue: dQ[l, d] = dQ^T[d, q] + dQ_c[i, d] / count(i)
      {
        uint32_t o0[32], o1[32];
        if (k > 0) {
          tc::tmem_ld32(lane_addr + 256, o0);
          tc::tmem_ld32(lane_addr + 256 + 32, o1);
          tc::tmem_ld_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) { o0[c] = 0u; o1[c] = 0u; }
        }
        if (row < D) {
#pragma unroll
          for (int qi = 0; qi < 64; ++qi) {
            const int l = misc->tok[tb][qi];
            if (l < 0) continue;
            const float acc = __uint_as_float(qi < 32 ? o0[qi & 31] : o1[qi & 31]);
            store_out(a.dq, ((size_t)bhq * g.L + l) * D + row, acc + coarse_d, g.out_f32);
          }
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
  if (warp == 1) tc::tmem_dealloc(tmem_base, 512);
}

// ================================================================================================
// dK/dV pass
// ================================================================================================
struct DkvArgs {
  const float* lse;
  const float* delta;
  const int* col_ptr;
  const int* row_idx;
  const float* dkc;     // [B, Hq, N, D] per query head, or null
  const float* dvc;
  void* dk;
  void* dv;
  StatusBlock* status;
};

constexpr int kMaxRep = 16;   // query heads per KV head the dK/dV pass supports

// entry e of the concatenated column lists of the group's query heads -> (query head, query block)
__device__ __forceinline__ void dkv_entry(const Geo& g, const DkvArgs& a, int b, int hk, int j, const int* cnt_prefix,
                                          int e, int& bhq, int& i) {
  int hh = 0;
  while (hh + 1 < g.rep && e >= cnt_prefix[hh + 1]) ++hh;
  bhq = b * g.Hq + hk * g.rep + hh;
  const int beg = a.col_ptr[(size_t)bhq * (g.N + 1) + j];
  i = a.row_idx[(size_t)bhq * g.nnz_cap + beg + (e - cnt_prefix[hh])];
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
fine_bwd_dkv_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, Geo g,
                       DkvArgs a) {
  using C = BwdTc<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* k_tile = smem + C::OFF_ST0;
  unsigned char* v_tile = smem + C::OFF_ST1;
  unsigned char* p_tile = smem + C::OFF_P;                 // P  [128 q, 64 kv]
  unsigned char* ds_tile = smem + C::OFF_P + C::PBYTES;    // dS [128 q, 64 kv]
  BwdMisc* misc = reinterpret_cast<BwdMisc*>(smem + C::OFF_MISC);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hkv * g.N;
  const float c2 = g.scale * 1.4426950408889634f;

  if (tid == 0) {
    misc->abort_flag = 0;
    tc::mbar_init(&misc->st_full, 1);
    tc::mbar_init(&misc->st_empty, 1);
    tc::mbar_init(&misc->o_full, 1);
    tc::mbar_init(&misc->o_empty, 128);
    for (int s = 0; s < kBwdSlots; ++s) {
      tc::mbar_init(&misc->ring_full[s], 1);
      tc::mbar_init(&misc->ring_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->sdp_full[s], 1);
      tc::mbar_init(&misc->ds_ready[s], 128);
      tc::mbar_init(&misc->ds_free[s], 1);
    }
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
    tc::prefetch_tmap(&tm_do);
  }
  if (warp == 1) {
    tc::tmem_alloc(&misc->tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  // tensor-memory columns: S buffers 0, 64; dP buffers 128, 192; dK^T 256; dV^T 320

  // per item: prefix of the per-head column counts (every role recomputes it)
#define VSA2_DKV_ITEM_SETUP()                                                            \
  const int j = item % g.N, bhk = item / g.N;                                            \
  const int b = bhk / g.Hkv, hk = bhk % g.Hkv;                                           \
  int cnt_prefix[kMaxRep + 1];                                                           \
  cnt_prefix[0] = 0;                                                                     \
  for (int hh = 0; hh < g.rep; ++hh) {                                                   \
    const size_t base = (size_t)(b * g.Hq + hk * g.rep + hh) * (g.N + 1) + j;            \
    cnt_prefix[hh + 1] = cnt_prefix[hh] + (a.col_ptr[base + 1] - a.col_ptr[base]);       \
  }                                                                                      \
  const int k = cnt_prefix[g.rep];

  if (warp == 0) {
    if (lane == 0) {
      uint32_t seq = 0, n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        VSA2_DKV_ITEM_SETUP();
        if (k == 0) continue;
        int jt, jh, jw;
        cube_coords(g, j, jt, jh, jw);
        VSA2_WAIT(&misc->st_empty, (n_items & 1) ^ 1);
        tc::mbar_expect_tx(&misc->st_full, 2 * C::TILE);
        for (int h = 0; h < C::DH; ++h) {
          tc::tma_load_5d(k_tile + h * kSlab, &tm_k, &misc->st_full, h * 64, jw * g.Bw, jh * g.Bh, jt * g.Bt, bhk);
          tc::tma_load_5d(v_tile + h * kSlab, &tm_v, &misc->st_full, h * 64, jw * g.Bw, jh * g.Bh, jt * g.Bt, bhk);
        }
        ++n_items;
        const int nt = (k + 1) >> 1;
        for (int t = 0; t < nt; ++t) {
          int bhq_a, ia, bhq_b, ib;
          dkv_entry(g, a, b, hk, j, cnt_prefix, 2 * t, bhq_a, ia);
          if (2 * t + 1 < k) dkv_entry(g, a, b, hk, j, cnt_prefix, 2 * t + 1, bhq_b, ib);
          else { bhq_b = bhq_a; ib = ia; }
          int at, ah, aw, bt, bh_, bw;
          cube_coords(g, ia, at, ah, aw);
          cube_coords(g, ib, bt, bh_, bw);
          for (int which = 0; which < 2; ++which, ++seq) {   // Q pair, then dO pair
            const CUtensorMap* tm = which == 0 ? &tm_q : &tm_do;
            const uint32_t slot = seq % kBwdSlots, par = (seq / kBwdSlots) & 1;
            unsigned char* dst = smem + slot * C::SLOT;
            VSA2_WAIT(&misc->ring_empty[slot], par ^ 1);
            tc::mbar_expect_tx(&misc->ring_full[slot], C::SLOT);
            for (int h = 0; h < C::DH; ++h) {
              tc::tma_load_5d(dst + (2 * h + 0) * kSlab, tm, &misc->ring_full[slot], h * 64, aw * g.Bw, ah * g.Bh, at * g.Bt, bhq_a);
              tc::tma_load_5d(dst + (2 * h + 1) * kSlab, tm, &misc->ring_full[slot], h * 64, bw * g.Bw, bh_ * g.Bh, bt * g.Bt, bhq_b);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t k_addr = tc::smem_u32(k_tile), v_addr = tc::smem_u32(v_tile);
      const uint32_t p_addr = tc::smem_u32(p_tile), ds_addr = tc::smem_u32(ds_tile), slot0 = tc::smem_u32(smem);
      uint32_t seq0 = 0, tt = 0, n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        VSA2_DKV_ITEM_SETUP();
        (void)b; (void)hk;
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->st_full, n_items & 1);
        tc::tc_fence_after();
        for (int t = 0; t <= nt; ++t) {
          if (t < nt) {
            const uint32_t sq = seq0 + 2 * t, sd = sq + 1;
            const uint32_t slot_q = sq % kBwdSlots, slot_d = sd % kBwdSlots, buf = (tt + t) & 1;
            VSA2_WAIT(&misc->ring_full[slot_q], (sq / kBwdSlots) & 1);
            VSA2_WAIT(&misc->ring_full[slot_d], (sd / kBwdSlots) & 1);
            tc::tc_fence_after();
            mma_pair_kmajor<D>(tmem_base + buf * 64, slot0 + slot_q * C::SLOT, k_addr);
            mma_pair_kmajor<D>(tmem_base + 128 + buf * 64, slot0 + slot_d * C::SLOT, v_addr);
            tc::mma_commit(&misc->sdp_full[buf]);
            if (t == nt - 1) tc::mma_commit(&misc->st_empty);
          }
          if (t >= 1) {
            const uint32_t tp = tt + t - 1;
            const uint32_t sq = seq0 + 2 * (t - 1), slot_q = sq % kBwdSlots, slot_d = (sq + 1) % kBwdSlots;
            VSA2_WAIT(&misc->ds_ready[0], tp & 1);
            if (t == 1) VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);
            tc::tc_fence_after();
            mma_pairT_mnmajor<D>(tmem_base + 320, slot0 + slot_d * C::SLOT, p_addr, t > 1);    // dV^T += dO^T P
            mma_pairT_mnmajor<D>(tmem_base + 256, slot0 + slot_q * C::SLOT, ds_addr, t > 1);   // dK^T += Q^T dS
            tc::mma_commit(&misc->ring_empty[slot_q]);
            tc::mma_commit(&misc->ring_empty[slot_d]);
            tc::mma_commit(&misc->ds_free[0]);
            if (t == nt) tc::mma_commit(&misc->o_full);
          }
        }
        seq0 += 2 * nt;
        tt += nt;
        ++n_items;
      }
    }
  } else {
    const int quad = warp & 3;
    const int row = (quad << 5) | lane;      // query row of the tile (S, dP) / channel (dK^T, dV^T)
    const int sm_tid = tid - 64;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t tt = 0, n_items = 0, n_all = 0;
    for (int item = blockIdx.x; item < total_items; item += gridDim.x, ++n_all) {
      VSA2_DKV_ITEM_SETUP();
      const int tb = n_all & 1;
      int jt, jh, jw;
      cube_coords(g, j, jt, jh, jw);
      if (sm_tid < 64) misc->tok[tb][sm_tid] = cube_token(g, jt, jh, jw, sm_tid);
      unsigned long long kvmask = 0ull;
      if (k > 0)
        for (int p = 0; p < 64; ++p)
          if (cube_token(g, jt, jh, jw, p) >= 0) kvmask |= 1ull << p;
      float coarse_k = 0.f, coarse_v = 0.f;
      if (a.dkc != nullptr && row < D) {
        for (int hh = 0; hh < g.rep; ++hh) {
          const size_t cidx = ((size_t)(b * g.Hq + hk * g.rep + hh) * g.N + j) * D + row;
          coarse_k += a.dkc[cidx];
          coarse_v += a.dvc[cidx];
        }
        const float inv_cnt = 1.f / (float)cube_count(g, j);
        coarse_k *= inv_cnt;
        coarse_v *= inv_cnt;
      }
      tc::named_bar_sync(1, 128);
      if (k > 0) {
        const int nt = (k + 1) >> 1;
        for (int t = 0; t < nt; ++t, ++tt) {
          const uint32_t buf = tt & 1, use = (tt >> 1) & 1;
          // this thread's query row: which (head, block, token)
          const int blk = row >> 6;
          const bool dup = (blk == 1) && (2 * t + 1 >= k);
          int bhq, i;
          dkv_entry(g, a, b, hk, j, cnt_prefix, dup ? 2 * t : 2 * t + blk, bhq, i);
          int it_, ih_, iw_;
          cube_coords(g, i, it_, ih_, iw_);
          const int l = dup ? -1 : cube_token(g, it_, ih_, iw_, row & 63);
          const float lse2 = l >= 0 ? a.lse[(size_t)bhq * g.L + l] * 1.4426950408889634f : INFINITY;
          const float dlt = l >= 0 ? a.delta[(size_t)bhq * g.L + l] : 0.f;
          VSA2_WAIT(&misc->sdp_full[buf], use);
          tc::tc_fence_after();
          uint32_t pp[32], pd[32];
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t s[32], dp[32];
            tc::tmem_ld32(lane_addr + buf * 64 + half * 32, s);
            tc::tmem_ld32(lane_addr + 128 + buf * 64 + half * 32, dp);
            tc::tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              const int c0 = half * 32 + c;
              float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), c2, -lse2));
              float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), c2, -lse2));
              p0 = ((kvmask >> c0) & 1ull) ? p0 : 0.f;
              p1 = ((kvmask >> (c0 + 1)) & 1ull) ? p1 : 0.f;
              const float d0 = p0 * (__uint_as_float(dp[c]) - dlt) * g.scale;
              const float d1 = p1 * (__uint_as_float(dp[c + 1]) - dlt) * g.scale;
              pp[half * 16 + (c >> 1)] = pack_bf16x2(p0, p1);
              pd[half * 16 + (c >> 1)] = pack_bf16x2(d0, d1);
            }
          }
          VSA2_WAIT(&misc->ds_free[0], (tt & 1) ^ 1);
          store_row_sw128(p_tile, row, pp);
          store_row_sw128(ds_tile, row, pd);
          tc::fence_proxy_async_smem();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->ds_ready[0]);
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
      }
      {
        uint32_t k0[32], k1[32], v0[32], v1[32];
        if (k > 0) {
          tc::tmem_ld32(lane_addr + 256, k0);
          tc::tmem_ld32(lane_addr + 256 + 32, k1);
          tc::tmem_ld32(lane_addr + 320, v0);
          tc::tmem_ld32(lane_addr + 320 + 32, v1);
          tc::tmem_ld_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) { k0[c] = 0u; k1[c] = 0u; v0[c] = 0u; v1[c] = 0u; }
        }
        if (row < D) {
#pragma unroll
          for (int ki = 0; ki < 64; ++ki) {
            const int l = misc->tok[tb][ki];
            if (l < 0) continue;
            const size_t idx = ((size_t)bhk * g.L + l) * D + row;
            store_out(a.dk, idx, __uint_as_float(ki < 32 ? k0[ki & 31] : k1[ki & 31]) + coarse_k, g.out_f32);
            store_out(a.dv, idx, __uint_as_float(ki < 32 ? v0[ki & 31] : v1[ki & 31]) + coarse_v, g.out_f32);
          }
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
  if (warp == 1) tc::tmem_dealloc(tmem_base, 512);
}

// ================================================================================================
// launchers
// ================================================================================================
static cudaError_t sm_count(int* sms) {
  int dev = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  return cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
}

cudaError_t launch_fine_bwd_dq_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                  const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                                  const float* dqc, void* dq, StatusBlock* status, cudaStream_t st) {
  CUtensorMap tq, tk, tv, tdo;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_cube_tmap(&tdo, d_o, g, g.Hq))
    return cudaErrorInvalidValue;
  int sms = 0;
  cudaError_t e;
  if ((e = sm_count(&sms)) != cudaSuccess) return e;
  DqArgs a{lse, delta, row_ptr, col_idx, dqc, dq, status};
  const int total = g.batch * g.Hq * g.N;
  const int grid = total < sms ? total : sms;
  if (g.D == 128) {
    if ((e = cudaFuncSetAttribute(fine_bwd_dq_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwdTc<128>::smem_bytes))) return e;
    fine_bwd_dq_tc_kernel<128><<<grid, kBwdThreads, BwdTc<128>::smem_bytes, st>>>(tq, tk, tv, tdo, g, a);
  } else {
    if ((e = cudaFuncSetAttribute(fine_bwd_dq_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwdTc<64>::smem_bytes))) return e;
    fine_bwd_dq_tc_kernel<64><<<grid, kBwdThreads, BwdTc<64>::smem_bytes, st>>>(tq, tk, tv, tdo, g, a);
  }
  return cudaGetLastError();
}

cudaError_t launch_fine_bwd_dkv_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                   const float* lse, const float* delta, const int* col_ptr, const int* row_idx,
                                   const float* dkc, const float* dvc, void* dk, void* dv, StatusBlock* status,
                                   cudaStream_t st) {
  if (g.rep > kMaxRep) return cudaErrorInvalidValue;
  CUtensorMap tq, tk, tv, tdo;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_cube_tmap(&tdo, d_o, g, g.Hq))
    return cudaErrorInvalidValue;
  int sms = 0;
  cudaError_t e;
  if ((e = sm_count(&sms)) != cudaSuccess) return e;
  DkvArgs a{lse, delta, col_ptr, row_idx, dkc, dvc, dk, dv, status};
  const int total = g.batch * g.Hkv * g.N;
  const int grid = total < sms ? total : sms;
  if (g.D == 128) {
    if ((e = cudaFuncSetAttribute(fine_bwd_dkv_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwdTc<128>::smem_bytes))) return e;
    fine_bwd_dkv_tc_kernel<128><<<grid, kBwdThreads, BwdTc<128>::smem_bytes, st>>>(tq, tk, tv, tdo, g, a);
  } else {
    if ((e = cudaFuncSetAttribute(fine_bwd_dkv_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwdTc<64>::smem_bytes))) return e;
    fine_bwd_dkv_tc_kernel<64><<<grid, kBwdThreads, BwdTc<64>::smem_bytes, st>>>(tq, tk, tv, tdo, g, a);
  }
  return cudaGetLastError();
}

}  // namespace vsa2
