// Fine branch forward (paper Eq. 12) + gated merge (Eq. 14) for TWO query blocks that keep the same KV blocks: the two
// halves of a 128-token cube (the paper's 4 x 4 x 8 cube), or one query block of two query heads of a KV group that share
// their map ("group head" routing).  Same formulation as fine_fwd_rows_tc.cu with twice the rows, which is what the tensor
// cores want:
//     S [128 q, 128 kv] = Q_pair [128, D] * K_pair^T       (A = Q_pair from shared memory, B = K_pair, N = 128 keys)
//     O [128 q, D]     += P [128, 128 kv] * V_pair         (A = P from TENSOR MEMORY,      B = V_pair, N = D)
// M = 128 runs the tensor pipe at its full rate (64 cycles per step), every K / V tile is fetched from shared memory once
// for 128 queries, P never touches shared memory: per 8.4 MFLOP tile 64 KB of TMA writes + 96 KB of operand fetches.
// A query row lives in ONE thread (row m of an M = 128 accumulator is tensor-memory lane m), so the reference maximum, the
// fp32 row sum (log-sum-exp) and the sum of the bf16-rounded weights (the normaliser of the output, see
// fine_fwd_rows_tc.cu) are thread-local scalars.
//
// Tensor memory (512 columns): two S buffers (2 x 128), two P buffers (2 x 64 columns of bf16 pairs), O (D columns).
// Roles (512 threads): warps 0..3 = TMA producers (K / V ring x first / second block of a pair; warp 0 also brings the Q
// pair and schedules the CTA's work items), warp 4 = issuer of S, warp 5 = issuer of O, warp 6 = loader of the per-item
// tables, warps 8..15 = two softmax + epilogue warpgroups that alternate tiles (thread r of a warpgroup owns query row r).
// Persistent CTAs draw items from a global counter.  Every wait is bounded.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kF2Threads = 512;
constexpr int kF2KSlots = 3;
constexpr int kF2VSlots = 2;
constexpr int kF2MaxCubes = 8192;

template <int D>
struct FwdRows2 {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLOT = 2 * DH * kSlab;     // a K, V or Q pair: [channel half][block A | block B]
  static constexpr uint32_t OFF_Q = (kF2KSlots + kF2VSlots) * SLOT;
  static constexpr uint32_t OFF_MISC = OFF_Q + SLOT;
  static constexpr uint32_t MISC_BYTES = 8192;
  static constexpr uint32_t TM_S = 0, TM_P = 256, TM_O = 384;
  static size_t smem_bytes(int n_blocks) { return OFF_MISC + MISC_BYTES + ((size_t)n_blocks + 15) / 16 * 16 + 1024; }
};

struct FwdRows2Misc {
  uint64_t q_full, q_empty, o_full, o_empty;
  uint64_t tab_full[2], tab_free[2];
  uint64_t k_full[kF2KSlots], k_empty[kF2KSlots];
  uint64_t v_full[kF2VSlots], v_empty[kF2VSlots];
  uint64_t s_full[2], s_free[2];
  uint64_t p_ready[2], p_free[2];
  ItemQueue items;
  uint64_t all_sync;               // group barrier of the 256 softmax threads
  uint32_t tmem_base;
  int abort_flag;
  int rescue_flag[2];              // per member of the item
  unsigned long long vmask[17];    // [table row of a block]: which of its 64 positions hold tokens
  alignas(16) float m_ref[128];    // per query row: reference exponent (log2 units)
  float red[2][2][128];            // [warpgroup][exact sum | sum of the bf16 roundings][query row]
  alignas(16) float oc[2][2][128]; // [item parity][member][channel]: coarse output row of the member's cube
  int tok[2][128];                 // [item parity][query row]: row of the token tensors (-1 = padding)
  float gate[2][128];
  int list_k[2], list_beg[2];
  int list_head[2][4];
};
static_assert(sizeof(FwdRows2Misc) <= 8192, "misc region too small");

struct FwdRows2Args {
  int pair_heads;       // 0: an item is a query cube of 128 tokens (two half-cubes of one head); 1: an item is one query
                        // block of two consecutive query heads of a KV group whose maps are identical
  int* item_counter;    // global, zero before the launch
  const float* gate;
  const int* row_ptr;   // map at 64-token-block level (expanded for 128-token cubes)
  const int* col_idx;
  const float* oc_hat;  // per 64-token block
  void* o;
  bf16* o_res;
  float* lse;
  StatusBlock* status;
  int* rescue_count;
  int* rescue_items;
  int rescue_cap;
};

// The two "members" of an item share their list of key blocks: member m is query block i0 + m * di of head bhq0 + m * dh;
// the list is row i0 of head bhq0.
struct PairItem {
  int bhq0, i0, dh, di;
};
__device__ __forceinline__ PairItem decode_pair_item(const Geo& g, int pair_heads, int item) {
  PairItem w;
  if (pair_heads) {
    w.i0 = item % g.N;
    w.bhq0 = (item / g.N) * 2;
    w.dh = 1;
    w.di = 0;
  } else {
    w.i0 = (item % (g.N / 2)) * 2;
    w.bhq0 = item / (g.N / 2);
    w.dh = 0;
    w.di = 1;
  }
  return w;
}

template <int D>
__global__ void __launch_bounds__(kF2Threads, 1)
fine_fwd_rows2_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, Geo g, FwdRows2Args a) {
  using C = FwdRows2<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = smem + C::OFF_Q;
  FwdRows2Misc* misc = reinterpret_cast<FwdRows2Misc*>(smem + C::OFF_MISC);
  unsigned char* edge = smem + C::OFF_MISC + C::MISC_BYTES;      // validity-table row of every block

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hq * g.N / 2;
  const float c2 = g.scale * 1.4426950408889634f;

  for (int n = tid; n < g.N; n += blockDim.x) edge[n] = (unsigned char)cube_edge_flags(g, n);
  if (tid < 16) {
    unsigned long long m = 0;
    for (int pos = 0; pos < 64; ++pos) {
      CubePos cp;
      cp.init(g, pos);
      if (cp.valid((unsigned)tid, g)) m |= 1ull << pos;
    }
    misc->vmask[tid] = m;
  }
  if (tid == 0) {
    misc->abort_flag = 0;
    misc->vmask[16] = 0ull;
    tc::mbar_init(&misc->q_full, 1);
    tc::mbar_init(&misc->q_empty, 1);
    tc::mbar_init(&misc->o_full, 1);
    tc::mbar_init(&misc->o_empty, 256);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->tab_full[s], 32);
      tc::mbar_init(&misc->tab_free[s], 256);
      tc::mbar_init(&misc->s_full[s], 1);
      tc::mbar_init(&misc->s_free[s], 128);
      tc::mbar_init(&misc->p_ready[s], 128);
      tc::mbar_init(&misc->p_free[s], 1);
    }
    for (int s = 0; s < kF2KSlots; ++s) {
      tc::mbar_init(&misc->k_full[s], 2);
      tc::mbar_init(&misc->k_empty[s], 1);
    }
    for (int s = 0; s < kF2VSlots; ++s) {
      tc::mbar_init(&misc->v_full[s], 2);
      tc::mbar_init(&misc->v_empty[s], 1);
    }
    tc::mbar_init(&misc->all_sync, 256);
    item_queue_init(&misc->items, 4 + 2 + 1 + 256);
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
  }
  if (warp == 4) {
    tc::tmem_alloc(&misc->tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;

  if (warp < 8) {
    tc::reg_dec<56>();
    if (warp < 4) {
      // ---------------------------------------------------------------- TMA producers
      const int which = warp & 1;                           // 0: K ring (+ Q pair), 1: V ring
      const int my_blk = warp >> 1;                         // 0: first block of the pair, 1: second
      const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
      const uint32_t nslots = which == 0 ? kF2KSlots : kF2VSlots;
      uint64_t* full = which == 0 ? misc->k_full : misc->v_full;
      uint64_t* empty = which == 0 ? misc->k_empty : misc->v_empty;
      unsigned char* ring = smem + (which == 0 ? 0 : kF2KSlots * C::SLOT);
      const int my_h = lane;
      const bool issuer = lane < C::DH;
      uint32_t tg = 0, n_items = 0, published = 0;
      for (uint32_t seq = 0;; ++seq) {
        int item = 0;
        if (lane == 0) {
          if (warp == 0 && !item_publish_ahead(&misc->items, seq, published, a.item_counter, total_items, &misc->abort_flag)) item = -2;
          else item = item_get(&misc->items, seq, &misc->abort_flag);
        }
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item == -2) goto done;
        if (item < 0) break;
        const PairItem wi = decode_pair_item(g, a.pair_heads, item);
        const int b = wi.bhq0 / g.Hq, hq = wi.bhq0 % g.Hq, bhk = b * g.Hkv + hq / g.rep;
        const int beg = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0], end = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1];
        const int k = end - beg;
        if (k == 0) continue;
        const int* cols = a.col_idx + (size_t)wi.bhq0 * g.nnz_cap + beg;
        if (warp == 0) {
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&misc->q_empty, (n_items & 1) ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&misc->q_full, C::SLOT);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (lane < 2 * C::DH) {
            const int m = lane & 1, h = lane >> 1;          // member and channel half of this lane's box
            int it_, ih_, iw_;
            cube_coords(g, wi.i0 + m * wi.di, it_, ih_, iw_);
            tc::tma_load_5d(q_tile + (2 * h + m) * kSlab, &tm_q, &misc->q_full, h * 64, iw_ * g.Bw, ih_ * g.Bh, it_ * g.Bt,
                            wi.bhq0 + m * wi.dh);
          }
        }
        ++n_items;
        const int nt = (k + 1) >> 1;
        int j = cols[(my_blk == 1 && k > 1) ? 1 : 0];
        for (int t = 0; t < nt; ++t, ++tg) {
          int jt, jh, jw;
          cube_coords(g, j, jt, jh, jw);
          if (t + 1 < nt) j = cols[(my_blk == 1 && 2 * t + 3 < k) ? 2 * t + 3 : 2 * t + 2];
          const uint32_t slot = tg % nslots, par = (tg / nslots) & 1;
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&empty[slot], par ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&full[slot], C::SLOT / 2);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (issuer)
            tc::tma_load_5d(ring + slot * C::SLOT + (2 * my_h + my_blk) * kSlab, tm, &full[slot], my_h * 64, jw * g.Bw,
                            jh * g.Bh, jt * g.Bt, bhk);
        }
      }
    } else if (warp == 4) {
      // ---------------------------------------------------------------- issuer of S(t) = Q_pair * K_pair^T (converged warp)
      constexpr uint32_t idesc = tc::idesc_bf16(128, 128, false, false);
      const uint64_t dq = tc::smem_desc_sw128(tc::smem_u32(q_tile), 16, 1024);
      const uint32_t slot0 = tc::smem_u32(smem);
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        const PairItem wi = decode_pair_item(g, a.pair_heads, item);
        const int k = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1] - a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0];
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->q_full, n_items & 1);
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t slot = tg % kF2KSlots, buf = tg & 1;
          VSA2_WAIT(&misc->k_full[slot], (tg / kF2KSlots) & 1);
          VSA2_WAIT(&misc->s_free[buf], ((tg >> 1) & 1) ^ 1);
          tc::tc_fence_after();
          if (tc::elect_one()) {
            const uint64_t dk = tc::smem_desc_sw128(slot0 + slot * C::SLOT, 16, 1024);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint64_t off = (uint64_t)(((ks / 4) * 2 * kSlab + (ks % 4) * 32) >> 4);
              tc::mma_ss(tmem_base + C::TM_S + buf * 128, dq + off, dk + off, idesc, ks > 0);
            }
            tc::mma_commit(&misc->s_full[buf]);
            tc::mma_commit(&misc->k_empty[slot]);
            if (t == nt - 1) tc::mma_commit(&misc->q_empty);
          }
          __syncwarp();
        }
        ++n_items;
      }
    } else if (warp == 5) {
      // ---------------------------------------------------------------- issuer of O += P(t) * V_pair (converged warp)
      constexpr uint32_t idesc = tc::idesc_bf16(128, D, false, true);
      constexpr uint32_t lbo = (D == 128) ? 2 * kSlab : 0;
      const uint32_t slot0 = tc::smem_u32(smem) + kF2KSlots * C::SLOT;
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        const PairItem wi = decode_pair_item(g, a.pair_heads, item);
        const int k = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1] - a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0];
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t slot = tg % kF2VSlots, buf = tg & 1;
          VSA2_WAIT(&misc->v_full[slot], (tg / kF2VSlots) & 1);
          VSA2_WAIT(&misc->p_ready[buf], (tg >> 1) & 1);
          tc::tc_fence_after();
          if (tc::elect_one()) {
            const uint64_t dv = tc::smem_desc_sw128(slot0 + slot * C::SLOT, lbo, 1024);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint64_t ob = (uint64_t)(((ks / 4) * kSlab + (ks % 4) * 2048) >> 4);
              tc::mma_ts(tmem_base + C::TM_O, tmem_base + C::TM_P + buf * 64 + ks * 8, dv + ob, idesc, t > 0 || ks > 0);
            }
            tc::mma_commit(&misc->v_empty[slot]);
            tc::mma_commit(&misc->p_free[buf]);
            if (t == nt - 1) tc::mma_commit(&misc->o_full);
          }
          __syncwarp();
        }
        ++n_items;
      }
    } else if (warp == 6) {
      // ---------------------------------------------------------------- per-item tables, one item ahead of the softmax warps
      const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && a.gate != nullptr;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        const PairItem wi = decode_pair_item(g, a.pair_heads, item);
        const uint32_t tb = seq & 1;
        const int beg_ = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0];
        const int k_ = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1] - beg_;
        const int head_ = (lane < 4 && lane < k_) ? a.col_idx[(size_t)wi.bhq0 * g.nnz_cap + beg_ + lane] : 0;
        int l4[4];
        float g4[4], oc8[8];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int row = lane + 32 * r, m = row >> 6;
          int it_, ih_, iw_;
          cube_coords(g, wi.i0 + m * wi.di, it_, ih_, iw_);
          l4[r] = cube_token(g, it_, ih_, iw_, row & 63);
          g4[r] = (coarse && l4[r] >= 0) ? a.gate[(size_t)(wi.bhq0 + m * wi.dh) * g.L + l4[r]] : 0.f;
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          const int e = lane + 32 * r, m = e >> 7, d = e & 127;
          oc8[r] = (coarse && d < D) ? a.oc_hat[((size_t)(wi.bhq0 + m * wi.dh) * g.N + wi.i0 + m * wi.di) * D + d] : 0.f;
        }
        VSA2_WAIT_PARKED(&misc->tab_free[tb], ((seq >> 1) & 1) ^ 1);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          misc->tok[tb][lane + 32 * r] = l4[r];
          misc->gate[tb][lane + 32 * r] = g4[r];
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) (&misc->oc[tb][0][0])[lane + 32 * r] = oc8[r];
        if (lane < 4) misc->list_head[tb][lane] = head_;
        if (lane == 0) {
          misc->list_k[tb] = k_;
          misc->list_beg[tb] = beg_;
        }
        tc::mbar_arrive(&misc->tab_full[tb]);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (2 x 128 threads)
    tc::reg_inc<200>();
    const int wg = (warp >> 2) - 2;              // 0 or 1: the tiles with (global tile index & 1) == wg
    const int quad = warp & 3;
    const int row = (quad << 5) | lane;          // query row of the item (0..127) = tensor-memory lane
    const int member = row >> 6;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t tg = 0, n_items = 0, all_phase = 0;
    for (uint32_t n_all = 0;; ++n_all) {
      VSA2_NEXT_ITEM(item, n_all);
      const PairItem wi = decode_pair_item(g, a.pair_heads, item);
      const int tb = n_all & 1;
      VSA2_WAIT(&misc->tab_full[tb], (n_all >> 1) & 1);
      const int k = misc->list_k[tb];
      const int* cols = a.col_idx + (size_t)wi.bhq0 * g.nnz_cap + misc->list_beg[tb];
      const int* head = misc->list_head[tb];
      if (wg == 0 && row < 2) misc->rescue_flag[row] = 0;
      const int nt = (k + 1) >> 1;
      const uint32_t tg0 = tg;
      float m_row = 0.f;
      if (k > 0 && (tg & 1) == (uint32_t)wg) {
        // this warpgroup owns tile 0: reference exponent of its row = exact row maximum of that tile (thread-local)
        const uint32_t buf = tg & 1;
        const unsigned long long ma = misc->vmask[edge[head[0]]], mb = k > 1 ? misc->vmask[edge[head[1]]] : 0ull;
        VSA2_WAIT(&misc->s_full[buf], (tg >> 1) & 1);
        tc::tc_fence_after();
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t sv[32];
          tc::tmem_ld32(lane_addr + C::TM_S + buf * 128 + 32 * c, sv);
          tc::tmem_ld_wait();
          const unsigned vm = (unsigned)((c < 2 ? ma : mb) >> (32 * (c & 1)));
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if ((vm >> e) & 1u) mx = fmaxf(mx, __uint_as_float(sv[e]));
        }
        misc->m_ref[row] = (mx > -INFINITY) ? mx * c2 : 0.f;
      }
      VSA2_GROUP_SYNC(&misc->all_sync, all_phase);       // reference exponents visible to both warpgroups

      float l_sum = 0.f, r_sum = 0.f;                     // exact sum and sum of the bf16 roundings of this row
      if (k > 0) {
        m_row = misc->m_ref[row];
        const int t_first = ((tg0 & 1) == (uint32_t)wg) ? 0 : 1;
        int ja = head[2 * t_first < k ? 2 * t_first : 0], jb = head[2 * t_first + 1 < k ? 2 * t_first + 1 : 0];
        for (int t = t_first; t < nt; t += 2) {
          const uint32_t tgt = tg0 + t, buf = tgt & 1;
          const bool dup = 2 * t + 1 >= k;
          const unsigned long long ma = misc->vmask[edge[ja]], mb = dup ? 0ull : misc->vmask[edge[jb]];
          if (t + 2 < nt) {
            ja = cols[2 * t + 4];
            jb = cols[2 * t + 5 < k ? 2 * t + 5 : 2 * t + 4];
          }
          const bool fast = (ma & mb) == ~0ull;
          VSA2_WAIT(&misc->s_full[buf], (tgt >> 1) & 1);
          tc::tc_fence_after();
          VSA2_WAIT(&misc->p_free[buf], ((tgt >> 1) & 1) ^ 1);      // (the P buffer: PV of the tile two back has read it)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t sv[32], pk[16];
            tc::tmem_ld32(lane_addr + C::TM_S + buf * 128 + 32 * c, sv);
            tc::tmem_ld_wait();
            if (c == 3) {
              tc::tc_fence_before();
              tc::mbar_arrive(&misc->s_free[buf]);
            }
            const unsigned vm = (unsigned)((c < 2 ? ma : mb) >> (32 * (c & 1)));
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              float p0 = ex2_approx(fmaf(__uint_as_float(sv[2 * e]), c2, -m_row));
              float p1 = ex2_approx(fmaf(__uint_as_float(sv[2 * e + 1]), c2, -m_row));
              if (!fast) {
                p0 = ((vm >> (2 * e)) & 1u) ? p0 : 0.f;
                p1 = ((vm >> (2 * e + 1)) & 1u) ? p1 : 0.f;
              }
              l_sum += p0 + p1;
              const uint32_t w = pack_bf16x2(p0, p1);
              r_sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
              pk[e] = w;
            }
            tc::tmem_st_32x32b_x16(lane_addr + C::TM_P + buf * 64 + 16 * c, pk);
          }
          tc::tmem_st_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->p_ready[buf]);
        }
        tg += nt;
        misc->red[wg][0][row] = l_sum;
        misc->red[wg][1][row] = r_sum;
      }
      VSA2_GROUP_SYNC(&misc->all_sync, all_phase);
      const int bhq = wi.bhq0 + member * wi.dh;
      const int tk = misc->tok[tb][row];
      float inv = 0.f;
      if (k > 0) {
        const float l = misc->red[0][0][row] + misc->red[1][0][row], r = misc->red[0][1][row] + misc->red[1][1][row];
        inv = 1.f / r;
        if (wg == 0) {
          if (!(l > 1e-30f && l < 1e30f && r > 1e-30f)) misc->rescue_flag[member] = 1;
          if (tk >= 0) a.lse[(size_t)bhq * g.L + tk] = (m_row + __log2f(l)) * 0.6931471805599453f;
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
      } else if (wg == 0 && tk >= 0) {
        a.lse[(size_t)bhq * g.L + tk] = -INFINITY;
      }

      // O[l, d] = O_acc[q, d] / (rounded row sum) + gate[q] * O_c[d]; this warpgroup writes D / 2 channels of every row
      {
        constexpr int COLS = D / 2;
        const float gt = misc->gate[tb][row];
        const float* oc = misc->oc[tb][member];
#pragma unroll
        for (int c = 0; c < COLS / 32; ++c) {
          const int col0 = wg * COLS + 32 * c;
          uint32_t acc[32];
          if (k > 0) {
            tc::tmem_ld32(lane_addr + C::TM_O + col0, acc);
            tc::tmem_ld_wait();
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] = 0u;
          }
          if (tk >= 0) {
            const size_t idx = ((size_t)bhq * g.L + tk) * D + col0;
            if (g.out_f32) {
              float* dst = reinterpret_cast<float*>(a.o) + idx;
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4*>(dst + e) =
                    make_float4(fmaf(gt, oc[col0 + e], __uint_as_float(acc[e]) * inv), fmaf(gt, oc[col0 + e + 1], __uint_as_float(acc[e + 1]) * inv),
                                fmaf(gt, oc[col0 + e + 2], __uint_as_float(acc[e + 2]) * inv), fmaf(gt, oc[col0 + e + 3], __uint_as_float(acc[e + 3]) * inv));
            } else {
              bf16* dst = reinterpret_cast<bf16*>(a.o) + idx;
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  split_bf16x2(fmaf(gt, oc[col0 + e + 2 * q], __uint_as_float(acc[e + 2 * q]) * inv),
                               fmaf(gt, oc[col0 + e + 2 * q + 1], __uint_as_float(acc[e + 2 * q + 1]) * inv), hi[q], lo[q]);
                *reinterpret_cast<uint4*>(dst + e) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                if (a.o_res != nullptr) *reinterpret_cast<uint4*>(a.o_res + idx + e) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
              }
            }
          }
        }
        if (k > 0) {
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        }
      }
      VSA2_GROUP_SYNC(&misc->all_sync, all_phase);       // rescue flags complete
      tc::mbar_arrive(&misc->tab_free[tb]);
      if (k > 0 && wg == 0 && row < 2 && misc->rescue_flag[row]) {
        // the exact kernel works on 64-token blocks: one list entry per member whose sums left the safe range
        const int slot = atomicAdd(a.rescue_count, 1);
        if (slot < a.rescue_cap) a.rescue_items[slot] = block_item(g, wi.bhq0 + row * wi.dh, wi.i0 + row * wi.di);
        else atomicExch(&a.status->status, VSA2_ERR_UNSUPPORTED);
      }
      if (k > 0) ++n_items;
    }
  }

done:
  tc::tc_fence_before();
  __syncthreads();
  if (misc->abort_flag) {
    if (tid == 0) atomicExch(&a.status->status, VSA2_ERR_DEVICE_TIMEOUT);
    if (tid == 0) {
      const unsigned long long t0 = tc::global_timer_ns();
      while (tc::global_timer_ns() - t0 < 200000ull) {
      }
    }
    __syncthreads();
  }
  if (warp == 4) tc::tmem_dealloc(tmem_base, 512);
}

cudaError_t launch_fine_fwd_list(const Geo& g, const int* count, int cap, const int* items, const bf16* q, const bf16* k,
                                 const bf16* v, const float* gate, const int* row_ptr, const int* col_idx,
                                 const float* oc_hat, void* o, bf16* o_res, float* lse, cudaStream_t st);

bool fine_fwd_rows2_supported(const Geo& g, bool pair_heads) {
  return g.Lt == 0 && g.N <= kF2MaxCubes && (pair_heads ? (g.rep % 2 == 0) : (g.N % 2 == 0));
}

// pair_heads = false: `g` is the half-cube geometry of a 128-token-cube problem, row_ptr / col_idx the expanded map, oc_hat per
// half-cube.  pair_heads = true: `g` is an ordinary 64-token-cube problem with an even number of query heads per KV head whose
// maps are identical inside each group (group-shared routing); consecutive heads are paired.  Workspace as for the 64-query kernel.
cudaError_t launch_fine_fwd_rows2_tc(const Geo& g, bool pair_heads, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                                     const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                                     float* lse, StatusBlock* status, cudaStream_t st) {
  if (!fine_fwd_rows2_supported(g, pair_heads)) return cudaErrorInvalidValue;
  CUtensorMap tq, tk, tv;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  FwdRows2Args a;
  a.pair_heads = pair_heads ? 1 : 0;
  a.gate = gate; a.row_ptr = row_ptr; a.col_idx = col_idx; a.oc_hat = oc_hat; a.o = o; a.o_res = o_res; a.lse = lse;
  a.status = status;
  a.rescue_count = &status->pad[0];
  a.item_counter = &status->pad[1];
  a.rescue_items = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(status) + 256);
  a.rescue_cap = fwd_rescue_capacity();
  const int total = g.batch * g.Hq * g.N / 2;
  const int grid = total < sms ? total : sms;
  {
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, g.D == 128 ? (const void*)fine_fwd_rows2_tc_kernel<128> : (const void*)fine_fwd_rows2_tc_kernel<64>)) != cudaSuccess) return e;
    if (fa.numRegs * kF2Threads < 256 * 56 + 256 * 200) return cudaErrorLaunchOutOfResources;
  }
  if (g.D == 128) {
    const size_t smb = FwdRows2<128>::smem_bytes(g.N);
    if (smb > 227 * 1024) return cudaErrorInvalidValue;
    if ((e = cudaFuncSetAttribute(fine_fwd_rows2_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_rows2_tc_kernel<128><<<grid, kF2Threads, smb, st>>>(tq, tk, tv, g, a);
  } else {
    const size_t smb = FwdRows2<64>::smem_bytes(g.N);
    if ((e = cudaFuncSetAttribute(fine_fwd_rows2_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_rows2_tc_kernel<64><<<grid, kF2Threads, smb, st>>>(tq, tk, tv, g, a);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  return launch_fine_fwd_list(g, a.rescue_count, a.rescue_cap, a.rescue_items, q, k, v, gate, row_ptr, col_idx, oc_hat, o, o_res, lse, st);
}

}  // namespace vsa2
