// Fine branch forward (paper Eq. 12) + gated merge (Eq. 14) for cubes of 128 tokens, on the Blackwell tensor cores.
//
// A query cube of 128 tokens is two 64-token half-cubes that keep the same KV cubes, so both halves ride on the same
// operand tiles: the products of fine_fwd_tc.cu are taken with N = 128 query columns,
//     S^T [128 kv, 128 q] = K_pair [128, D] * Q_pair^T        (M = 128 keys,   N = 128 queries, K = D)
//     O^T [D,      128 q] += V_pair^T [D, 128] * P^T          (M = D channels, N = 128 queries, K = 128 keys)
// where K_pair / V_pair are the two halves of ONE key cube and Q_pair the two halves of the query cube.  Per FLOP this
// halves the TMA traffic into shared memory and cuts the operand fetches of the MMAs by a third against the N = 64
// kernel, which is bound by exactly that traffic.
//
// The kernel works on the half-cube problem (geometry, expanded block map, per-half coarse rows) that the library
// builds for 128-token cubes: row 2c of the expanded map lists the half-cubes (2j, 2j+1, ...) of query cube c.
//
// Roles (640 threads): warp 0 = TMA producer of the K pairs and the Q pair (lane 0 is also the CTA's scheduler), warp 1
// = TMA producer of the V pairs, warp 2 = issuer of S^T, warp 3 = issuer of O^T, then four softmax + epilogue
// warpgroups: warpgroup w owns query columns 32w .. 32w+31 of EVERY tile (its thread r holds key row r of them), so
// each keeps its own reference exponents, row sums and output rows and they meet only at the operand barriers and once
// per cube.  With 32 columns per thread the role fits the 96 registers a 640-thread CTA gets, so no register
// re-balancing is needed.  Softmax as in fine_fwd_tc.cu: fixed reference exponent per query column (exact column
// maximum of the first tile), row sums checked at the end, a half-cube whose sums left the safe range goes to the
// exact-maximum kernel.  (One reference for all columns would save re-reading 4 KB of references per warp and tile
// from shared memory, 5 % of the time; but with its own maximum as reference a column's largest P of the first tile
// is exactly 1, while any other reference rounds it to bf16 and scales the whole output row of a sharply peaked query
// by up to 2^-9 against its fp32 row sum, which the backward amplifies: measured dK error 5e-2 instead of 1e-2.)
// Every wait is bounded.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kFwwThreads = 640;      // 4 service warps + 4 softmax warpgroups
constexpr int kFwwKSlots = 2;
constexpr int kFwwVSlots = 2;
constexpr int kFwwSBufs = 2;          // S^T buffers of 128 columns
constexpr int kFwwRescueCap = 16384;  // must match the list the N = 64 launcher sizes (fine_fwd_tc_workspace_bytes)
constexpr int kFwwMaxCubes = 12288;

template <int D>
struct FwdWide {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLAB = kSlab;
  static constexpr uint32_t SLOT = 2 * DH * SLAB;    // a K, V or Q pair: [channel half][block A | block B]
  static constexpr uint32_t PBYTES = 128 * 128;      // P^T of one query half: 128 key rows x 64 queries bf16
  static constexpr uint32_t OFF_Q = (kFwwKSlots + kFwwVSlots) * SLOT;
  static constexpr uint32_t OFF_P = OFF_Q + SLOT;
  static constexpr uint32_t OFF_MISC = OFF_P + 2 * PBYTES;
  static constexpr uint32_t MISC_BYTES = 6144;
  static size_t smem_bytes(int n_half_cubes) { return OFF_MISC + MISC_BYTES + ((size_t)n_half_cubes + 15) / 16 * 16 + 1024; }
};

struct FwdWideMisc {
  uint64_t q_full, q_empty, o_full, o_empty;
  uint64_t k_full[kFwwKSlots], k_empty[kFwwKSlots];
  uint64_t v_full[kFwwVSlots], v_empty[kFwwVSlots];
  uint64_t s_full[kFwwSBufs], s_free[kFwwSBufs];
  uint64_t p_ready, p_free;
  ItemQueue items;
  uint64_t wg_sync[4], all_sync;   // group barriers of one softmax warpgroup (128 threads) and of all four (512)
  uint32_t tmem_base;
  int abort_flag;
  int rescue_flag[4];
  alignas(16) float m_ref[128];    // per query column of the cube: reference exponent (log2 units)
  alignas(16) float l_inv[128];
  alignas(16) float red[16][32];   // per-warp partial column reductions (warps 4w .. 4w+3 belong to warpgroup w)
  int tok[2][128];                 // [item parity][query column]: raster token (-1 = padding)
  float gate[2][128];
};
static_assert(sizeof(FwdWideMisc) <= 6144, "misc region too small");

struct FwdWideArgs {
  int pair_heads;       // 0: an item is a query cube of 128 tokens (two half-cubes of one head); 1: an item is one query
                        // block of two consecutive query heads of a KV group whose maps are identical
  int* item_counter;    // global, zero before the launch
  const float* gate;
  const int* row_ptr;   // expanded map (half-cube level)
  const int* col_idx;
  const float* oc_hat;  // per half-cube
  void* o;
  bf16* o_res;
  float* lse;
  StatusBlock* status;
  int* rescue_count;
  int* rescue_items;
  int rescue_cap;       // entries the list holds
};

// The two "members" of an item share their list of key blocks: member m is query block i0 + m * di of head bhq0 + m * dh;
// the list is row i0 of head bhq0.
struct WideItem {
  int bhq0, i0, dh, di;
};
__device__ __forceinline__ WideItem decode_item(const Geo& g, int pair_heads, int item) {
  WideItem w;
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

// acc[128, 128] = A_pair[128, D] * B_pair[128, D]^T, both operands in the [channel half][block A | block B] layout
template <int D>
__device__ __forceinline__ void mma_pair_pair_kmajor(uint32_t tm_acc, uint32_t a_slot, uint32_t b_slot) {
  constexpr uint32_t idesc = tc::idesc_bf16(128, 128, false, false);
  const uint64_t da = tc::smem_desc_sw128(a_slot, 16, 1024), db = tc::smem_desc_sw128(b_slot, 16, 1024);
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const uint64_t off = (uint64_t)(((ks / 4) * 2 * kSlab + (ks % 4) * 32) >> 4);
    tc::mma_ss(tm_acc, da + off, db + off, idesc, ks > 0);
  }
}

// acc[D, 128] (+)= A_pair^T[D, 128] * B[128, 128]: A_pair a slot (rows = the 128 keys), B two 128-row swizzled tiles of
// 64 query columns each, `b_stride` bytes apart
template <int D>
__device__ __forceinline__ void mma_pairT_wide_mnmajor(uint32_t tm_acc, uint32_t a_slot, uint32_t b_tile, uint32_t b_stride,
                                                       bool accumulate_first) {
  constexpr uint32_t idesc = tc::idesc_bf16(128, 128, true, true);
  constexpr uint32_t lbo = (D == 128) ? 2 * kSlab : 0;
  const uint64_t da = tc::smem_desc_sw128(a_slot, lbo, 1024), db = tc::smem_desc_sw128(b_tile, b_stride, 1024);
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint64_t oa = (uint64_t)(((ks / 4) * kSlab + (ks % 4) * 2048) >> 4);
    const uint64_t ob = (uint64_t)((ks * 2048) >> 4);
    tc::mma_ss(tm_acc, da + oa, db + ob, idesc, accumulate_first || (ks > 0));
  }
}

template <int D>
__global__ void __launch_bounds__(kFwwThreads, 1)
fine_fwd_wide_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, Geo g, FwdWideArgs a) {
  using C = FwdWide<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = smem + C::OFF_Q;
  unsigned char* p_tile = smem + C::OFF_P;
  FwdWideMisc* misc = reinterpret_cast<FwdWideMisc*>(smem + C::OFF_MISC);
  unsigned char* edge = smem + C::OFF_MISC + C::MISC_BYTES;      // edge flags of every half-cube

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hq * g.N / 2;              // pairs of query blocks either way
  const float c2 = g.scale * 1.4426950408889634f;

  for (int n = tid; n < g.N; n += blockDim.x) edge[n] = (unsigned char)cube_edge_flags(g, n);
  if (tid == 0) {
    misc->abort_flag = 0;
    tc::mbar_init(&misc->q_full, 1);
    tc::mbar_init(&misc->q_empty, 1);
    tc::mbar_init(&misc->o_full, 1);
    tc::mbar_init(&misc->o_empty, 512);
    for (int s = 0; s < kFwwKSlots; ++s) {
      tc::mbar_init(&misc->k_full[s], 1);
      tc::mbar_init(&misc->k_empty[s], 1);
    }
    for (int s = 0; s < kFwwVSlots; ++s) {
      tc::mbar_init(&misc->v_full[s], 1);
      tc::mbar_init(&misc->v_empty[s], 1);
    }
    for (int s = 0; s < kFwwSBufs; ++s) {
      tc::mbar_init(&misc->s_full[s], 1);
      tc::mbar_init(&misc->s_free[s], 512);
    }
    tc::mbar_init(&misc->p_ready, 512);
    tc::mbar_init(&misc->p_free, 1);
    for (int s = 0; s < 4; ++s) tc::mbar_init(&misc->wg_sync[s], 128);
    tc::mbar_init(&misc->all_sync, 512);
    item_queue_init(&misc->items, 2 + 2 + 512);     // lane 0 of the producers, two issuers, the softmax threads
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
  }
  if (warp == 2) {
    tc::tmem_alloc(&misc->tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  // tensor-memory columns: S^T buffers at 0 and 128; O^T at 256 .. 383

  if (warp < 4) {
    if (warp < 2) {
      // ---------------------------------------------------------------- TMA producers
      const int which = warp;                               // 0: K ring (+ Q pair), 1: V ring
      const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
      const uint32_t nslots = which == 0 ? kFwwKSlots : kFwwVSlots;
      uint64_t* full = which == 0 ? misc->k_full : misc->v_full;
      uint64_t* empty = which == 0 ? misc->k_empty : misc->v_empty;
      unsigned char* ring = smem + (which == 0 ? 0 : kFwwKSlots * C::SLOT);
      const int my_h = lane >> 1, my_blk = lane & 1;
      const bool issuer = lane < 2 * C::DH;
      uint32_t tg = 0, n_items = 0, published = 0;
      for (uint32_t seq = 0;; ++seq) {
        int item = 0;
        if (lane == 0) {
          if (which == 0 && !item_publish_ahead(&misc->items, seq, published, a.item_counter, total_items, &misc->abort_flag)) item = -2;
          else item = item_get(&misc->items, seq, &misc->abort_flag);
        }
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item == -2) goto done;
        if (item < 0) break;
        const WideItem wi = decode_item(g, a.pair_heads, item);
        const int bhq = wi.bhq0;
        const int b = bhq / g.Hq, hq = bhq % g.Hq, bhk = b * g.Hkv + hq / g.rep;
        const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + wi.i0], end = a.row_ptr[(size_t)bhq * (g.N + 1) + wi.i0 + 1];
        const int k = end - beg;
        const int nt = (k + 1) >> 1;                        // two key blocks per tile (an odd list repeats its last block)
        if (nt == 0) continue;
        const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
        if (which == 0) {
          int it_, ih_, iw_;
          cube_coords(g, wi.i0 + my_blk * wi.di, it_, ih_, iw_);
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&misc->q_empty, (n_items & 1) ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&misc->q_full, C::SLOT);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (issuer)
            tc::tma_load_5d(q_tile + (2 * my_h + my_blk) * C::SLAB, &tm_q, &misc->q_full, my_h * 64, iw_ * g.Bw, ih_ * g.Bh,
                            it_ * g.Bt, bhq + my_blk * wi.dh);
        }
        ++n_items;
        int j = cols[(my_blk == 1 && k > 1) ? 1 : 0];
        for (int t = 0; t < nt; ++t, ++tg) {
          int jt, jh, jw;
          cube_coords(g, j, jt, jh, jw);
          if (t + 1 < nt) j = cols[(my_blk == 1 && 2 * t + 3 < k) ? 2 * t + 3 : 2 * t + 2];   // next tile, fetched early
          const uint32_t slot = tg % nslots, par = (tg / nslots) & 1;
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&empty[slot], par ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&full[slot], C::SLOT);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (issuer)
            tc::tma_load_5d(ring + slot * C::SLOT + (2 * my_h + my_blk) * C::SLAB, tm, &full[slot], my_h * 64,
                            jw * g.Bw, jh * g.Bh, jt * g.Bt, bhk);
        }
      }
    } else if (warp == 2) {
      // ---------------------------------------------------------------- issuer of S^T(t) = K_pair * Q_pair^T
      if (lane == 0) {
        const uint32_t q_addr = tc::smem_u32(q_tile), slot0 = tc::smem_u32(smem);
        uint32_t tg = 0, n_items = 0;
        for (uint32_t seq = 0;; ++seq) {
          VSA2_NEXT_ITEM(item, seq);
          const WideItem wi = decode_item(g, a.pair_heads, item);
          const int nt = (a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1] - a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0] + 1) >> 1;
          if (nt == 0) continue;
          VSA2_WAIT(&misc->q_full, n_items & 1);
          for (int t = 0; t < nt; ++t, ++tg) {
            const uint32_t slot = tg % kFwwKSlots, buf = tg % kFwwSBufs;
            VSA2_WAIT(&misc->k_full[slot], (tg / kFwwKSlots) & 1);
            VSA2_WAIT(&misc->s_free[buf], ((tg / kFwwSBufs) & 1) ^ 1);
            tc::tc_fence_after();
            mma_pair_pair_kmajor<D>(tmem_base + buf * 128, slot0 + slot * C::SLOT, q_addr);
            tc::mma_commit(&misc->s_full[buf]);
            tc::mma_commit(&misc->k_empty[slot]);
          }
          tc::mma_commit(&misc->q_empty);          // the Q pair may be replaced once these products are done
          ++n_items;
        }
      }
    } else {
      // ---------------------------------------------------------------- issuer of O^T += V_pair^T * P^T (warp 3)
      if (lane == 0) {
        const uint32_t p_addr = tc::smem_u32(p_tile), slot0 = tc::smem_u32(smem);
        const uint32_t tm_o = tmem_base + 256;
        uint32_t tg = 0, n_items = 0;
        for (uint32_t seq = 0;; ++seq) {
          VSA2_NEXT_ITEM(item, seq);
          const WideItem wi = decode_item(g, a.pair_heads, item);
          const int nt = (a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1] - a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0] + 1) >> 1;
          if (nt == 0) continue;
          VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);      // the previous cube's accumulator was read out
          for (int t = 0; t < nt; ++t, ++tg) {
            const uint32_t slot = tg % kFwwVSlots;
            VSA2_WAIT(&misc->v_full[slot], (tg / kFwwVSlots) & 1);
            VSA2_WAIT(&misc->p_ready, tg & 1);
            tc::tc_fence_after();
            mma_pairT_wide_mnmajor<D>(tm_o, slot0 + (kFwwKSlots + slot) * C::SLOT, p_addr, C::PBYTES, t > 0);
            tc::mma_commit(&misc->v_empty[slot]);
            tc::mma_commit(&misc->p_free);
          }
          tc::mma_commit(&misc->o_full);
          ++n_items;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (4 x 128 threads)
    const int wg = (warp - 4) >> 2;              // warpgroup 0..3: query columns 32 wg .. 32 wg + 31 of every tile
    const int half = wg >> 1;                    // the query half-cube those columns belong to
    const int quad = warp & 3;
    const int row = (quad << 5) | lane;          // tensor-memory lane: key row in S^T, channel in O^T
    const int sm_tid = (tid - 128) & 127;
    const int sm_warp = warp - 4;                // 4 * wg + quad
    const int q0 = 32 * wg;                      // first query column (0..127 over the cube) of this warpgroup
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && a.gate != nullptr;
    unsigned char* p_row = p_tile + half * C::PBYTES + row * 128;   // this thread's key row of P^T of its query half
    const int chunk0 = (wg & 1) * 4;             // its 32 queries are the 16-byte chunks chunk0 .. chunk0 + 3 of that row
    CubePos cpos;
    cpos.init(g, row & 63);
    const int blk = row >> 6;                    // which half of the key cube this thread's row belongs to
    uint32_t tg = 0, n_items = 0, n_all = 0, wg_phase = 0;
    for (;; ++n_all) {
      VSA2_NEXT_ITEM(item, n_all);
      const WideItem wi = decode_item(g, a.pair_heads, item);
      const int bhq = wi.bhq0 + half * wi.dh;    // head and query block of this warpgroup's member
      const int i = wi.i0 + half * wi.di;
      const int beg = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0], end = a.row_ptr[(size_t)wi.bhq0 * (g.N + 1) + wi.i0 + 1];
      const int k = end - beg;
      const int nt = (k + 1) >> 1;
      const int* cols = a.col_idx + (size_t)wi.bhq0 * g.nnz_cap + beg;
      const int tb = n_all & 1;
      if (sm_tid < 32) {
        int it_, ih_, iw_;
        cube_coords(g, i, it_, ih_, iw_);
        const int l = cube_token(g, it_, ih_, iw_, (q0 + sm_tid) & 63);
        misc->tok[tb][q0 + sm_tid] = l;
        misc->gate[tb][q0 + sm_tid] = (coarse && l >= 0) ? a.gate[(size_t)bhq * g.L + l] : 0.f;
      }
      const float oc_d = (coarse && row < D) ? a.oc_hat[((size_t)bhq * g.N + i) * D + row] : 0.f;
      if (sm_tid == 0) misc->rescue_flag[wg] = 0;

      float l_part[32];
#pragma unroll
      for (int cc = 0; cc < 32; ++cc) l_part[cc] = 0.f;
      const uint32_t tg0 = tg;
      if (nt > 0) {
        // reference exponent of this warpgroup's query columns = exact column maximum of the first tile
        const uint32_t buf = tg % kFwwSBufs;
        const bool valid = !((blk == 1) && k < 2) && cpos.valid(edge[cols[(blk == 1 && k > 1) ? 1 : 0]], g);
        VSA2_WAIT(&misc->s_full[buf], (tg / kFwwSBufs) & 1);
        tc::tc_fence_after();
        uint32_t s0[32];
        tc::tmem_ld32(lane_addr + buf * 128 + q0, s0);
        tc::tmem_ld_wait();
        float mx[32];
#pragma unroll
        for (int cc = 0; cc < 32; ++cc) mx[cc] = valid ? __uint_as_float(s0[cc]) : -INFINITY;
        warp_reduce_cols32<true>(mx, lane);
        misc->red[sm_warp][lane] = mx[0];
        VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);
        if (sm_tid < 32) {
          const float m4 = fmaxf(fmaxf(misc->red[4 * wg][sm_tid], misc->red[4 * wg + 1][sm_tid]),
                                 fmaxf(misc->red[4 * wg + 2][sm_tid], misc->red[4 * wg + 3][sm_tid]));
          misc->m_ref[q0 + sm_tid] = (m4 > -INFINITY) ? m4 * c2 : 0.f;
        }
      }
      VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);       // tables and reference exponents visible to the warpgroup

      if (nt > 0) {
        int j_next = cols[(blk == 1 && k > 1) ? 1 : 0];
        for (int t = 0; t < nt; ++t) {
          const uint32_t tgt = tg0 + t, buf = tgt % kFwwSBufs;
          const bool dup = (blk == 1) && (2 * t + 1 >= k);       // odd list: the last tile holds one key block twice
          const bool valid = !dup && cpos.valid(edge[j_next], g);
          if (t + 1 < nt) j_next = cols[(blk == 1 && 2 * t + 3 < k) ? 2 * t + 3 : 2 * t + 2];
          const bool all_valid = __all_sync(0xffffffffu, valid);
          VSA2_WAIT(&misc->s_full[buf], (tgt / kFwwSBufs) & 1);
          tc::tc_fence_after();
          uint32_t sa[32];
          tc::tmem_ld32(lane_addr + buf * 128 + q0, sa);
          tc::tmem_ld_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->s_free[buf]);
          uint32_t packed[16];
          const float4* mref4 = reinterpret_cast<const float4*>(misc->m_ref + q0);
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            const float4 m = mref4[c4];
            float p0 = ex2_approx(fmaf(__uint_as_float(sa[4 * c4 + 0]), c2, -m.x));
            float p1 = ex2_approx(fmaf(__uint_as_float(sa[4 * c4 + 1]), c2, -m.y));
            float p2 = ex2_approx(fmaf(__uint_as_float(sa[4 * c4 + 2]), c2, -m.z));
            float p3 = ex2_approx(fmaf(__uint_as_float(sa[4 * c4 + 3]), c2, -m.w));
            if (!all_valid) { p0 = valid ? p0 : 0.f; p1 = valid ? p1 : 0.f; p2 = valid ? p2 : 0.f; p3 = valid ? p3 : 0.f; }
            l_part[4 * c4 + 0] += p0;
            l_part[4 * c4 + 1] += p1;
            l_part[4 * c4 + 2] += p2;
            l_part[4 * c4 + 3] += p3;
            packed[2 * c4] = pack_bf16x2(p0, p1);
            packed[2 * c4 + 1] = pack_bf16x2(p2, p3);
          }
          VSA2_WAIT(&misc->p_free, (tgt & 1) ^ 1);           // the previous tile's O^T product has read P^T
#pragma unroll
          for (int ch = 0; ch < 4; ++ch)
            *reinterpret_cast<uint4*>(p_row + (((chunk0 + ch) ^ (row & 7)) << 4)) =
                make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
          tc::fence_proxy_async_smem();
          tc::mbar_arrive(&misc->p_ready);
        }
        tg += nt;

        // ---- epilogue of these 32 query columns: row sums over the 128 key rows x tiles
        warp_reduce_cols32<false>(l_part, lane);
        misc->red[sm_warp][lane] = l_part[0];
        VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);
        if (sm_tid < 32) {
          const float l = (misc->red[4 * wg][sm_tid] + misc->red[4 * wg + 1][sm_tid]) +
                          (misc->red[4 * wg + 2][sm_tid] + misc->red[4 * wg + 3][sm_tid]);
          if (!(l > 1e-30f && l < 1e30f)) misc->rescue_flag[wg] = 1;
          misc->l_inv[q0 + sm_tid] = 1.f / l;
          const int tk = misc->tok[tb][q0 + sm_tid];
          if (tk >= 0) a.lse[(size_t)bhq * g.L + tk] = (misc->m_ref[q0 + sm_tid] + __log2f(l)) * 0.6931471805599453f;
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
        VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);
      }

      // O[l, d] = O^T[d, q] / l[q] + gate[q] * O_c[d] for the 32 queries of this warpgroup
      {
        float acc[32];
        if (nt > 0) {
          uint32_t o0[32];
          tc::tmem_ld32(lane_addr + 256 + q0, o0);
          tc::tmem_ld_wait();
#pragma unroll
          for (int cc = 0; cc < 32; ++cc) acc[cc] = __uint_as_float(o0[cc]);
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        } else {
#pragma unroll
          for (int cc = 0; cc < 32; ++cc) acc[cc] = 0.f;
        }
        if (row < D) {
#pragma unroll
          for (int qq = 0; qq < 32; ++qq)
            acc[qq] = fmaf(misc->gate[tb][q0 + qq], oc_d, nt > 0 ? acc[qq] * misc->l_inv[q0 + qq] : 0.f);
        }
        if (g.out_f32 || a.o_res == nullptr) {
          // plain stores (validation paths): one element per thread and query
          if (row < D) {
#pragma unroll
            for (int qq = 0; qq < 32; ++qq) {
              const int l = misc->tok[tb][q0 + qq];
              if (l < 0) continue;
              const size_t idx = ((size_t)bhq * g.L + l) * D + row;
              store_out(a.o, idx, acc[qq], g.out_f32);
              if (a.o_res != nullptr) a.o_res[idx] = __float2bfloat16_rn(acc[qq] - __bfloat162float(__float2bfloat16_rn(acc[qq])));
            }
          }
        } else {
          // bf16 output, then its rounding residual: transpose through this warpgroup's quarter of the P^T region (idle
          // now: every product of the cube has completed), 16-byte stores
          bf16* st = reinterpret_cast<bf16*>(p_tile) + (size_t)wg * 32 * D;      // [32 q][D]
          constexpr int CH = D / 8;                                      // 16-byte chunks per token row
#pragma unroll 1
          for (int round = 0; round < 2; ++round) {
            if (row < D) {
#pragma unroll
              for (int qq = 0; qq < 32; ++qq) {
                const bf16 vb = __float2bfloat16_rn(acc[qq]);
                st[qq * D + row] = round == 0 ? vb : __float2bfloat16_rn(acc[qq] - __bfloat162float(vb));
              }
            }
            VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);
            bf16* dst = round == 0 ? reinterpret_cast<bf16*>(a.o) : a.o_res;
            for (int e = sm_tid; e < 32 * CH; e += 128) {
              const int qi = e / CH, ch = e % CH;
              const int l = misc->tok[tb][q0 + qi];
              if (l < 0) continue;
              *reinterpret_cast<uint4*>(dst + ((size_t)bhq * g.L + l) * D + ch * 8) =
                  *reinterpret_cast<const uint4*>(st + qi * D + ch * 8);
            }
            VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);    // staging buffer free before it is rewritten
          }
        }
      }
      if (nt == 0 && sm_tid < 32 && misc->tok[tb][q0 + sm_tid] >= 0)
        a.lse[(size_t)bhq * g.L + misc->tok[tb][q0 + sm_tid]] = -INFINITY;
      if (nt > 0 && sm_tid == 0 && misc->rescue_flag[wg]) {
        int slot = atomicAdd(a.rescue_count, 1);
        if (slot < a.rescue_cap) a.rescue_items[slot] = block_item(g, bhq, i);      // half-cube item in the list kernel's numbering
        else atomicExch(&a.status->status, VSA2_ERR_UNSUPPORTED);
      }
      if (nt > 0) ++n_items;
      // a warpgroup's staging quarter lies inside the P^T half that two warpgroups write: nobody starts the next
      // cube's P^T before every warpgroup has drained its staging area
      VSA2_GROUP_SYNC_AT(&misc->all_sync, n_all);
    }
  }

done:
  tc::tc_fence_before();
  __syncthreads();
  if (misc->abort_flag) {
    if (tid == 0) atomicExch(&a.status->status, VSA2_ERR_DEVICE_TIMEOUT);
    // let copies that are still in flight land before the CTA's shared memory is released
    if (tid == 0) {
      const unsigned long long t0 = tc::global_timer_ns();
      while (tc::global_timer_ns() - t0 < 200000ull) {
      }
    }
    __syncthreads();
  }
  if (warp == 2) tc::tmem_dealloc(tmem_base, 512);
}

cudaError_t launch_fine_fwd_list(const Geo& g, const int* count, int cap, const int* items, const bf16* q, const bf16* k,
                                 const bf16* v, const float* gate, const int* row_ptr, const int* col_idx,
                                 const float* oc_hat, void* o, bf16* o_res, float* lse, cudaStream_t st);

// pair_heads = false: `g` is the half-cube geometry of a 128-token-cube problem, row_ptr / col_idx the expanded map, oc_hat per
// half-cube.  pair_heads = true: `g` is an ordinary 64-token-cube problem with an even number of query heads per KV head whose
// maps are identical inside each group (group-shared routing); consecutive heads are paired.  Workspace as for the N = 64 launcher.
cudaError_t launch_fine_fwd_wide_tc(const Geo& g, bool pair_heads, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                                    const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                                    float* lse, StatusBlock* status, cudaStream_t st) {
  CUtensorMap tq, tk, tv;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if (fine_fwd_tc_workspace_bytes() < 256 + (size_t)kFwwRescueCap * sizeof(int)) return cudaErrorInvalidValue;
  FwdWideArgs a;
  a.pair_heads = pair_heads ? 1 : 0;
  a.gate = gate; a.row_ptr = row_ptr; a.col_idx = col_idx; a.oc_hat = oc_hat; a.o = o; a.o_res = o_res; a.lse = lse;
  a.status = status;
  a.rescue_count = &status->pad[0];
  a.item_counter = &status->pad[1];
  a.rescue_items = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(status) + 256);
  a.rescue_cap = fwd_rescue_capacity() < kFwwRescueCap ? fwd_rescue_capacity() : kFwwRescueCap;
  const int total = g.batch * g.Hq * g.N / 2;         // pairs of query blocks (Hq or N is even)
  const int grid = total < sms ? total : sms;
  if (g.N > kFwwMaxCubes || (pair_heads ? (g.rep & 1) : (g.N & 1))) return cudaErrorInvalidValue;
  if (g.D == 128) {
    const size_t smb = FwdWide<128>::smem_bytes(g.N);
    if (smb > 227 * 1024) return cudaErrorInvalidValue;
    if ((e = cudaFuncSetAttribute(fine_fwd_wide_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_wide_tc_kernel<128><<<grid, kFwwThreads, smb, st>>>(tq, tk, tv, g, a);
  } else {
    const size_t smb = FwdWide<64>::smem_bytes(g.N);
    if (smb > 227 * 1024) return cudaErrorInvalidValue;
    if ((e = cudaFuncSetAttribute(fine_fwd_wide_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_wide_tc_kernel<64><<<grid, kFwwThreads, smb, st>>>(tq, tk, tv, g, a);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // half-cubes whose row sums left the safe range are redone with the exact running maximum
  return launch_fine_fwd_list(g, a.rescue_count, a.rescue_cap, a.rescue_items, q, k, v, gate, row_ptr, col_idx, oc_hat, o, o_res, lse, st);
}

}  // namespace vsa2
