// Fine branch forward (paper Eq. 12) + gated merge (Eq. 14) on the Blackwell tensor cores.
//
// Formulation.  A query block has only B = 64 tokens, half of the 128 rows a tcgen05 MMA wants, so the
// products are taken transposed and two selected KV blocks are stacked per tile:
//     S^T [128 kv, 64 q] = K_pair [128, D] * Q^T          (M = 128 keys,      N = 64 queries, K = D)
//     O^T [D,      64 q] += V_pair^T [D, 128] * P^T       (M = D channels,    N = 64 queries, K = 128 keys)
// K and V tiles arrive by 5-D TMA straight from the raster tensors (one box = one cube, zero-filled outside
// the grid) into 128-byte-swizzled shared memory; the same V tile that TMA wrote row-per-key is read as an
// MN-major operand, so nothing is transposed in memory.  Accumulators live in tensor memory: four S^T
// buffers (64 columns each) and two O^T accumulators (even and odd tiles, summed in the epilogue).
//
// Softmax.  One thread owns one key row of S^T, so a query's maximum would need a reduction across 128
// threads per tile.  Instead each query column keeps a fixed reference M (the exact column maximum of the
// first tile, in log2 units): P = 2^(s*scale*log2e - M).  Any reference gives the same softmax as long as
// nothing overflows; the row sums are checked at the end of the query block and a block whose sums left
// the safe range is recomputed by the exact-maximum kernel (see fine_fwd.cu).  Row sums are accumulated per
// thread and reduced across the key rows once per query block, deterministically.
//
// Roles (512 threads): two TMA producer warps, four MMA issuer warps, two softmax + epilogue warpgroups (see the
// comment above the kernel).  Persistent CTAs draw their query blocks from a global counter (ItemQueue).  Every wait
// is bounded.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kFwdThreads = 512;
constexpr int kFwdKSlots = 3;   // ring of K pairs: filled by warp 0, drained by the S^T issuers
constexpr int kFwdVSlots = 2;   // ring of V pairs: filled by warp 1, drained by the O^T issuers
constexpr int kFwdSBufs = 4;
constexpr int kRescueCap = 16384;
constexpr int kFwdMaxCubes = 12288;   // edge-flag table in shared memory: one byte per cube

template <int D>
struct FwdTc {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLAB = kSlab;            // one cube x 64 channels
  static constexpr uint32_t SLOT = 2 * DH * SLAB;    // a K pair or a V pair, [half][A | B]
  static constexpr uint32_t QBYTES = DH * SLAB;
  static constexpr uint32_t PBYTES = 128 * 128;      // P^T: 128 key rows x 64 queries bf16
  static constexpr uint32_t OFF_Q = (kFwdKSlots + kFwdVSlots) * SLOT;
  static constexpr uint32_t OFF_P = OFF_Q + QBYTES;
  static constexpr uint32_t OFF_MISC = OFF_P + 2 * PBYTES;
  static constexpr uint32_t MISC_BYTES = 5120;
  static size_t smem_bytes(int n_cubes) { return OFF_MISC + MISC_BYTES + ((size_t)n_cubes + 15) / 16 * 16 + 1024; }
};

struct FwdMisc {
  uint64_t q_full, q_empty, o_full, o_empty;
  uint64_t k_full[kFwdKSlots], k_empty[kFwdKSlots];
  uint64_t v_full[kFwdVSlots], v_empty[kFwdVSlots];
  uint64_t s_full[kFwdSBufs], s_free[kFwdSBufs];
  uint64_t p_ready[2], p_free[2];
  ItemQueue items;                 // work items of this CTA (see tc_attn.cuh)
  uint64_t wg_sync[2], all_sync;   // group barriers of one softmax warpgroup (128 threads) and of both (256)
  uint32_t tmem_base;
  int abort_flag;
  int rescue_flag;
  alignas(16) float m_ref[64];     // per query column: reference exponent (log2 units); read as float4
  alignas(16) float l_inv[64];
  alignas(16) float red[8][64];    // per-warp partial column reductions
  int tok[2][64];                  // raster token of each query position (-1 = padding), by item parity
  float gate[2][64];
};
static_assert(sizeof(FwdMisc) <= 5120, "misc region too small");

struct FwdArgs {
  int* item_counter;    // global, zero before the launch
  const float* gate;
  const int* row_ptr;
  const int* col_idx;
  const float* oc_hat;
  void* o;
  bf16* o_res;
  float* lse;
  StatusBlock* status;
  int* rescue_count;
  int* rescue_items;
  int rescue_cap;       // entries the list holds
};

// Roles (512 threads = 4 warpgroups).  An issuing thread needs ~60 cycles per MMA plus ~100-200 per barrier
// operation, more than the 48 cycles an N = 64 MMA takes to execute, so issue and copy work is spread:
//   warpgroups 0, 1 (few registers): warps 0, 6 = TMA producers of the K pairs (first / second block; warp 0 also
//       brings the Q tile), warps 1, 7 = TMA producers of the V pairs (lane 0 owns the barriers, lanes 0 .. D/64-1 each
//       issue one box), warps 2, 3 = issuers of the S^T products of the even / odd tiles, warps 4, 5 = issuers of the
//       O^T products of the even / odd tiles (each into its own accumulator, summed in the epilogue).
//   warpgroups 2, 3: softmax + epilogue; warpgroup w handles the tiles with (global tile index & 1) == w - 2, so two
//       tiles are in the exponential unit at any time.  A warp owns tensor-memory lane quadrant warp % 4.
// Every mbarrier has one producing role and one consuming role (or all consumers see every phase), so a phase can
// never run two ahead of a waiter.
template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
fine_fwd_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, Geo g, FwdArgs a) {
  using C = FwdTc<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = smem + C::OFF_Q;
  unsigned char* p_tile = smem + C::OFF_P;
  FwdMisc* misc = reinterpret_cast<FwdMisc*>(smem + C::OFF_MISC);
  unsigned char* edge = smem + C::OFF_MISC + C::MISC_BYTES;      // edge flags of every cube

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hq * g.N;
  const float c2 = g.scale * 1.4426950408889634f;

  for (int n = tid; n < g.N; n += blockDim.x) edge[n] = (unsigned char)cube_edge_flags(g, n);
  if (tid == 0) {
    misc->abort_flag = 0;
    tc::mbar_init(&misc->q_full, 1);
    tc::mbar_init(&misc->q_empty, 2);      // both S^T issuers
    tc::mbar_init(&misc->o_full, 2);       // both O^T issuers
    tc::mbar_init(&misc->o_empty, 256);
    for (int s = 0; s < kFwdKSlots; ++s) {
      tc::mbar_init(&misc->k_full[s], 2);    // the two producer warps of the ring
      tc::mbar_init(&misc->k_empty[s], 2);   // the issuing S^T warp (on completion) and the observing one
    }
    for (int s = 0; s < kFwdVSlots; ++s) {
      tc::mbar_init(&misc->v_full[s], 2);
      tc::mbar_init(&misc->v_empty[s], 1);
    }
    for (int s = 0; s < kFwdSBufs; ++s) {
      tc::mbar_init(&misc->s_full[s], 1);
      tc::mbar_init(&misc->s_free[s], 128);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->p_ready[s], 128);
      tc::mbar_init(&misc->p_free[s], 1);
    }
    tc::mbar_init(&misc->wg_sync[0], 128);
    tc::mbar_init(&misc->wg_sync[1], 128);
    tc::mbar_init(&misc->all_sync, 256);
    item_queue_init(&misc->items, 4 + 4 + 256);     // lane 0 of the producers, four issuers, the softmax threads
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
  // tensor-memory columns: S^T buffers 0, 64, 128, 192; O^T of the even tiles 256, of the odd tiles 320

  if (warp < 8) {
    tc::reg_dec<56>();
    if (warp < 2 || warp >= 6) {
      // ---------------------------------------------------------------- TMA producers
      // One warp sustains only ~24 B/clk of 5-D boxes (the copy instructions of a warp issue one after the other,
      // ~350 cycles per 8 KB box), so every ring has two producer warps: warps 0, 1 bring the first block of each
      // pair, warps 6, 7 the second.  Both arrive on the slot's full barrier with their half of the bytes.
      const int which = warp & 1;                           // 0: K ring (+ Q tile), 1: V ring
      const int my_blk = warp >> 2;                         // 0: first block of the pair, 1: second
      const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
      const uint32_t nslots = which == 0 ? kFwdKSlots : kFwdVSlots;
      uint64_t* full = which == 0 ? misc->k_full : misc->v_full;
      uint64_t* empty = which == 0 ? misc->k_empty : misc->v_empty;
      unsigned char* ring = smem + (which == 0 ? 0 : kFwdKSlots * C::SLOT);
      const int my_h = lane;
      const bool issuer = lane < C::DH;
      uint32_t tg = 0, n_items = 0, published = 0;
      for (uint32_t seq = 0;; ++seq) {
        // warp 0, lane 0 is the CTA's scheduler
        int item = 0;
        if (lane == 0) {
          if (warp == 0 && !item_publish_ahead(&misc->items, seq, published, a.item_counter, total_items, &misc->abort_flag)) item = -2;
          else item = item_get(&misc->items, seq, &misc->abort_flag);
        }
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item == -2) goto done;
        if (item < 0) break;
        const int i = item % g.N, bhq = item / g.N;
        const int b = bhq / g.Hq, hq = bhq % g.Hq, bhk = b * g.Hkv + hq / g.rep;
        const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
        const int k = end - beg;
        if (k == 0) continue;
        const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
        if (warp == 0) {
          int it_, ih_, iw_;
          cube_coords(g, i, it_, ih_, iw_);
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&misc->q_empty, (n_items & 1) ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&misc->q_full, C::QBYTES);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (lane < C::DH)
            tc::tma_load_5d(q_tile + lane * C::SLAB, &tm_q, &misc->q_full, lane * 64, iw_ * g.Bw, ih_ * g.Bh, it_ * g.Bt, bhq);
        }
        ++n_items;
        const int nt = (k + 1) >> 1;
        int j = cols[(my_blk == 1 && k > 1) ? 1 : 0];           // this lane's KV block of tile 0
        for (int t = 0; t < nt; ++t, ++tg) {
          int jt, jh, jw;
          cube_coords(g, j, jt, jh, jw);
          if (t + 1 < nt) j = cols[(my_blk == 1 && 2 * t + 3 < k) ? 2 * t + 3 : 2 * t + 2];   // next tile, fetched early
          const uint32_t slot = tg % nslots, par = (tg / nslots) & 1;
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&empty[slot], par ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&full[slot], C::SLOT / 2);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (issuer)
            tc::tma_load_5d(ring + slot * C::SLOT + (2 * my_h + my_blk) * C::SLAB, tm, &full[slot], my_h * 64,
                            jw * g.Bw, jh * g.Bh, jt * g.Bt, bhk);
        }
      }
    } else if (warp < 4) {
      // ---------------------------------------------------------------- issuers of S^T(t) = K_pair * Q^T
      if (lane == 0) {
        const uint32_t mine = warp - 2;            // parity of the tiles this warp issues
        const uint32_t q_addr = tc::smem_u32(q_tile), slot0 = tc::smem_u32(smem);
        uint32_t tg = 0, n_items = 0;
        for (uint32_t seq = 0;; ++seq) {
          VSA2_NEXT_ITEM(item, seq);
          const int i = item % g.N, bhq = item / g.N;
          const int k = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - a.row_ptr[(size_t)bhq * (g.N + 1) + i];
          if (k == 0) continue;
          const int nt = (k + 1) >> 1;
          VSA2_WAIT(&misc->q_full, n_items & 1);
          bool issued = false;
          for (int t = 0; t < nt; ++t, ++tg) {
            // Both issuers pass through every phase of the K ring (a slot alternates between them): the issuer that
            // does not own the tile only observes the load and adds its arrival to the slot's release.
            const uint32_t slot = tg % kFwdKSlots, buf = tg % kFwdSBufs;
            VSA2_WAIT(&misc->k_full[slot], (tg / kFwdKSlots) & 1);
            if ((tg & 1) != mine) {
              tc::mbar_arrive(&misc->k_empty[slot]);
              continue;
            }
            VSA2_WAIT(&misc->s_free[buf], ((tg / kFwdSBufs) & 1) ^ 1);
            tc::tc_fence_after();
            mma_pair_kmajor<D>(tmem_base + buf * 64, slot0 + slot * C::SLOT, q_addr);
            tc::mma_commit(&misc->s_full[buf]);
            tc::mma_commit(&misc->k_empty[slot]);
            issued = true;
          }
          // the Q tile may be replaced once both issuers are through with it
          if (issued) tc::mma_commit(&misc->q_empty);
          else tc::mbar_arrive(&misc->q_empty);
          ++n_items;
        }
      }
    } else if (warp < 6) {
      // ---------------------------------------------------------------- issuers of O^T += V_pair^T * P^T
      if (lane == 0) {
        const uint32_t mine = warp - 4;
        const uint32_t p_addr = tc::smem_u32(p_tile), slot0 = tc::smem_u32(smem);
        const uint32_t tm_o = tmem_base + 256 + mine * 64;
        uint32_t tg = 0, n_items = 0;
        for (uint32_t seq = 0;; ++seq) {
          VSA2_NEXT_ITEM(item, seq);
          const int i = item % g.N, bhq = item / g.N;
          const int k = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - a.row_ptr[(size_t)bhq * (g.N + 1) + i];
          if (k == 0) continue;
          const int nt = (k + 1) >> 1;
          VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);      // the previous query block's accumulators were read out
          bool issued = false;
          for (int t = 0; t < nt; ++t, ++tg) {
            if ((tg & 1) != mine) continue;
            const uint32_t slot = tg % kFwdVSlots;
            VSA2_WAIT(&misc->v_full[slot], (tg / kFwdVSlots) & 1);
            VSA2_WAIT(&misc->p_ready[mine], (tg >> 1) & 1);
            tc::tc_fence_after();
            mma_pairT_mnmajor<D>(tm_o, slot0 + (kFwdKSlots + slot) * C::SLOT, p_addr + mine * C::PBYTES, issued);
            tc::mma_commit(&misc->v_empty[slot]);
            tc::mma_commit(&misc->p_free[mine]);
            issued = true;
          }
          if (issued) tc::mma_commit(&misc->o_full);
          else tc::mbar_arrive(&misc->o_full);
          ++n_items;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (2 x 128 threads)
    tc::reg_inc<200>();
    const int wg = (warp >> 2) - 2;              // 0 or 1
    const int quad = warp & 3;
    const int row = (quad << 5) | lane;          // tensor-memory lane: key row in S^T, channel in O^T
    const int sm_tid = tid & 127;                // 0..127 inside this warpgroup
    const int sm_warp = warp - 8;                // 0..7 over both warpgroups
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && a.gate != nullptr;
    unsigned char* my_p = p_tile + wg * C::PBYTES;
    CubePos cpos;
    cpos.init(g, row & 63);
    const int blk = row >> 6;
    uint32_t tg = 0, n_items = 0, n_all = 0, wg_phase = 0, all_phase = 0;
    for (;; ++n_all) {
      VSA2_NEXT_ITEM(item, n_all);
      const int i = item % g.N, bhq = item / g.N;
      const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
      const int k = end - beg;
      const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
      const int tb = n_all & 1;
      if (wg == 0 && sm_tid < 64) {
        int it_, ih_, iw_;
        cube_coords(g, i, it_, ih_, iw_);
        const int l = cube_token(g, it_, ih_, iw_, sm_tid);
        misc->tok[tb][sm_tid] = l;
        misc->gate[tb][sm_tid] = (coarse && l >= 0) ? a.gate[(size_t)bhq * g.L + l] : 0.f;
      }
      const float oc_d = (coarse && row < D) ? a.oc_hat[((size_t)bhq * g.N + i) * D + row] : 0.f;
      if (wg == 0 && sm_tid == 0) misc->rescue_flag = 0;
      const int q0 = wg * 32;                    // this warpgroup writes query columns q0 .. q0 + 31 in the epilogue

      float l_part[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) l_part[c] = 0.f;
      const int nt = (k + 1) >> 1;
      const uint32_t tg0 = tg;
      if (k > 0) {
        const int first_wg = tg & 1;               // warpgroup that owns tile 0 of this query block
        if (wg == first_wg) {
          // reference exponent of every query column = exact column maximum of the first tile
          const uint32_t buf = tg % kFwdSBufs;
          const bool valid = !((blk == 1) && k < 2) && cpos.valid(edge[cols[(blk == 1 && k > 1) ? 1 : 0]], g);
          VSA2_WAIT(&misc->s_full[buf], (tg / kFwdSBufs) & 1);
          tc::tc_fence_after();
          uint32_t s0[32], s1[32];
          tc::tmem_ld32(lane_addr + buf * 64, s0);
          tc::tmem_ld32(lane_addr + buf * 64 + 32, s1);
          tc::tmem_ld_wait();
          float mx[64];
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            mx[c] = valid ? __uint_as_float(s0[c]) : -INFINITY;
            mx[c + 32] = valid ? __uint_as_float(s1[c]) : -INFINITY;
          }
          warp_reduce_cols64<true>(mx, lane);
          const int cb = warp_reduce_col(lane);
          misc->red[quad][cb] = mx[0];
          misc->red[quad][cb + 1] = mx[1];
          VSA2_GROUP_SYNC(&misc->wg_sync[wg], wg_phase);
          if (sm_tid < 64) {
            const float m4 = fmaxf(fmaxf(misc->red[0][sm_tid], misc->red[1][sm_tid]), fmaxf(misc->red[2][sm_tid], misc->red[3][sm_tid]));
            misc->m_ref[sm_tid] = (m4 > -INFINITY) ? m4 * c2 : 0.f;
          }
        }
      }
      VSA2_GROUP_SYNC(&misc->all_sync, all_phase);       // tables and reference exponents visible to both warpgroups

      if (k > 0) {
        // first own tile of this query block and the KV block of this thread's key row in it
        int t_own = ((tg & 1) == (uint32_t)wg) ? 0 : 1;
        int j_next = 0;
        if (t_own < nt) j_next = cols[(blk == 1 && 2 * t_own + 1 < k) ? 2 * t_own + 1 : 2 * t_own];
        for (int t = t_own; t < nt; t += 2) {
          const uint32_t tgt = tg0 + t, buf = tgt % kFwdSBufs;
          const bool dup = (blk == 1) && (2 * t + 1 >= k);
          const bool valid = !dup && cpos.valid(edge[j_next], g);
          if (t + 2 < nt) j_next = cols[(blk == 1 && 2 * t + 5 < k) ? 2 * t + 5 : 2 * t + 4];   // next own tile, fetched early
          const bool all_valid = __all_sync(0xffffffffu, valid);
          VSA2_WAIT(&misc->s_full[buf], (tgt / kFwdSBufs) & 1);
          tc::tc_fence_after();
          uint32_t sa[32], sb[32];
          tc::tmem_ld32(lane_addr + buf * 64, sa);
          tc::tmem_ld32(lane_addr + buf * 64 + 32, sb);
          tc::tmem_ld_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->s_free[buf]);
          uint32_t packed[32];
          const float4* mref4 = reinterpret_cast<const float4*>(misc->m_ref);
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
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            const float4 m = mref4[8 + c4];
            float p0 = ex2_approx(fmaf(__uint_as_float(sb[4 * c4 + 0]), c2, -m.x));
            float p1 = ex2_approx(fmaf(__uint_as_float(sb[4 * c4 + 1]), c2, -m.y));
            float p2 = ex2_approx(fmaf(__uint_as_float(sb[4 * c4 + 2]), c2, -m.z));
            float p3 = ex2_approx(fmaf(__uint_as_float(sb[4 * c4 + 3]), c2, -m.w));
            if (!all_valid) { p0 = valid ? p0 : 0.f; p1 = valid ? p1 : 0.f; p2 = valid ? p2 : 0.f; p3 = valid ? p3 : 0.f; }
            l_part[32 + 4 * c4 + 0] += p0;
            l_part[32 + 4 * c4 + 1] += p1;
            l_part[32 + 4 * c4 + 2] += p2;
            l_part[32 + 4 * c4 + 3] += p3;
            packed[16 + 2 * c4] = pack_bf16x2(p0, p1);
            packed[16 + 2 * c4 + 1] = pack_bf16x2(p2, p3);
          }
          VSA2_WAIT(&misc->p_free[wg], ((tgt >> 1) & 1) ^ 1);
          store_row_sw128(my_p, row, packed);
          tc::fence_proxy_async_smem();
          tc::mbar_arrive(&misc->p_ready[wg]);
        }
        tg += nt;

        // ---- epilogue of the query block (both warpgroups): row sums over all 256 key rows x tiles
        warp_reduce_cols64<false>(l_part, lane);
        {
          const int cb = warp_reduce_col(lane);
          misc->red[sm_warp][cb] = l_part[0];
          misc->red[sm_warp][cb + 1] = l_part[1];
        }
        VSA2_GROUP_SYNC(&misc->all_sync, all_phase);
        if (wg == 0 && sm_tid < 64) {
          float l = 0.f;
#pragma unroll
          for (int w = 0; w < 8; ++w) l += misc->red[w][sm_tid];
          // sums outside the safe range (overflow, NaN or total underflow): hand the block to the exact kernel
          if (!(l > 1e-30f && l < 1e30f)) misc->rescue_flag = 1;
          misc->l_inv[sm_tid] = 1.f / l;
          const int tk = misc->tok[tb][sm_tid];
          if (tk >= 0) a.lse[(size_t)bhq * g.L + tk] = (misc->m_ref[sm_tid] + __log2f(l)) * 0.6931471805599453f;
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
        VSA2_GROUP_SYNC(&misc->all_sync, all_phase);
      }

      // O[l, d] = (O_even^T + O_odd^T)[d, q] / l[q] + gate[q] * O_c[d]; this warpgroup owns 32 query columns
      {
        float acc[32];
        if (k > 0) {
          uint32_t o0[32];
          tc::tmem_ld32(lane_addr + 256 + (tg0 & 1) * 64 + q0, o0);       // accumulator of the parity that saw tile 0
          tc::tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) acc[c] = __uint_as_float(o0[c]);
          if (nt > 1) {
            tc::tmem_ld32(lane_addr + 256 + ((tg0 & 1) ^ 1) * 64 + q0, o0);
            tc::tmem_ld_wait();
#pragma unroll
            for (int c = 0; c < 32; ++c) acc[c] += __uint_as_float(o0[c]);
          }
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) acc[c] = 0.f;
        }
        if (g.out_f32 || a.o_res == nullptr) {
          // plain stores (validation paths): one element per thread and query
          if (row < D) {
#pragma unroll
            for (int qq = 0; qq < 32; ++qq) {
              const int qi = q0 + qq;
              const int l = misc->tok[tb][qi];
              if (l < 0) continue;
              const float val = fmaf(misc->gate[tb][qi], oc_d, k > 0 ? acc[qq] * misc->l_inv[qi] : 0.f);
              const size_t idx = ((size_t)bhq * g.L + l) * D + row;
              store_out(a.o, idx, val, g.out_f32);
              if (a.o_res != nullptr) a.o_res[idx] = __float2bfloat16_rn(val - __bfloat162float(__float2bfloat16_rn(val)));
            }
          }
        } else {
          // bf16 output and residual: transpose through shared memory (the P^T buffers are idle now), then 16-byte stores
          bf16* st_o = reinterpret_cast<bf16*>(p_tile);                 // [64 q][D]
          bf16* st_r = reinterpret_cast<bf16*>(p_tile + C::PBYTES);     // [64 q][D]
          if (row < D) {
#pragma unroll
            for (int qq = 0; qq < 32; ++qq) {
              const int qi = q0 + qq;
              const float val = fmaf(misc->gate[tb][qi], oc_d, k > 0 ? acc[qq] * misc->l_inv[qi] : 0.f);
              const bf16 vb = __float2bfloat16_rn(val);
              st_o[qi * D + row] = vb;
              st_r[qi * D + row] = __float2bfloat16_rn(val - __bfloat162float(vb));
            }
          }
          VSA2_GROUP_SYNC(&misc->all_sync, all_phase);
          constexpr int CH = D / 8;                                      // 16-byte chunks per token row
          const int t256 = tid - 256;
          for (int e = t256; e < 64 * CH; e += 256) {
            const int qi = e / CH, ch = e % CH;
            const int l = misc->tok[tb][qi];
            if (l < 0) continue;
            const size_t idx = ((size_t)bhq * g.L + l) * D + ch * 8;
            *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.o) + idx) = *reinterpret_cast<const uint4*>(st_o + qi * D + ch * 8);
            *reinterpret_cast<uint4*>(a.o_res + idx) = *reinterpret_cast<const uint4*>(st_r + qi * D + ch * 8);
          }
          VSA2_GROUP_SYNC(&misc->all_sync, all_phase);        // staging buffers free before the next query block writes P^T
        }
      }
      if (k == 0 && wg == 0 && sm_tid < 64 && misc->tok[tb][sm_tid] >= 0)
        a.lse[(size_t)bhq * g.L + misc->tok[tb][sm_tid]] = -INFINITY;
      if (k > 0 && wg == 0 && sm_tid == 0 && misc->rescue_flag) {
        int slot = atomicAdd(a.rescue_count, 1);
        if (slot < a.rescue_cap) a.rescue_items[slot] = block_item(g, bhq, i);   // the list kernel's item numbering
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

size_t fine_fwd_tc_workspace_bytes() { return 256 + (size_t)kRescueCap * sizeof(int); }

// Entries of the rescue list the kernels may use (<= kRescueCap, which sizes the workspace).  Process-wide; lowered only by
// tests that make the list overflow on a small problem.
static int g_rescue_cap = kRescueCap;
int fwd_rescue_capacity() { return g_rescue_cap; }
void set_fwd_rescue_capacity(int cap) { g_rescue_cap = cap < 1 ? 1 : (cap > kRescueCap ? kRescueCap : cap); }

// workspace: [StatusBlock][rescue list]; the rescue counter is StatusBlock.pad[0].
cudaError_t launch_fine_fwd_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                               const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                               float* lse, StatusBlock* status, cudaStream_t st) {
  CUtensorMap tq, tk, tv;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  FwdArgs a;
  a.gate = gate; a.row_ptr = row_ptr; a.col_idx = col_idx; a.oc_hat = oc_hat; a.o = o; a.o_res = o_res; a.lse = lse;
  a.status = status;
  a.rescue_count = &status->pad[0];
  a.item_counter = &status->pad[1];
  a.rescue_items = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(status) + 256);
  a.rescue_cap = g_rescue_cap;
  const int total = g.batch * g.Hq * g.N;
  const int grid = total < sms ? total : sms;
  if (g.N > kFwdMaxCubes) return cudaErrorInvalidValue;
  // The softmax warpgroups raise their register count to 200 with the registers the service warpgroups give up
  // (setmaxnreg); that request would block for ever if the launch allocation were smaller than 128 per thread.
  {
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, g.D == 128 ? (const void*)fine_fwd_tc_kernel<128> : (const void*)fine_fwd_tc_kernel<64>)) != cudaSuccess) return e;
    if (fa.numRegs * kFwdThreads < 256 * 56 + 256 * 200) return cudaErrorLaunchOutOfResources;
  }
  if (g.D == 128) {
    const size_t smb = FwdTc<128>::smem_bytes(g.N);
    if ((e = cudaFuncSetAttribute(fine_fwd_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_tc_kernel<128><<<grid, kFwdThreads, smb, st>>>(tq, tk, tv, g, a);
  } else {
    const size_t smb = FwdTc<64>::smem_bytes(g.N);
    if ((e = cudaFuncSetAttribute(fine_fwd_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_tc_kernel<64><<<grid, kFwdThreads, smb, st>>>(tq, tk, tv, g, a);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // query blocks whose row sums left the safe range are redone with the exact running maximum
  return launch_fine_fwd_list(g, a.rescue_count, a.rescue_cap, a.rescue_items, q, k, v, gate, row_ptr, col_idx, oc_hat, o, o_res, lse, st);
}

}  // namespace vsa2
