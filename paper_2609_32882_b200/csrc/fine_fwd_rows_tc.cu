// Fine branch forward (paper Eq. 12) + gated merge (Eq. 14) on the Blackwell tensor cores, queries in the lanes.
//
// Formulation.  A query block has B = 64 tokens.  Both products keep the 64 queries in the rows of the accumulator (M = 64)
// and stack two selected KV blocks per tile:
//     S [64 q, 128 kv] = Q [64, D] * K_pair^T            (A = Q from shared memory,  B = K_pair, N = 128 keys)
//     O [64 q, D]     += P [64, 128 kv] * V_pair         (A = P from TENSOR MEMORY,  B = V_pair, N = D)
// M = 64 runs the tensor pipe at half rate, but every K / V tile is fetched from shared memory exactly once per tile and P
// never touches shared memory: per tile 64 KB of TMA writes + 64 KB of B fetches + 16 KB of Q, against 176 KB for the
// transposed M = 128, N = 64 products, which were bound by that traffic.  K and V tiles arrive by 5-D TMA straight from the
// raster tensors (one box = one cube, zero-filled outside the grid); the V tile that TMA wrote row-per-key is read as an
// MN-major B operand, so nothing is transposed in memory.
//
// Tensor memory (512 columns): two S buffers (2 x 128 fp32 columns), two P buffers (2 x 64 columns of bf16 pairs) and the O
// accumulator (D columns).  An M = 64 accumulator keeps row m in lane (m % 16) + 32 (m / 16); the softmax warps read S with
// 16-lane loads that give a thread two query rows x 32 key columns, and the bf16 pairs it forms from neighbouring columns
// are exactly the words its 16-lane store writes into the P operand.
//
// Softmax.  Four threads share a query row.  Each row keeps a fixed reference M (the exact row maximum of the block's first
// tile, log2 units): P = 2^(s*scale*log2e - M); any reference gives the same softmax unless something overflows, the row
// sums are checked at the end of the query block and a block outside the safe range is redone by the exact-maximum kernel
// (fine_fwd.cu).  Two sums are kept per row: the fp32 sum of the exponentials, which gives the log-sum-exp, and the sum of
// their bf16 roundings, which is what the P V product really adds up -- the output is normalised by the latter, so the
// weights sum to one and the rounding of a dominant P cancels instead of scaling the whole output row (that scaling,
// 2^-9 relative, reached the backward through delta = rowsum(dO * O) and was its largest error on sharply peaked rows).
//
// Roles (512 threads): warps 0..3 = TMA producers (K / V ring x first / second block of a pair; warp 0 also brings the Q
// tile and schedules the CTA's work items), warp 4 = issuer of S, warp 5 = issuer of O, warps 8..15 = two softmax +
// epilogue warpgroups that alternate tiles.  Persistent CTAs draw query blocks from a global counter.  Every wait is bounded.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kFrThreads = 512;
constexpr int kFrKSlots = 3;
constexpr int kFrVSlots = 3;
constexpr int kFrMaxCubes = 8192;      // edge-flag table in shared memory: one byte per cube

template <int D>
struct FwdRows {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLOT = 2 * DH * kSlab;     // a K pair or a V pair, [half][A | B]
  static constexpr uint32_t QBYTES = DH * kSlab;
  static constexpr int NQ = 1;                                            // Q tiles (by item parity if 2)
  static constexpr uint32_t OFF_Q = (kFrKSlots + kFrVSlots) * SLOT;
  static constexpr uint32_t OFF_MISC = OFF_Q + NQ * QBYTES;
  static constexpr uint32_t MISC_BYTES = 4096;
  static constexpr uint32_t TM_S = 0, TM_P = 256, TM_O = 384;
  static size_t smem_bytes(int n_cubes) { return OFF_MISC + MISC_BYTES + ((size_t)n_cubes + 15) / 16 * 16 + 1024; }
};

struct FwdRowsMisc {
  uint64_t q_full[2], q_empty[2], o_full, o_empty;
  uint64_t tab_full[2], tab_free[2];   // per-item tables (tok, gate, oc) of the item with that parity
  uint64_t k_full[kFrKSlots], k_empty[kFrKSlots];
  uint64_t v_full[kFrVSlots], v_empty[kFrVSlots];
  uint64_t s_full[2], s_free[2];
  uint64_t p_ready[2], p_free[2];
  ItemQueue items;
  uint64_t all_sync;               // group barrier of the 256 softmax threads
  uint32_t tmem_base;
  int abort_flag;
  int rescue_flag;
  unsigned short vmask[17][4];     // [table row of the block][lane % 4]: which of a thread's 16 key columns are valid tokens
  alignas(16) float m_ref[64];     // per query row: reference exponent (log2 units)
  float red[2][2][64];             // [warpgroup][exact sum | sum of the bf16 roundings][query row]
  alignas(16) float oc[2][128];    // coarse output row of the query cube, by item parity
  int tok[2][64];                  // raster token of each query row (-1 = padding), by item parity
  float gate[2][64];
  int list_k[2], list_beg[2];      // length and start of the item's list of KV blocks
  int list_head[2][4];             // its first four entries (tiles 0 and 1)
};
static_assert(sizeof(FwdRowsMisc) <= 4096, "misc region too small");

struct FwdRowsArgs {
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
  int rescue_cap;
};

// 4 x 4 transpose of 32-bit words among the four lanes of a quad (cq = lane % 4): in, lane c holds x[n] = word c of chunk n;
// out, lane c holds the four words of chunk c in order.  Two rounds of exchanges (lane distance 1, then 2).
__device__ __forceinline__ void quad_transpose4(uint32_t (&x)[4], int cq) {
  const bool b0 = cq & 1, b1 = cq & 2;
  {
    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, b0 ? x[0] : x[1], 1), r1 = __shfl_xor_sync(0xffffffffu, b0 ? x[2] : x[3], 1);
    if (b0) { x[0] = r0; x[2] = r1; } else { x[1] = r0; x[3] = r1; }
  }
  {
    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, b1 ? x[0] : x[2], 2), r1 = __shfl_xor_sync(0xffffffffu, b1 ? x[1] : x[3], 2);
    if (b1) { x[0] = r0; x[1] = r1; } else { x[2] = r0; x[3] = r1; }
  }
}

template <int D>
__global__ void __launch_bounds__(kFrThreads, 1)
fine_fwd_rows_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_qt,
                        const __grid_constant__ CUtensorMap tm_kt, const __grid_constant__ CUtensorMap tm_vt, Geo g,
                        FwdRowsArgs a) {
  using C = FwdRows<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* q_tile = smem + C::OFF_Q;
  FwdRowsMisc* misc = reinterpret_cast<FwdRowsMisc*>(smem + C::OFF_MISC);
  unsigned char* edge = smem + C::OFF_MISC + C::MISC_BYTES;      // edge flags of every cube

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hq * g.N;
  const float c2 = g.scale * 1.4426950408889634f;

  // per block: the row of the validity table below -- the edge flags of a video cube (0 = nothing cut), 0 for a full text
  // block, 16 for the ragged last text block
  for (int n = tid; n < g.N; n += blockDim.x)
    edge[n] = (unsigned char)(n < g.Nvid ? cube_edge_flags(g, n) : (block_count(g, n) == kBlockTokens ? 0 : 16));
  if (tid < 68) {
    // validity of key columns 8n + 2c + e (n = 0..7, e = 0, 1) of a 64-token block, for lane % 4 == c: rows 0..15 by the
    // edge flags of a video cube, row 16 for the last text block when it holds fewer than 64 tokens
    const unsigned f = tid >> 2, c = tid & 3;
    const int text_tail = g.Lt % kBlockTokens;
    unsigned m = 0;
    for (int n = 0; n < 8; ++n)
      for (int e = 0; e < 2; ++e) {
        const int pos = 8 * n + 2 * (int)c + e;
        CubePos cp;
        cp.init(g, pos);
        if (f < 16 ? cp.valid(f, g) : pos < text_tail) m |= 1u << (2 * n + e);
      }
    misc->vmask[f][c] = (unsigned short)m;
  }
  if (tid == 0) {
    misc->abort_flag = 0;
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->q_full[s], 1);
      tc::mbar_init(&misc->q_empty[s], 1);
      tc::mbar_init(&misc->tab_full[s], 32);
      tc::mbar_init(&misc->tab_free[s], 256);
    }
    tc::mbar_init(&misc->o_full, 1);
    tc::mbar_init(&misc->o_empty, 256);
    for (int s = 0; s < kFrKSlots; ++s) {
      tc::mbar_init(&misc->k_full[s], 2);    // the two producer warps of the ring
      tc::mbar_init(&misc->k_empty[s], 1);
    }
    for (int s = 0; s < kFrVSlots; ++s) {
      tc::mbar_init(&misc->v_full[s], 2);
      tc::mbar_init(&misc->v_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->s_full[s], 1);
      tc::mbar_init(&misc->s_free[s], 128);
      tc::mbar_init(&misc->p_ready[s], 128);
      tc::mbar_init(&misc->p_free[s], 1);
    }
    tc::mbar_init(&misc->all_sync, 256);
    item_queue_init(&misc->items, 4 + 2 + 1 + 256); // lane 0 of the producers, of the two issuers and of the table loader, the softmax threads
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
    if (g.Lt > 0) {
      tc::prefetch_tmap(&tm_qt);
      tc::prefetch_tmap(&tm_kt);
      tc::prefetch_tmap(&tm_vt);
    }
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
      // One warp sustains only ~24 B/clk of 5-D boxes (the copy instructions of a warp issue one after the other), so every
      // ring has two producer warps, one per block of a pair; both arrive on the slot's full barrier with half the bytes.
      const int which = warp & 1;                           // 0: K ring (+ Q tile), 1: V ring
      const int my_blk = warp >> 1;                         // 0: first block of the pair, 1: second
      const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
      const CUtensorMap* tm_text = which == 0 ? &tm_kt : &tm_vt;
      const uint32_t nslots = which == 0 ? kFrKSlots : kFrVSlots;
      uint64_t* full = which == 0 ? misc->k_full : misc->v_full;
      uint64_t* empty = which == 0 ? misc->k_empty : misc->v_empty;
      unsigned char* ring = smem + (which == 0 ? 0 : kFrKSlots * C::SLOT);
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
        int i, bhq;
        item_block(g, item, bhq, i);
        const int b = bhq / g.Hq, hq = bhq % g.Hq, bhk = b * g.Hkv + hq / g.rep;
        const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
        const int k = end - beg;
        if (k == 0) continue;
        const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + beg;
        if (warp == 0) {
          int c1, c2, c3;
          block_box(g, i, c1, c2, c3);
          int ok = 1;
          const uint32_t qb = n_items % C::NQ;
          if (lane == 0) {
            ok = tc::mbar_wait(&misc->q_empty[qb], ((n_items / C::NQ) & 1) ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&misc->q_full[qb], C::QBYTES);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (lane < C::DH)
            tc::tma_load_5d(q_tile + qb * C::QBYTES + lane * kSlab, block_is_text(g, i) ? &tm_qt : &tm_q, &misc->q_full[qb],
                            lane * 64, c1, c2, c3, bhq);
        }
        ++n_items;
        const int nt = (k + 1) >> 1;
        int j = cols[(my_blk == 1 && k > 1) ? 1 : 0];           // this warp's KV block of tile 0
        for (int t = 0; t < nt; ++t, ++tg) {
          int c1, c2, c3;
          block_box(g, j, c1, c2, c3);
          const CUtensorMap* tm_j = block_is_text(g, j) ? tm_text : tm;
          if (t + 1 < nt) j = cols[(my_blk == 1 && 2 * t + 3 < k) ? 2 * t + 3 : 2 * t + 2];   // next tile, fetched early
          const uint32_t slot = tg % nslots, par = (tg / nslots) & 1;
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait(&empty[slot], par ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&full[slot], C::SLOT / 2);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (issuer)
            tc::tma_load_5d(ring + slot * C::SLOT + (2 * my_h + my_blk) * kSlab, tm_j, &full[slot], my_h * 64, c1, c2, c3, bhk);
        }
      }
    } else if (warp == 4) {
      // ---------------------------------------------------------------- issuer of S(t) = Q * K_pair^T
      // The whole warp runs the loop and one elected lane issues: with the warp converged the compiler keeps the
      // descriptors in uniform registers, and a tcgen05.mma then issues every ~74 cycles instead of ~117 from a lone lane.
      constexpr uint32_t idesc = tc::idesc_bf16(64, 128, false, false);
      const uint32_t slot0 = tc::smem_u32(smem);
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        int item = 0;
        if (lane == 0) item = item_get(&misc->items, seq, &misc->abort_flag);
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item == -2) goto done;
        if (item < 0) break;
        int i, bhq;
        item_block(g, item, bhq, i);
        const int k = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - a.row_ptr[(size_t)bhq * (g.N + 1) + i];
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        const uint32_t qb = n_items % C::NQ;
        const uint64_t dq = tc::smem_desc_sw128(tc::smem_u32(q_tile) + qb * C::QBYTES, 16, 1024);
        VSA2_WAIT(&misc->q_full[qb], (n_items / C::NQ) & 1);
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t slot = tg % kFrKSlots, buf = tg & 1;
          VSA2_WAIT(&misc->k_full[slot], (tg / kFrKSlots) & 1);
          VSA2_WAIT(&misc->s_free[buf], ((tg >> 1) & 1) ^ 1);
          tc::tc_fence_after();
          if (tc::elect_one()) {
            const uint64_t dk = tc::smem_desc_sw128(slot0 + slot * C::SLOT, 16, 1024);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint64_t oa = (uint64_t)(((ks / 4) * kSlab + (ks % 4) * 32) >> 4);
              const uint64_t ob = (uint64_t)(((ks / 4) * 2 * kSlab + (ks % 4) * 32) >> 4);
              tc::mma_ss(tmem_base + C::TM_S + buf * 128, dq + oa, dk + ob, idesc, ks > 0);
            }
            tc::mma_commit(&misc->s_full[buf]);
            tc::mma_commit(&misc->k_empty[slot]);
            if (t == nt - 1) tc::mma_commit(&misc->q_empty[qb]);   // the Q tile may be replaced once the last S of the block is done
          }
          __syncwarp();
        }
        ++n_items;
      }
    } else if (warp == 5) {
      // ---------------------------------------------------------------- issuer of O += P(t) * V_pair
      constexpr uint32_t idesc = tc::idesc_bf16(64, D, false, true);
      constexpr uint32_t lbo = (D == 128) ? 2 * kSlab : 0;       // distance between the two 64-channel halves of V
      const uint32_t slot0 = tc::smem_u32(smem) + kFrKSlots * C::SLOT;
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        int item = 0;
        if (lane == 0) item = item_get(&misc->items, seq, &misc->abort_flag);
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item == -2) goto done;
        if (item < 0) break;
        int i, bhq;
        item_block(g, item, bhq, i);
        const int k = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - a.row_ptr[(size_t)bhq * (g.N + 1) + i];
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);      // the previous query block's accumulator was read out
        for (int t = 0; t < nt; ++t, ++tg) {
          const uint32_t slot = tg % kFrVSlots, buf = tg & 1;
          VSA2_WAIT(&misc->v_full[slot], (tg / kFrVSlots) & 1);
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
      // ---------------------------------------------------------------- per-item tables, one item ahead of the softmax warps:
      // raster token and gate of every query row, coarse output row of the cube (global loads kept off their critical path)
      const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && a.gate != nullptr;
      for (uint32_t seq = 0;; ++seq) {
        int item = 0;
        if (lane == 0) item = item_get(&misc->items, seq, &misc->abort_flag);
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item == -2) goto done;
        if (item < 0) break;
        int i, bhq;
        item_block(g, item, bhq, i);
        const uint32_t tb = seq & 1;
        const bool video = !block_is_text(g, i);      // text queries take no part in the coarse branch or the gate
        const int beg_ = a.row_ptr[(size_t)bhq * (g.N + 1) + i], k_ = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1] - beg_;
        const int head_ = (lane < 4 && lane < k_) ? a.col_idx[(size_t)bhq * g.nnz_cap + beg_ + lane] : 0;
        int l2[2];
        float g2[2], oc4[4];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          l2[r] = block_token(g, i, lane + 32 * r);
          g2[r] = (coarse && video && l2[r] >= 0) ? a.gate[(size_t)bhq * g.L + l2[r]] : 0.f;
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
          oc4[r] = (coarse && video && lane + 32 * r < D) ? a.oc_hat[((size_t)bhq * g.Nvid + i) * D + lane + 32 * r] : 0.f;
        VSA2_WAIT_PARKED(&misc->tab_free[tb], ((seq >> 1) & 1) ^ 1);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          misc->tok[tb][lane + 32 * r] = l2[r];
          misc->gate[tb][lane + 32 * r] = g2[r];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) misc->oc[tb][lane + 32 * r] = oc4[r];
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
    const int cq = lane & 3;
    const int row_a = quad * 16 + (lane >> 2), row_b = row_a + 8;     // the two query rows of this thread
    const int sm_tid = tid & 127;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    constexpr int COLS = D / 2;                  // output columns per warpgroup in the epilogue
    uint32_t tg = 0, n_items = 0, all_phase = 0;
    for (uint32_t n_all = 0;; ++n_all) {
      VSA2_NEXT_ITEM(item, n_all);
      int i, bhq;
      item_block(g, item, bhq, i);
      const int tb = n_all & 1;
      VSA2_WAIT(&misc->tab_full[tb], (n_all >> 1) & 1);  // the item's tables (loaded one item ahead by warp 6)
      const int k = misc->list_k[tb];
      const int* cols = a.col_idx + (size_t)bhq * g.nnz_cap + misc->list_beg[tb];
      const int* head = misc->list_head[tb];
      (void)i;
      if (wg == 0 && sm_tid == 0) misc->rescue_flag = 0;

      const int nt = (k + 1) >> 1;
      const uint32_t tg0 = tg;
      uint32_t sv[64];
      bool have_first = false;
      if (k > 0 && (tg & 1) == (uint32_t)wg) {
        // this warpgroup owns tile 0: reference exponent of every query row = exact row maximum of that tile
        const uint32_t buf = tg & 1;
        VSA2_WAIT(&misc->s_full[buf], (tg >> 1) & 1);
        tc::tc_fence_after();
        tc::tmem_ld_16x256b_x16(lane_addr + C::TM_S + buf * 128, sv);
        tc::tmem_ld_wait();
        tc::tc_fence_before();
        tc::mbar_arrive(&misc->s_free[buf]);
        have_first = true;
        const unsigned ma = misc->vmask[edge[head[0]]][cq];
        const unsigned mb = k > 1 ? misc->vmask[edge[head[1]]][cq] : 0u;
        float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
        for (int n = 0; n < 16; ++n) {
          const unsigned m = (n < 8 ? ma : mb) >> (2 * (n & 7));
          if (m & 1u) { mx_a = fmaxf(mx_a, __uint_as_float(sv[4 * n])); mx_b = fmaxf(mx_b, __uint_as_float(sv[4 * n + 2])); }
          if (m & 2u) { mx_a = fmaxf(mx_a, __uint_as_float(sv[4 * n + 1])); mx_b = fmaxf(mx_b, __uint_as_float(sv[4 * n + 3])); }
        }
        mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
        mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
        if (cq == 0) {
          misc->m_ref[row_a] = (mx_a > -INFINITY) ? mx_a * c2 : 0.f;
          misc->m_ref[row_b] = (mx_b > -INFINITY) ? mx_b * c2 : 0.f;
        }
      }
      VSA2_GROUP_SYNC(&misc->all_sync, all_phase);       // reference exponents visible to both warpgroups

      float l_a = 0.f, l_b = 0.f, r_a = 0.f, r_b = 0.f;   // exact sums and sums of the bf16 roundings of the two rows
      float m_a = 0.f, m_b = 0.f;
      if (k > 0) {
        m_a = misc->m_ref[row_a];
        m_b = misc->m_ref[row_b];
        const int t_first = ((tg0 & 1) == (uint32_t)wg) ? 0 : 1;
        // KV blocks of this warpgroup's tiles: the first from the item's table, the others fetched one own tile ahead
        int ja = head[2 * t_first < k ? 2 * t_first : 0], jb = head[2 * t_first + 1 < k ? 2 * t_first + 1 : 0];
        for (int t = t_first; t < nt; t += 2) {
          const uint32_t tgt = tg0 + t, buf = tgt & 1;
          const bool dup = 2 * t + 1 >= k;
          const unsigned ma = misc->vmask[edge[ja]][cq];
          const unsigned mb = dup ? 0u : misc->vmask[edge[jb]][cq];
          if (t + 2 < nt) {
            ja = cols[2 * t + 4];
            jb = cols[2 * t + 5 < k ? 2 * t + 5 : 2 * t + 4];
          }
          if (!(have_first && t == 0)) {
            VSA2_WAIT(&misc->s_full[buf], (tgt >> 1) & 1);
            tc::tc_fence_after();
            tc::tmem_ld_16x256b_x16(lane_addr + C::TM_S + buf * 128, sv);
            tc::tmem_ld_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&misc->s_free[buf]);
          }
          uint32_t pk[32];
          if ((ma & mb) == 0xffffu) {
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 0]), c2, -m_a));
              const float p1 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 1]), c2, -m_a));
              const float p2 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 2]), c2, -m_b));
              const float p3 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 3]), c2, -m_b));
              l_a += p0 + p1;
              l_b += p2 + p3;
              const uint32_t wa = pack_bf16x2(p0, p1), wb = pack_bf16x2(p2, p3);
              r_a += __uint_as_float(wa << 16) + __uint_as_float(wa & 0xffff0000u);
              r_b += __uint_as_float(wb << 16) + __uint_as_float(wb & 0xffff0000u);
              pk[2 * n] = wa;
              pk[2 * n + 1] = wb;
            }
          } else {
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              const unsigned m = (n < 8 ? ma : mb) >> (2 * (n & 7));
              float p0 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 0]), c2, -m_a));
              float p1 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 1]), c2, -m_a));
              float p2 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 2]), c2, -m_b));
              float p3 = ex2_approx(fmaf(__uint_as_float(sv[4 * n + 3]), c2, -m_b));
              if (!(m & 1u)) { p0 = 0.f; p2 = 0.f; }
              if (!(m & 2u)) { p1 = 0.f; p3 = 0.f; }
              l_a += p0 + p1;
              l_b += p2 + p3;
              const uint32_t wa = pack_bf16x2(p0, p1), wb = pack_bf16x2(p2, p3);
              r_a += __uint_as_float(wa << 16) + __uint_as_float(wa & 0xffff0000u);
              r_b += __uint_as_float(wb << 16) + __uint_as_float(wb & 0xffff0000u);
              pk[2 * n] = wa;
              pk[2 * n + 1] = wb;
            }
          }
          VSA2_WAIT(&misc->p_free[buf], ((tgt >> 1) & 1) ^ 1);
          tc::tmem_st_16x128b_x16(lane_addr + C::TM_P + buf * 64, pk);
          tc::tmem_st_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->p_ready[buf]);
        }
        tg += nt;
        // row sums: over the four threads of a row here, over the two warpgroups through shared memory
        l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
        l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
        r_a += __shfl_xor_sync(0xffffffffu, r_a, 1);
        r_b += __shfl_xor_sync(0xffffffffu, r_b, 1);
        l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
        l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
        r_a += __shfl_xor_sync(0xffffffffu, r_a, 2);
        r_b += __shfl_xor_sync(0xffffffffu, r_b, 2);
        if (cq == 0) {
          misc->red[wg][0][row_a] = l_a;
          misc->red[wg][0][row_b] = l_b;
          misc->red[wg][1][row_a] = r_a;
          misc->red[wg][1][row_b] = r_b;
        }
      }
      VSA2_GROUP_SYNC(&misc->all_sync, all_phase);
      float inv_a = 0.f, inv_b = 0.f;
      if (k > 0) {
        const float la = misc->red[0][0][row_a] + misc->red[1][0][row_a], lb = misc->red[0][0][row_b] + misc->red[1][0][row_b];
        const float ra = misc->red[0][1][row_a] + misc->red[1][1][row_a], rb = misc->red[0][1][row_b] + misc->red[1][1][row_b];
        inv_a = 1.f / ra;
        inv_b = 1.f / rb;
        if (wg == 0 && cq == 0) {
          // sums outside the safe range (overflow, NaN or total underflow): hand the block to the exact kernel
          if (!(la > 1e-30f && la < 1e30f && ra > 1e-30f) || !(lb > 1e-30f && lb < 1e30f && rb > 1e-30f)) misc->rescue_flag = 1;
          const int ta = misc->tok[tb][row_a], tk_b = misc->tok[tb][row_b];
          if (ta >= 0) a.lse[(size_t)bhq * g.S + ta] = (m_a + __log2f(la)) * 0.6931471805599453f;
          if (tk_b >= 0) a.lse[(size_t)bhq * g.S + tk_b] = (m_b + __log2f(lb)) * 0.6931471805599453f;
        }
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
      } else if (wg == 0 && cq == 0) {
        const int ta = misc->tok[tb][row_a], tk_b = misc->tok[tb][row_b];
        if (ta >= 0) a.lse[(size_t)bhq * g.S + ta] = -INFINITY;
        if (tk_b >= 0) a.lse[(size_t)bhq * g.S + tk_b] = -INFINITY;
      }

      // O[l, d] = O_acc[q, d] / (rounded row sum) + gate[q] * O_c[d]; this warpgroup owns COLS output columns
      {
        // The accumulator is read in slices of 32 columns inside a rolled loop: what runs once per query block is fetched
        // from the instruction cache once per query block (the tile loop has evicted it by then).
        const float ga = misc->gate[tb][row_a], gb = misc->gate[tb][row_b];
        const int ta = misc->tok[tb][row_a], tk_b = misc->tok[tb][row_b];
        bf16* ob = reinterpret_cast<bf16*>(a.o);
        const size_t base_a = ((size_t)bhq * g.S + (ta >= 0 ? ta : 0)) * D + wg * COLS, base_b = ((size_t)bhq * g.S + (tk_b >= 0 ? tk_b : 0)) * D + wg * COLS;
#pragma unroll 1
        for (int n0 = 0; n0 < COLS / 8; n0 += 4) {
          uint32_t acc[16];
          if (k > 0) {
            tc::tmem_ld_16x256b_x4(lane_addr + C::TM_O + wg * COLS + 8 * n0, acc);
            tc::tmem_ld_wait();
            if (n0 + 4 >= COLS / 8) {
              tc::tc_fence_before();
              tc::mbar_arrive(&misc->o_empty);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 16; ++c) acc[c] = 0u;
          }
          float v[16];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float2 oc2 = *reinterpret_cast<const float2*>(&misc->oc[tb][wg * COLS + 8 * (n0 + u) + 2 * cq]);
            v[4 * u] = fmaf(ga, oc2.x, __uint_as_float(acc[4 * u]) * inv_a);
            v[4 * u + 1] = fmaf(ga, oc2.y, __uint_as_float(acc[4 * u + 1]) * inv_a);
            v[4 * u + 2] = fmaf(gb, oc2.x, __uint_as_float(acc[4 * u + 2]) * inv_b);
            v[4 * u + 3] = fmaf(gb, oc2.y, __uint_as_float(acc[4 * u + 3]) * inv_b);
          }
          if (g.out_f32) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int col = 8 * (n0 + u) + 2 * cq;
              if (ta >= 0) *reinterpret_cast<float2*>(reinterpret_cast<float*>(a.o) + base_a + col) = make_float2(v[4 * u], v[4 * u + 1]);
              if (tk_b >= 0) *reinterpret_cast<float2*>(reinterpret_cast<float*>(a.o) + base_b + col) = make_float2(v[4 * u + 2], v[4 * u + 3]);
            }
          } else {
            // bf16 output and its rounding residual.  A thread holds bf16 pairs (columns 8n + 2cq, +1 of its two rows); stored
            // as such, every warp store touched eight lines with 16 bytes each and the 32 stores per thread kept the SM's
            // store path busy for ~2000 cycles per query block (clock64 trace: 3500 cycles from the last product to the end
            // of the epilogue).  The four threads of a row transpose 4 x 4 words with shuffles, so that a thread stores 16
            // contiguous bytes: 8 stores per thread instead of 32.
            uint32_t ha[4], la4[4], hb[4], lb4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              split_bf16x2(v[4 * u], v[4 * u + 1], ha[u], la4[u]);
              split_bf16x2(v[4 * u + 2], v[4 * u + 3], hb[u], lb4[u]);
            }
            quad_transpose4(ha, cq);
            quad_transpose4(hb, cq);
            const int col = 8 * (n0 + cq);
            if (ta >= 0) *reinterpret_cast<uint4*>(ob + base_a + col) = make_uint4(ha[0], ha[1], ha[2], ha[3]);
            if (tk_b >= 0) *reinterpret_cast<uint4*>(ob + base_b + col) = make_uint4(hb[0], hb[1], hb[2], hb[3]);
            if (a.o_res != nullptr) {
              quad_transpose4(la4, cq);
              quad_transpose4(lb4, cq);
              if (ta >= 0) *reinterpret_cast<uint4*>(a.o_res + base_a + col) = make_uint4(la4[0], la4[1], la4[2], la4[3]);
              if (tk_b >= 0) *reinterpret_cast<uint4*>(a.o_res + base_b + col) = make_uint4(lb4[0], lb4[1], lb4[2], lb4[3]);
            }
          }
        }
      }
      tc::mbar_arrive(&misc->tab_free[tb]);
      if (k > 0 && wg == 0 && sm_tid == 0 && misc->rescue_flag) {
        int slot = atomicAdd(a.rescue_count, 1);
        if (slot < a.rescue_cap) a.rescue_items[slot] = item;
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
  if (warp == 4) tc::tmem_dealloc(tmem_base, 512);
}

cudaError_t launch_fine_fwd_list(const Geo& g, const int* count, int cap, const int* items, const bf16* q, const bf16* k,
                                 const bf16* v, const float* gate, const int* row_ptr, const int* col_idx,
                                 const float* oc_hat, void* o, bf16* o_res, float* lse, cudaStream_t st);

bool fine_fwd_rows_supported(const Geo& g) { return g.N <= kFrMaxCubes; }

// workspace: [StatusBlock][rescue list] as for launch_fine_fwd_tc; the rescue counter is StatusBlock.pad[0].
cudaError_t launch_fine_fwd_rows_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                                    const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                                    float* lse, StatusBlock* status, cudaStream_t st) {
  CUtensorMap tq, tk, tv, tqt, tkt, tvt;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_text_tmap(&tqt, q, g, g.Hq) || !make_text_tmap(&tkt, k, g, g.Hkv) || !make_text_tmap(&tvt, v, g, g.Hkv))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if (g.N > kFrMaxCubes) return cudaErrorInvalidValue;
  FwdRowsArgs a;
  a.gate = gate; a.row_ptr = row_ptr; a.col_idx = col_idx; a.oc_hat = oc_hat; a.o = o; a.o_res = o_res; a.lse = lse;
  a.status = status;
  a.rescue_count = &status->pad[0];
  a.item_counter = &status->pad[1];
  a.rescue_items = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(status) + 256);
  a.rescue_cap = fwd_rescue_capacity();
  const int total = g.batch * g.Hq * g.N;
  const int grid = total < sms ? total : sms;
  // The softmax warpgroups raise their register count to 200 with the registers the service warpgroups give up
  // (setmaxnreg); that request would block for ever if the launch allocation were smaller than 128 per thread.
  {
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, g.D == 128 ? (const void*)fine_fwd_rows_tc_kernel<128> : (const void*)fine_fwd_rows_tc_kernel<64>)) != cudaSuccess) return e;
    if (fa.numRegs * kFrThreads < 256 * 56 + 256 * 200) return cudaErrorLaunchOutOfResources;
  }
  if (g.D == 128) {
    const size_t smb = FwdRows<128>::smem_bytes(g.N);
    if ((e = cudaFuncSetAttribute(fine_fwd_rows_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_rows_tc_kernel<128><<<grid, kFrThreads, smb, st>>>(tq, tk, tv, tqt, tkt, tvt, g, a);
  } else {
    const size_t smb = FwdRows<64>::smem_bytes(g.N);
    if ((e = cudaFuncSetAttribute(fine_fwd_rows_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smb))) return e;
    fine_fwd_rows_tc_kernel<64><<<grid, kFrThreads, smb, st>>>(tq, tk, tv, tqt, tkt, tvt, g, a);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // query blocks whose row sums left the safe range are redone with the exact running maximum
  return launch_fine_fwd_list(g, a.rescue_count, a.rescue_cap, a.rescue_items, q, k, v, gate, row_ptr, col_idx, oc_hat, o, o_res, lse, st);
}

}  // namespace vsa2
