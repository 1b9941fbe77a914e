// Backward of the fine branch (gradient of paper Eq. 12) for cubes of 128 tokens (the paper's 4 x 4 x 8 cube): both
// passes on 128 x 128 tiles with the tokens of the STATIONARY cube in the 128 rows of every accumulator.
//
// With P = exp(S * scale - lse), dP = dO V^T and dS = P * (dP - delta) * scale:
//
//   dQ pass (query cube i stationary, its kept key cubes j streamed, CSR map):
//     S  [128 q, 128 kv] = Q_i K_j^T        dP [128 q, 128 kv] = dO_i V_j^T         (A, B from shared memory, N = 128)
//     dQ [128 q, D]     += dS K_j                                                   (A = dS from TENSOR MEMORY)
//   dK/dV pass (key cube j stationary, the query cubes i that keep it streamed, CSC map, heads of a GQA group in turn):
//     S^T [128 kv, 128 q] = K_j Q_i^T       dP^T [128 kv, 128 q] = V_j dO_i^T
//     dV [128 kv, D]    += P^T dO_i         dK [128 kv, D]      += dS^T Q_i         (A = P^T, dS^T from tensor memory)
//
// Both passes are one kernel: "X0, X1" are the stationary pair of tiles (Q, dO or K, V), "Y0, Y1" the streamed pairs
// (K, V or Q, dO); S = X0 Y0^T, dP = X1 Y1^T, and the outputs are dS Y0 (and P Y1).  M = N = 128 runs the tensor pipe at
// its full rate; P and dS never touch shared memory (they overwrite, as bf16, the accumulator columns they were computed
// from), so a tile costs 64 KB of TMA writes and 160 KB (dQ) / 192 KB (dK/dV) of operand fetches for 12.6 / 16.8 MFLOP.
// A thread of the elementwise stage owns one row and 64 of the 128 columns of a tile; lse and delta are per-thread scalars
// in the dQ pass and per-column vectors (loaded one tile ahead by a service warp) in the dK/dV pass.
// SPLIT: P and dS enter the last products as [bf16(X) | bf16(X - bf16(X))] along the contraction (twice the steps), which
// removes their bf16 rounding from the gradients (see fine_bwd_tc.cu).
// Accumulators stay in tensor memory for the whole list of a cube: every output element is written once, by one thread,
// in a fixed order -- no floating-point atomics, bitwise reproducible.  Persistent CTAs, every wait bounded.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kW2Threads = 512;
constexpr int kW2RingA = 3;   // Y0 pairs: read by the S product and by the last product of a tile
constexpr int kW2RingB = 2;   // Y1 pairs

template <int D>
struct Bwd128 {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLOT = 2 * DH * kSlab;     // a pair of 64-token tiles: [channel half][block A | block B]
  static constexpr uint32_t OFF_RING_B = kW2RingA * SLOT;
  static constexpr uint32_t OFF_X0 = (kW2RingA + kW2RingB) * SLOT;
  static constexpr uint32_t OFF_X1 = OFF_X0 + SLOT;
  static constexpr uint32_t OFF_MISC = OFF_X1 + SLOT;
  static constexpr uint32_t MISC_BYTES = 2048;
  static constexpr size_t smem_bytes = OFF_MISC + MISC_BYTES + 1024;
};

struct Bwd128Misc {
  uint64_t st_full, st_empty, o_full, o_empty;
  uint64_t a_full[kW2RingA], a_empty[kW2RingA], b_full[kW2RingB], b_empty[kW2RingB];
  uint64_t s_full, s_free, dp_full[2], dp_free[2], p_ready, ds_ready, stat_full, stat_free, dlt_full, dlt_free, s_loaded, p_free, ds_free;
  ItemQueue items;
  uint32_t tmem_base;
  int abort_flag;
  unsigned char edge[kW2RingA][2];   // dQ pass: validity-table row of the two key blocks in each ring-A slot
  unsigned long long vmask[17];      // [table row of a block]: which of its 64 positions hold tokens
  alignas(16) float lse2[128];       // dK/dV pass: per query column of the current tile, lse * log2(e) (+inf = padding)
  alignas(16) float dlt[128];        // and delta
};
static_assert(sizeof(Bwd128Misc) <= 2048, "misc region too small");

struct Bwd128Args {
  int* item_counter;    // global, zero before the launch
  const float* lse;
  const float* delta;
  const int* ptr;       // map at 64-token-block level whose rows are the stationary blocks: CSR (dQ pass) or CSC (dK/dV pass)
  const int* idx;
  const float* c0;      // coarse terms per 64-token block and query head, or null: dQ_c (dQ pass) / dK_c (dK/dV pass)
  const float* c1;      // dV_c (dK/dV pass)
  void* out0;           // dQ / dK
  void* out1;           // dV
  StatusBlock* status;
  int* range_flag;      // fp16 form of the dQ pass and its fallback: as in DqArgs of the 64-token pass (when = 0: always runs)
  int when;
};

// The stationary cube of a work item and the lists of streamed cubes that meet it.
template <int PASS>
struct ItemLists {
  int bh_stat;    // head of the stationary pair (dQ pass: query head, dK/dV pass: KV head)
  int blk0;       // its first 64-token block (the cube is blocks blk0, blk0 + 1)
  int nl;         // number of lists: 1 (dQ pass) or the query heads per KV head
  int bhq0;       // query head of list 0 (lists belong to consecutive query heads)
  int bh_y0;      // head of the streamed tiles of list 0; list l streams head bh_y0 + l * y_step
  int y_step;
  __device__ __forceinline__ void init(const Geo& g, int item) {
    const int cubes = g.N / 2;
    blk0 = (item % cubes) * 2;
    bh_stat = item / cubes;
    if (PASS == 0) {
      const int b = bh_stat / g.Hq, hq = bh_stat % g.Hq;
      nl = 1;
      bhq0 = bh_stat;
      bh_y0 = b * g.Hkv + hq / g.rep;
      y_step = 0;
    } else {
      const int b = bh_stat / g.Hkv, hk = bh_stat % g.Hkv;
      nl = g.rep;
      bhq0 = b * g.Hq + hk * g.rep;
      bh_y0 = bhq0;
      y_step = 1;
    }
  }
  // tiles of the whole item (a list holds the two halves of every streamed cube, one after the other)
  __device__ __forceinline__ int tiles(const Geo& g, const Bwd128Args& a) const {
    int n = 0;
    for (int l = 0; l < nl; ++l) {
      const size_t p = (size_t)(bhq0 + l) * (g.N + 1) + blk0;
      n += (a.ptr[p + 1] - a.ptr[p]) >> 1;
    }
    return n;
  }
};

// loop over the tiles of an item: `tt` counts them inside the item, `tg` over the life of the CTA; ent[2 t], ent[2 t + 1] are
// the two streamed blocks of tile t of the list, bh_y the head they belong to, mh_ the query head of the list
#define VSA2_W2_TILES_BEGIN                                                                  \
  {                                                                                          \
    int tt = 0;                                                                              \
    for (int l_ = 0; l_ < il.nl; ++l_) {                                                     \
      const int mh_ = il.bhq0 + l_;                                                          \
      const int bh_y = il.bh_y0 + l_ * il.y_step;                                            \
      const int beg_ = a.ptr[(size_t)mh_ * (g.N + 1) + il.blk0];                             \
      const int nt_l = (a.ptr[(size_t)mh_ * (g.N + 1) + il.blk0 + 1] - beg_) >> 1;           \
      const int* ent = a.idx + (size_t)mh_ * g.nnz_cap + beg_;                               \
      (void)bh_y; (void)ent; (void)mh_;                                                      \
      for (int t = 0; t < nt_l; ++t, ++tt, ++tg) {
#define VSA2_W2_TILES_END \
      }                   \
    }                     \
  }

// acc[128, D] (+)= A[128, 128 (x2)] * Y[128 tokens, D]: A from tensor memory at `tm_a` (a 128-column region: the 32 values
// of column chunk c as bf16 pairs in columns 32 c .. 32 c + 15, with SPLIT their low-order parts in 32 c + 16 .. 32 c + 31),
// Y a ring slot (MN-major B operand).
// COMPACT (not with SPLIT): the 128 values of a row as 64 consecutive columns of bf16 pairs.
// F16: A and Y hold fp16.
template <int D, bool SPLIT, bool COMPACT, bool F16 = false>
__device__ __forceinline__ void mma_out_ts(uint32_t tm_acc, uint32_t tm_a, uint32_t slot_addr, bool accumulate_first) {
  constexpr uint32_t idesc = F16 ? tc::idesc_f16(128, D, false, true) : tc::idesc_bf16(128, D, false, true);
  constexpr uint32_t lbo = (D == 128) ? 2 * kSlab : 0;
  const uint64_t db = tc::smem_desc_sw128(slot_addr, lbo, 1024);
  constexpr int STEPS = SPLIT ? 16 : 8;
#pragma unroll
  for (int ks = 0; ks < STEPS; ++ks) {
    const int c = SPLIT ? ks / 4 : ks / 2, part = SPLIT ? (ks / 2) % 2 : 0, sub = ks % 2;
    const int rr = 32 * c + 16 * sub;                                   // first token row of this step
    const uint64_t ob = (uint64_t)(((rr / 64) * kSlab + (rr % 64) * 128) >> 4);
    tc::mma_ts(tm_acc, tm_a + (COMPACT ? 8 * ks : 32 * c + 16 * part + 8 * sub), db + ob, idesc, accumulate_first || ks > 0);
  }
}

// 32 values -> bf16 pairs (and their low-order parts) into the tensor-memory columns they came from
template <bool SPLIT>
__device__ __forceinline__ void store_operand_chunk(uint32_t taddr, const float (&v)[32]) {
  uint32_t hi[16];
  if constexpr (SPLIT) {
    uint32_t lo[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) split_bf16x2(v[2 * e], v[2 * e + 1], hi[e], lo[e]);
    tc::tmem_st_32x32b_x16(taddr, hi);
    tc::tmem_st_32x32b_x16(taddr + 16, lo);
  } else {
#pragma unroll
    for (int e = 0; e < 16; ++e) hi[e] = pack_bf16x2(v[2 * e], v[2 * e + 1]);
    tc::tmem_st_32x32b_x16(taddr, hi);
  }
}

// the same as fp16 pairs (clamped at the largest fp16 value); `sat` collects the largest magnitude
__device__ __forceinline__ void store_operand_chunk_f16(uint32_t taddr, const float (&v)[32], float& sat) {
  uint32_t h[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    h[e] = pack_f16x2_sat(v[2 * e], v[2 * e + 1]);
    sat = max3_abs(sat, v[2 * e], v[2 * e + 1]);
  }
  tc::tmem_st_32x32b_x16(taddr, h);
}

// Roles (512 threads): warps 0..3 = TMA producers (ring A / ring B x first / second block of a pair; warp 0 also brings the
// stationary tiles and schedules the CTA's work items), warp 4 = issuer of S, warp 5 = issuer of dP, warp 6 = issuer of
// the output products, warp 7 = loader of the per-column lse and delta (dK/dV pass), warps 8..15 = elementwise stage +
// epilogue (thread = row r of the tile x one half of its columns).
// F16 (without SPLIT): the maps of X0 and Y0 (Q and K, in the order of the pass) point at fp16 copies and dS is rounded to fp16,
// so S and the dQ (dK) product are fp16 x fp16 instructions; dP, P and the dV product stay bf16.  See the 64-token passes; as
// there, only the dQ pass tracks the magnitude of dS.
template <int D, int PASS, bool SPLIT, bool F16 = false>
__global__ void __launch_bounds__(kW2Threads, 1)
fine_bwd128_tc_kernel(const __grid_constant__ CUtensorMap tm_x0, const __grid_constant__ CUtensorMap tm_x1,
                      const __grid_constant__ CUtensorMap tm_y0, const __grid_constant__ CUtensorMap tm_y1, Geo g,
                      Bwd128Args a) {
  using C = Bwd128<D>;
  static_assert(PASS == 0 || !SPLIT, "the dK/dV pass has no room for the low-order parts of P and dS");
  static_assert(!F16 || !SPLIT, "the fp16 forms carry no pairs");
  if (a.when != 0 && ((*a.range_flag != 0) != (a.when == 2))) return;     // (the flag is final before this launch starts)
  constexpr uint32_t NDP = PASS == 0 ? 2 : 1;                  // dP buffers
  // dQ pass: S 0; dP buffers 128, 256 (dS overwrites the dP it came from); dQ 384.
  // dK/dV pass: S^T and dP^T take turns in the staging columns 0..127 (each is pulled into registers as soon as it is
  // complete, so the next product can start while the elementwise stage still computes); P^T at 128 and dS^T at 192 as
  // bf16 pairs (64 columns each); dK 256, dV 384.
  constexpr uint32_t TM_S = 0, TM_DP = PASS == 0 ? 128 : 0, TM_P = 128, TM_DS = 192, TM_ACC0 = PASS == 0 ? 384 : 256, TM_ACC1 = 384;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* x0_tile = smem + C::OFF_X0;
  unsigned char* x1_tile = smem + C::OFF_X1;
  Bwd128Misc* misc = reinterpret_cast<Bwd128Misc*>(smem + C::OFF_MISC);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * (PASS == 0 ? g.Hq : g.Hkv) * (g.N / 2);
  const float c2 = g.scale * 1.4426950408889634f;

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
    tc::mbar_init(&misc->st_full, 1);
    tc::mbar_init(&misc->st_empty, 2);                      // the issuers of S and dP
    tc::mbar_init(&misc->o_full, PASS == 0 ? 1 : 2);
    tc::mbar_init(&misc->o_empty, 256);
    for (int s = 0; s < kW2RingA; ++s) {
      tc::mbar_init(&misc->a_full[s], 2);
      tc::mbar_init(&misc->a_empty[s], 1);
    }
    for (int s = 0; s < kW2RingB; ++s) {
      tc::mbar_init(&misc->b_full[s], 2);
      tc::mbar_init(&misc->b_empty[s], PASS == 0 ? 1 : 2);  // a Y1 slot is read by dP and, in the dK/dV pass, by dV
    }
    tc::mbar_init(&misc->s_full, 1);
    tc::mbar_init(&misc->s_free, 256);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->dp_full[s], 1);
      tc::mbar_init(&misc->dp_free[s], 1);
    }
    tc::mbar_init(&misc->p_ready, 256);
    tc::mbar_init(&misc->ds_ready, 256);
    tc::mbar_init(&misc->stat_full, 32);
    tc::mbar_init(&misc->stat_free, 256);
    tc::mbar_init(&misc->dlt_full, 32);
    tc::mbar_init(&misc->dlt_free, 256);
    tc::mbar_init(&misc->s_loaded, 256);
    tc::mbar_init(&misc->p_free, 1);
    tc::mbar_init(&misc->ds_free, 1);
    item_queue_init(&misc->items, 4 + 3 + (PASS == 0 ? 0 : 1) + 256);
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_x0);
    tc::prefetch_tmap(&tm_x1);
    tc::prefetch_tmap(&tm_y0);
    tc::prefetch_tmap(&tm_y1);
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
      const int which = warp & 1;                           // 0: ring A (Y0) + the stationary tiles, 1: ring B (Y1)
      const int my_blk = warp >> 1;                         // 0: first block of a pair, 1: second
      const CUtensorMap* tm = which == 0 ? &tm_y0 : &tm_y1;
      const uint32_t nslots = which == 0 ? kW2RingA : kW2RingB;
      uint64_t* full = which == 0 ? misc->a_full : misc->b_full;
      uint64_t* empty = which == 0 ? misc->a_empty : misc->b_empty;
      unsigned char* ring = smem + (which == 0 ? 0 : C::OFF_RING_B);
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
        ItemLists<PASS> il;
        il.init(g, item);
        if (il.tiles(g, a) == 0) continue;
        if (warp == 0) {
          int ok = 1;
          if (lane == 0) {
            ok = tc::mbar_wait_parked(&misc->st_empty, (n_items & 1) ^ 1, &misc->abort_flag);
            if (ok) tc::mbar_expect_tx(&misc->st_full, 2 * C::SLOT);
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
          if (lane < 4 * C::DH) {
            const int x = lane / (2 * C::DH), rem = lane % (2 * C::DH), h = rem >> 1, m = rem & 1;
            int c1, c2_, c3;
            block_box(g, il.blk0 + m, c1, c2_, c3);
            tc::tma_load_5d((x == 0 ? x0_tile : x1_tile) + (2 * h + m) * kSlab, x == 0 ? &tm_x0 : &tm_x1, &misc->st_full,
                            h * 64, c1, c2_, c3, il.bh_stat);
          }
        }
        ++n_items;
        for (int l_ = 0; l_ < il.nl; ++l_) {
          const int mh = il.bhq0 + l_, bh_y = il.bh_y0 + l_ * il.y_step;
          const int beg = a.ptr[(size_t)mh * (g.N + 1) + il.blk0];
          const int nt_l = (a.ptr[(size_t)mh * (g.N + 1) + il.blk0 + 1] - beg) >> 1;
          if (nt_l == 0) continue;
          const int* ent = a.idx + (size_t)mh * g.nnz_cap + beg;
          int j = ent[my_blk];
          for (int t = 0; t < nt_l; ++t, ++tg) {
            int c1, c2_, c3;
            block_box(g, j, c1, c2_, c3);
            const unsigned ef = cube_edge_flags(g, j);
            if (t + 1 < nt_l) j = ent[2 * t + 2 + my_blk];        // the next entry is on its way while this warp waits
            const uint32_t slot = tg % nslots, par = (tg / nslots) & 1;
            int ok = 1;
            if (lane == 0) {
              ok = tc::mbar_wait_parked(&empty[slot], par ^ 1, &misc->abort_flag);
              if (ok) {
                if (PASS == 0 && which == 0) misc->edge[slot][my_blk] = (unsigned char)ef;
                tc::mbar_expect_tx(&full[slot], C::SLOT / 2);
              }
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) goto done;
            if (lane < C::DH)
              tc::tma_load_5d(ring + slot * C::SLOT + (2 * lane + my_blk) * kSlab, tm, &full[slot], lane * 64, c1, c2_, c3, bh_y);
          }
        }
      }
    } else if (warp == 4 || warp == 5) {
      // ---------------------------------------------------------------- issuers of S = X0 Y0^T (warp 4) and dP = X1 Y1^T
      // (warp 5): the whole warp runs the loop, one elected lane issues
      const bool is_s = warp == 4;
      const uint32_t idesc = (F16 && is_s) ? tc::idesc_f16(128, 128, false, false) : tc::idesc_bf16(128, 128, false, false);
      const uint64_t dx = tc::smem_desc_sw128(tc::smem_u32(is_s ? x0_tile : x1_tile), 16, 1024);
      const uint32_t ring0 = tc::smem_u32(smem) + (is_s ? 0 : C::OFF_RING_B);
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        ItemLists<PASS> il;
        il.init(g, item);
        const int nt_all = il.tiles(g, a);
        if (nt_all == 0) continue;
        VSA2_WAIT(&misc->st_full, n_items & 1);
        VSA2_W2_TILES_BEGIN
          uint32_t slot;
          if (is_s) {
            slot = tg % kW2RingA;
            VSA2_WAIT(&misc->a_full[slot], (tg / kW2RingA) & 1);
            VSA2_WAIT(&misc->s_free, (tg & 1) ^ 1);
          } else {
            slot = tg % kW2RingB;
            VSA2_WAIT(&misc->b_full[slot], (tg / kW2RingB) & 1);
            if (PASS == 0) VSA2_WAIT(&misc->dp_free[tg % NDP], ((tg / NDP) & 1) ^ 1);
            else VSA2_WAIT(&misc->s_loaded, tg & 1);        // S^T of this tile has left the staging columns
          }
          tc::tc_fence_after();
          if (tc::elect_one()) {
            const uint64_t dy = tc::smem_desc_sw128(ring0 + slot * C::SLOT, 16, 1024);
            const uint32_t acc = tmem_base + (is_s ? TM_S : TM_DP + (tg % NDP) * 128);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint64_t off = (uint64_t)(((ks / 4) * 2 * kSlab + (ks % 4) * 32) >> 4);
              tc::mma_ss(acc, dx + off, dy + off, idesc, ks > 0);
            }
            if (is_s) {
              tc::mma_commit(&misc->s_full);
            } else {
              tc::mma_commit(&misc->dp_full[tg % NDP]);
              tc::mma_commit(&misc->b_empty[slot]);
            }
            if (tt == nt_all - 1) tc::mma_commit(&misc->st_empty);
          }
          __syncwarp();
        VSA2_W2_TILES_END
        ++n_items;
      }
    } else if (warp == 6) {
      // ---------------------------------------------------------------- issuer of the output products (converged warp)
      const uint32_t ring_a = tc::smem_u32(smem), ring_b = tc::smem_u32(smem) + C::OFF_RING_B;
      uint32_t tg = 0, n_items = 0;
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        ItemLists<PASS> il;
        il.init(g, item);
        const int nt_all = il.tiles(g, a);
        if (nt_all == 0) continue;
        VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);
        VSA2_W2_TILES_BEGIN
          const uint32_t sa = tg % kW2RingA, sb = tg % kW2RingB;
          if (PASS == 1) {
            // dV += P^T dO_i: P depends on S only, so it can be ready before the dO pair of the tile has landed
            VSA2_WAIT(&misc->b_full[sb], (tg / kW2RingB) & 1);
            VSA2_WAIT(&misc->p_ready, tg & 1);
            tc::tc_fence_after();
            if (tc::elect_one()) {
              mma_out_ts<D, SPLIT, true>(tmem_base + TM_ACC1, tmem_base + TM_P, ring_b + sb * C::SLOT, tt > 0);
              tc::mma_commit(&misc->b_empty[sb]);
              tc::mma_commit(&misc->p_free);
              if (tt == nt_all - 1) tc::mma_commit(&misc->o_full);
            }
            __syncwarp();
          }
          VSA2_WAIT(&misc->ds_ready, tg & 1);
          tc::tc_fence_after();
          if (tc::elect_one()) {
            if (PASS == 0) mma_out_ts<D, SPLIT, false, F16>(tmem_base + TM_ACC0, tmem_base + TM_DP + (tg % NDP) * 128, ring_a + sa * C::SLOT, tt > 0);
            else mma_out_ts<D, SPLIT, true, F16>(tmem_base + TM_ACC0, tmem_base + TM_DS, ring_a + sa * C::SLOT, tt > 0);
            tc::mma_commit(&misc->a_empty[sa]);
            tc::mma_commit(PASS == 0 ? &misc->dp_free[tg % NDP] : &misc->ds_free);
            if (tt == nt_all - 1) tc::mma_commit(&misc->o_full);
          }
          __syncwarp();
        VSA2_W2_TILES_END
        ++n_items;
      }
    } else if (PASS == 1) {
      // ---------------------------------------------------------------- warp 7, dK/dV pass: lse and delta of the 128 query
      // columns of every tile.  Global loads take a microsecond under this kernel's TMA traffic, so the values of tile
      // t + 1 and the list entries of tile t + 2 are requested before the warp waits to publish tile t.
      uint32_t tg = 0;
      // (a thread issues in order: nothing may depend on a load before the iteration that publishes it, so the raw values
      // and the validity bits travel, and the arithmetic is done when they are written.  The index arithmetic avoids
      // divisions inside the tile loop: they run on the same unit as the exponentials of the elementwise warps and
      // would wait behind them.)
      int pos_off[2];            // raster offset of this lane's two positions inside a block
      unsigned pos_ok[2];        // bit f: the position holds a token in a block with edge flags f
#pragma unroll
      for (int pp = 0; pp < 2; ++pp) {
        CubePos cp;
        cp.init(g, lane + 32 * pp);
        pos_off[pp] = (cp.bt * g.H + cp.bh) * g.W + cp.bw;
        pos_ok[pp] = 0u;
        for (unsigned f = 0; f < 16; ++f)
          if (cp.valid(f, g)) pos_ok[pp] |= 1u << f;
      }
      // list entry -> (raster offset of the block's first position, edge flags)
      auto entry_geo = [&](int e, int& base, int& fl) {
        int nt, nh, nw;
        cube_coords(g, e, nt, nh, nw);
        base = ((nt * g.Bt) * g.H + nh * g.Bh) * g.W + nw * g.Bw;
        fl = (int)cube_edge_flags_at(g, nt, nh, nw);
      };
      auto load_stats = [&](int mh, int base0, int fl0, int base1, int fl1, float (&ls)[4], float (&dl)[4], unsigned& ok) {
        ok = 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool v = (pos_ok[u & 1] >> (u < 2 ? fl0 : fl1)) & 1u;
          const int l = (u < 2 ? base0 : base1) + pos_off[u & 1];
          const size_t p = (size_t)mh * g.S + (v ? l : 0);
          ls[u] = a.lse[p];
          dl[u] = a.delta[p];
          if (v) ok |= 1u << u;
        }
      };
      for (uint32_t seq = 0;; ++seq) {
        VSA2_NEXT_ITEM_WARP(item, seq);
        ItemLists<PASS> il;
        il.init(g, item);
        for (int l_ = 0; l_ < il.nl; ++l_) {
          const int mh = il.bhq0 + l_;
          const int beg = a.ptr[(size_t)mh * (g.N + 1) + il.blk0];
          const int nt_l = (a.ptr[(size_t)mh * (g.N + 1) + il.blk0 + 1] - beg) >> 1;
          if (nt_l == 0) continue;
          const int* ent = a.idx + (size_t)mh * g.nnz_cap + beg;
          // Three register sets rotate through "being published", "in flight", "being requested" (a copy between sets
          // would be a use, and stall).  The list entries come 16 tiles at a time, one per lane, a batch ahead.
          float a_ls[4], a_dl[4], b_ls[4], b_dl[4], c_ls[4], c_dl[4];
          unsigned a_ok = 0u, b_ok = 0u, c_ok = 0u;
#pragma unroll
          for (int u = 0; u < 4; ++u) a_ls[u] = a_dl[u] = b_ls[u] = b_dl[u] = c_ls[u] = c_dl[u] = 0.f;
          const int n_ent = 2 * nt_l;
          int cur_base, cur_fl, nxt_base, nxt_fl;           // lane k: entry k of the current / next batch of 32 entries
          entry_geo(ent[min(lane, n_ent - 1)], cur_base, cur_fl);
          entry_geo(ent[min(32 + lane, n_ent - 1)], nxt_base, nxt_fl);
          int t0 = 0;                                       // first tile of the current batch of entries
          // the two blocks of tile T (T - t0 in 0 .. 31)
#define VSA2_W2_ENTRY(T, B0, F0, B1, F1)                                                                      \
  {                                                                                                           \
    const int k_ = 2 * ((T) - t0);                                                                            \
    const bool first_ = k_ < 32;                                                                              \
    const int cb0_ = __shfl_sync(0xffffffffu, cur_base, k_ & 31), nb0_ = __shfl_sync(0xffffffffu, nxt_base, k_ & 31);          \
    const int cb1_ = __shfl_sync(0xffffffffu, cur_base, (k_ + 1) & 31), nb1_ = __shfl_sync(0xffffffffu, nxt_base, (k_ + 1) & 31); \
    const int cf0_ = __shfl_sync(0xffffffffu, cur_fl, k_ & 31), nf0_ = __shfl_sync(0xffffffffu, nxt_fl, k_ & 31);              \
    const int cf1_ = __shfl_sync(0xffffffffu, cur_fl, (k_ + 1) & 31), nf1_ = __shfl_sync(0xffffffffu, nxt_fl, (k_ + 1) & 31);  \
    B0 = first_ ? cb0_ : nb0_;                                                                                \
    B1 = first_ ? cb1_ : nb1_;                                                                                \
    F0 = first_ ? cf0_ : nf0_;                                                                                \
    F1 = first_ ? cf1_ : nf1_;                                                                                \
  }
          {
            int b0, f0, b1, f1;
            VSA2_W2_ENTRY(0, b0, f0, b1, f1)
            load_stats(mh, b0, f0, b1, f1, a_ls, a_dl, a_ok);
            if (nt_l > 1) {
              VSA2_W2_ENTRY(1, b0, f0, b1, f1)
              load_stats(mh, b0, f0, b1, f1, b_ls, b_dl, b_ok);
            }
          }
#define VSA2_W2_STAT_STEP(CUR, FREE, T)                                                                       \
  {                                                                                                           \
    if ((T) - t0 == 16) {                                                                                     \
      t0 += 16;                                                                                               \
      cur_base = nxt_base;                                                                                    \
      cur_fl = nxt_fl;                                                                                        \
      entry_geo(ent[min(2 * t0 + 32 + lane, n_ent - 1)], nxt_base, nxt_fl);                                   \
    }                                                                                                         \
    if ((T) + 2 < nt_l) {                                                                                     \
      int b0_, f0_, b1_, f1_;                                                                                 \
      VSA2_W2_ENTRY((T) + 2, b0_, f0_, b1_, f1_)                                                              \
      load_stats(mh, b0_, f0_, b1_, f1_, FREE##_ls, FREE##_dl, FREE##_ok);                                    \
    }                                                                                                         \
    VSA2_WAIT_PARKED(&misc->stat_free, (tg & 1) ^ 1);                                                         \
    _Pragma("unroll") for (int u = 0; u < 4; ++u)                                                             \
        misc->lse2[lane + 32 * u] = ((CUR##_ok >> u) & 1u) ? CUR##_ls[u] * 1.4426950408889634f : INFINITY;    \
    tc::mbar_arrive(&misc->stat_full);                                                                        \
    VSA2_WAIT_PARKED(&misc->dlt_free, (tg & 1) ^ 1);                                                          \
    _Pragma("unroll") for (int u = 0; u < 4; ++u)                                                             \
        misc->dlt[lane + 32 * u] = ((CUR##_ok >> u) & 1u) ? CUR##_dl[u] : 0.f;                                \
    tc::mbar_arrive(&misc->dlt_full);                                                                         \
    ++tg;                                                                                                     \
  }
          // (the two vectors are freed at different times: lse after the exponentials of the previous tile, delta after its dS)
          for (int t = 0; t < nt_l; t += 3) {
            VSA2_W2_STAT_STEP(a, c, t)
            if (t + 1 < nt_l) VSA2_W2_STAT_STEP(b, a, t + 1)
            if (t + 2 < nt_l) VSA2_W2_STAT_STEP(c, b, t + 2)
          }
#undef VSA2_W2_ENTRY
#undef VSA2_W2_STAT_STEP
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ elementwise stage + epilogue (256 threads)
    tc::reg_inc<200>();
    const int quad = warp & 3;
    const int half = (warp - 8) >> 2;            // which 64 columns of a tile, and which D / 2 channels in the epilogue
    const int row = (quad << 5) | lane;          // row of the tile = token of the stationary cube = tensor-memory lane
    const int member = row >> 6;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint32_t tg = 0, n_items = 0;
    float sat = 0.f;          // F16: largest magnitude of the dS values this thread rounded
    for (uint32_t n_all = 0;; ++n_all) {
      if constexpr (F16) {
        // a dS beyond the fp16 range (it was clamped): the result of this launch is not to be used, the fallback launch redoes it
        if (sat >= 65504.f) {
          atomicExch(a.range_flag, 1);
          sat = 0.f;
        }
      }
      VSA2_NEXT_ITEM(item, n_all);
      ItemLists<PASS> il;
      il.init(g, item);
      const int nt_all = il.tiles(g, a);
      const int blk = il.blk0 + member;
      const int l_tok = block_token(g, blk, row & 63);
      float lse2 = INFINITY, dlt = 0.f;
      if (PASS == 0 && l_tok >= 0) {
        lse2 = a.lse[(size_t)il.bh_stat * g.S + l_tok] * 1.4426950408889634f;
        dlt = a.delta[(size_t)il.bh_stat * g.S + l_tok];
      }
      if (nt_all > 0) {
        VSA2_W2_TILES_BEGIN
          const uint32_t dpb = (tg % NDP) * 128;
          uint32_t pf[64];                 // S, then P (as float bits) of this thread's 64 columns
          VSA2_WAIT(&misc->s_full, tg & 1);
          tc::tc_fence_after();
          unsigned long long vm = ~0ull;
          if (PASS == 0) vm = misc->vmask[misc->edge[tg % kW2RingA][half]];
          else VSA2_WAIT(&misc->stat_full, tg & 1);
          tc::tmem_ld32(lane_addr + TM_S + 64 * half, *reinterpret_cast<uint32_t(*)[32]>(&pf[0]));
          tc::tmem_ld32(lane_addr + TM_S + 64 * half + 32, *reinterpret_cast<uint32_t(*)[32]>(&pf[32]));
          if (PASS == 0) {
            // dP of this tile is normally there already (two buffers): fetch it together with S, then one pass over the
            // registers: P = exp2(S c2 - lse), dS = P (dP - delta); the factor `scale` goes into the epilogue
            uint32_t dp[64];
            VSA2_WAIT(&misc->dp_full[tg % NDP], (tg / NDP) & 1);
            tc::tc_fence_after();
            tc::tmem_ld32(lane_addr + TM_DP + dpb + 64 * half, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
            tc::tmem_ld32(lane_addr + TM_DP + dpb + 64 * half + 32, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
            tc::tmem_ld_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&misc->s_free);          // S is in registers: the next tile's S product may overwrite it
            const bool full = vm == ~0ull;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              float ds[32];
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float p = ex2_approx(fmaf(__uint_as_float(pf[32 * c + e]), c2, -lse2));
                const float d = p * (__uint_as_float(dp[32 * c + e]) - dlt);
                ds[e] = (full || ((vm >> (32 * c + e)) & 1ull)) ? d : 0.f;
              }
              // dS over the dP columns it came from
              if constexpr (F16) store_operand_chunk_f16(lane_addr + TM_DP + dpb + 64 * half + 32 * c, ds, sat);
              else store_operand_chunk<SPLIT>(lane_addr + TM_DP + dpb + 64 * half + 32 * c, ds);
            }
          } else {
            tc::tmem_ld_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&misc->s_loaded);        // S^T is in registers: dP^T may take the staging columns
            VSA2_WAIT(&misc->p_free, (tg & 1) ^ 1);  // dV of the previous tile has read its P^T
            tc::tc_fence_after();
            uint32_t dp[64];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              const float4* l4 = reinterpret_cast<const float4*>(misc->lse2 + 64 * half + 32 * c);
              float pc[32];
#pragma unroll
              for (int e4 = 0; e4 < 8; ++e4) {
                const float4 ls = l4[e4];
                pc[4 * e4 + 0] = ex2_approx(fmaf(__uint_as_float(pf[32 * c + 4 * e4 + 0]), c2, -ls.x));
                pc[4 * e4 + 1] = ex2_approx(fmaf(__uint_as_float(pf[32 * c + 4 * e4 + 1]), c2, -ls.y));
                pc[4 * e4 + 2] = ex2_approx(fmaf(__uint_as_float(pf[32 * c + 4 * e4 + 2]), c2, -ls.z));
                pc[4 * e4 + 3] = ex2_approx(fmaf(__uint_as_float(pf[32 * c + 4 * e4 + 3]), c2, -ls.w));
              }
#pragma unroll
              for (int e = 0; e < 32; ++e) pf[32 * c + e] = __float_as_uint(pc[e]);
              store_operand_chunk<false>(lane_addr + TM_P + 32 * half + 16 * c, pc);
              if (c == 0) {
                // half way through the exponentials dP^T of this tile is complete: pull it into registers now, so that
                // S^T of the next tile can be computed while this stage finishes the tile
                VSA2_WAIT(&misc->dp_full[0], tg & 1);
                tc::tc_fence_after();
                tc::tmem_ld32(lane_addr + TM_DP + 64 * half, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
                tc::tmem_ld32(lane_addr + TM_DP + 64 * half + 32, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
                tc::tmem_ld_wait();
                tc::tc_fence_before();
                tc::mbar_arrive(&misc->s_free);
              }
            }
            tc::mbar_arrive(&misc->stat_free);       // the lse vector may be replaced
            tc::tmem_st_wait();
            tc::tc_fence_before();
            tc::mbar_arrive(&misc->p_ready);
            VSA2_WAIT(&misc->dlt_full, tg & 1);
            VSA2_WAIT(&misc->ds_free, (tg & 1) ^ 1); // dK of the previous tile has read its dS^T
            tc::tc_fence_after();
            // dS^T = P^T (dP^T - delta)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              float ds[32];
              const float4* d4 = reinterpret_cast<const float4*>(misc->dlt + 64 * half + 32 * c);
#pragma unroll
              for (int e4 = 0; e4 < 8; ++e4) {
                const float4 dl = d4[e4];
                ds[4 * e4 + 0] = __uint_as_float(pf[32 * c + 4 * e4 + 0]) * (__uint_as_float(dp[32 * c + 4 * e4 + 0]) - dl.x);
                ds[4 * e4 + 1] = __uint_as_float(pf[32 * c + 4 * e4 + 1]) * (__uint_as_float(dp[32 * c + 4 * e4 + 1]) - dl.y);
                ds[4 * e4 + 2] = __uint_as_float(pf[32 * c + 4 * e4 + 2]) * (__uint_as_float(dp[32 * c + 4 * e4 + 2]) - dl.z);
                ds[4 * e4 + 3] = __uint_as_float(pf[32 * c + 4 * e4 + 3]) * (__uint_as_float(dp[32 * c + 4 * e4 + 3]) - dl.w);
              }
              if constexpr (F16) {     // (a dS at the clamp: the dQ pass has met the same value and raised the flag)
                uint32_t h[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) h[e] = pack_f16x2_sat(ds[2 * e], ds[2 * e + 1]);
                tc::tmem_st_32x32b_x16(lane_addr + TM_DS + 32 * half + 16 * c, h);
              } else {
                store_operand_chunk<false>(lane_addr + TM_DS + 32 * half + 16 * c, ds);
              }
            }
          }
          if (PASS == 1) tc::mbar_arrive(&misc->dlt_free);
          tc::tmem_st_wait();
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->ds_ready);
        VSA2_W2_TILES_END
        VSA2_WAIT(&misc->o_full, n_items & 1);
        tc::tc_fence_after();
      }

      // epilogue: out[l, d] = acc[row, d] + (sum over the query heads of) coarse[block, d] / count(block); this thread
      // writes D / 2 channels of its row
      {
        constexpr int COLS = D / 2;
        constexpr int NOUT = PASS == 0 ? 1 : 2;
        const float inv_cnt = 1.f / (float)cube_count(g, blk);
#pragma unroll
        for (int o = 0; o < NOUT; ++o) {
          const float* cterm = o == 0 ? a.c0 : a.c1;
          void* out = o == 0 ? a.out0 : a.out1;
#pragma unroll
          for (int c = 0; c < COLS / 32; ++c) {
            const int col0 = half * COLS + 32 * c;
            uint32_t acc[32];
            if (nt_all > 0) {
              tc::tmem_ld32(lane_addr + (o == 0 ? TM_ACC0 : TM_ACC1) + col0, acc);
              tc::tmem_ld_wait();
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e) acc[e] = 0u;
            }
            if (l_tok < 0) continue;
            float val[32];
            const float sc = (PASS == 0 || o == 0) ? g.scale : 1.f;      // dQ, dK = scale * (dS Y0); dV = P Y1
#pragma unroll
            for (int e = 0; e < 32; ++e) val[e] = __uint_as_float(acc[e]) * sc;
            if (cterm != nullptr) {
              for (int l = 0; l < il.nl; ++l) {
                const float4* c4 = reinterpret_cast<const float4*>(cterm + ((size_t)(il.bhq0 + l) * g.Nvid + blk) * D + col0);
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) {
                  const float4 cv = c4[e4];
                  val[4 * e4 + 0] = fmaf(cv.x, inv_cnt, val[4 * e4 + 0]);
                  val[4 * e4 + 1] = fmaf(cv.y, inv_cnt, val[4 * e4 + 1]);
                  val[4 * e4 + 2] = fmaf(cv.z, inv_cnt, val[4 * e4 + 2]);
                  val[4 * e4 + 3] = fmaf(cv.w, inv_cnt, val[4 * e4 + 3]);
                }
              }
            }
            const size_t idx = ((size_t)il.bh_stat * g.S + l_tok) * D + col0;
            if (g.out_f32) {
              float* dst = reinterpret_cast<float*>(out) + idx;
#pragma unroll
              for (int e = 0; e < 32; e += 4) *reinterpret_cast<float4*>(dst + e) = make_float4(val[e], val[e + 1], val[e + 2], val[e + 3]);
            } else {
              bf16* dst = reinterpret_cast<bf16*>(out) + idx;
#pragma unroll
              for (int e = 0; e < 32; e += 8)
                *reinterpret_cast<uint4*>(dst + e) = make_uint4(pack_bf16x2(val[e], val[e + 1]), pack_bf16x2(val[e + 2], val[e + 3]),
                                                                pack_bf16x2(val[e + 4], val[e + 5]), pack_bf16x2(val[e + 6], val[e + 7]));
            }
          }
        }
        if (nt_all > 0) {
          tc::tc_fence_before();
          tc::mbar_arrive(&misc->o_empty);
        }
      }
      if (nt_all > 0) ++n_items;
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
  if (warp == 4) tc::tmem_dealloc(tmem_base, 512);
}

// A KV cube of a GQA group sums rep times as many query cubes: there the plain bf16 rounding of P and dS passes 2e-2 and
// the dK/dV pass carries them as bf16 pairs, which only the 64-token kernel has room for.
bool fine_bwd_dkv_wants_pair(const Geo& g) {
  return (g.flags & VSA2_FLAG_PRECISE_BWD) || (g.rep > 1 && !(g.flags & VSA2_FLAG_FAST_BWD));
}

// `g`: the half-cube geometry of a 128-token-cube problem (two consecutive blocks along w are one cube)
bool fine_bwd128_supported(const Geo& g) {
  return g.Lt == 0 && g.N % 2 == 0 && g.rep <= 16 && (g.D == 64 || g.D == 128);
}

template <int D, int PASS, bool SPLIT, bool F16 = false>
static cudaError_t launch_bwd128(const CUtensorMap& x0, const CUtensorMap& x1, const CUtensorMap& y0, const CUtensorMap& y1,
                                 const Geo& g, const Bwd128Args& a, int grid, cudaStream_t st) {
  cudaError_t e;
  cudaFuncAttributes fa;
  if ((e = cudaFuncGetAttributes(&fa, fine_bwd128_tc_kernel<D, PASS, SPLIT, F16>)) != cudaSuccess) return e;
  if (fa.numRegs * kW2Threads < 256 * 56 + 256 * 200) return cudaErrorLaunchOutOfResources;
  if ((e = cudaFuncSetAttribute(fine_bwd128_tc_kernel<D, PASS, SPLIT, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)Bwd128<D>::smem_bytes)))
    return e;
  fine_bwd128_tc_kernel<D, PASS, SPLIT, F16><<<grid, kW2Threads, Bwd128<D>::smem_bytes, st>>>(x0, x1, y0, y1, g, a);
  return cudaGetLastError();
}

// dQ pass: row_ptr / col_idx is the map expanded to 64-token blocks, dqc per block (or null); the other arguments as for
// launch_fine_bwd_dq_tc
cudaError_t launch_fine_bwd128_dq_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                     const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                                     const float* dqc, void* dq, StatusBlock* status, cudaStream_t st, void* q16, void* k16) {
  if (!fine_bwd128_supported(g)) return cudaErrorInvalidValue;
  const bool f16 = fine_bwd_dq_uses_f16(g) && q16 != nullptr && k16 != nullptr;
  CUtensorMap tq, tk, tv, tdo, tq16, tk16;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_cube_tmap(&tdo, d_o, g, g.Hq))
    return cudaErrorInvalidValue;
  if (f16 && (!make_cube_tmap(&tq16, reinterpret_cast<const bf16*>(q16), g, g.Hq) ||      // (same element size and layout)
              !make_cube_tmap(&tk16, reinterpret_cast<const bf16*>(k16), g, g.Hkv)))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  int* flag = &status->pad[kRangeFlagSlot];
  Bwd128Args a{&status->pad[2], lse, delta, row_ptr, col_idx, dqc, nullptr, dq, nullptr, status, flag, 0};
  const int total = g.batch * g.Hq * (g.N / 2);
  const int grid = total < sms ? total : sms;
  const bool split = !(g.flags & VSA2_FLAG_FAST_BWD);
  if (f16) {
    // the copy, the fp16 form, and the pair form that runs only if the range flag came up (see launch_fine_bwd_dq_tc)
    if ((e = launch_cast_bf16_to_f16(q, q16, (size_t)g.batch * g.Hq * g.S * g.D, k, k16, (size_t)g.batch * g.Hkv * g.S * g.D, flag,
                                     st)) != cudaSuccess)
      return e;
    a.when = 1;
    e = g.D == 128 ? launch_bwd128<128, 0, false, true>(tq16, tdo, tk16, tv, g, a, grid, st)
                   : launch_bwd128<64, 0, false, true>(tq16, tdo, tk16, tv, g, a, grid, st);
    if (e != cudaSuccess) return e;
    a.when = 2;
    a.item_counter = &status->pad[kRangeFlagSlot + 1];
    return g.D == 128 ? launch_bwd128<128, 0, true>(tq, tdo, tk, tv, g, a, grid, st) : launch_bwd128<64, 0, true>(tq, tdo, tk, tv, g, a, grid, st);
  }
  if (g.D == 128) return split ? launch_bwd128<128, 0, true>(tq, tdo, tk, tv, g, a, grid, st) : launch_bwd128<128, 0, false>(tq, tdo, tk, tv, g, a, grid, st);
  return split ? launch_bwd128<64, 0, true>(tq, tdo, tk, tv, g, a, grid, st) : launch_bwd128<64, 0, false>(tq, tdo, tk, tv, g, a, grid, st);
}

// dK/dV pass: col_ptr / row_idx is the transposed map expanded to 64-token blocks
cudaError_t launch_fine_bwd128_dkv_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                      const float* lse, const float* delta, const int* col_ptr, const int* row_idx,
                                      const float* dkc, const float* dvc, void* dk, void* dv, StatusBlock* status,
                                      cudaStream_t st, const void* q16, const void* k16) {
  if (!fine_bwd128_supported(g)) return cudaErrorInvalidValue;
  // `q16`, `k16`: null, or the fp16 copies of Q and K that the dQ pass of the same call has made (and whose range flag it has
  // settled): the pass then runs in its fp16 form, with the bf16 form behind the flag
  const bool f16 = fine_bwd_dq_uses_f16(g) && q16 != nullptr && k16 != nullptr;
  CUtensorMap tq, tk, tv, tdo, tq16, tk16;
  if (!make_cube_tmap(&tq, q, g, g.Hq) || !make_cube_tmap(&tk, k, g, g.Hkv) || !make_cube_tmap(&tv, v, g, g.Hkv) ||
      !make_cube_tmap(&tdo, d_o, g, g.Hq))
    return cudaErrorInvalidValue;
  if (f16 && (!make_cube_tmap(&tq16, reinterpret_cast<const bf16*>(q16), g, g.Hq) ||
              !make_cube_tmap(&tk16, reinterpret_cast<const bf16*>(k16), g, g.Hkv)))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  Bwd128Args a{&status->pad[3], lse, delta, col_ptr, row_idx, dkc, dvc, dk, dv, status, &status->pad[kRangeFlagSlot], 0};
  const int total = g.batch * g.Hkv * (g.N / 2);
  const int grid = total < sms ? total : sms;
  const bool split = fine_bwd_dkv_wants_pair(g);
  if (split) return cudaErrorInvalidValue;      // (the caller takes the 64-token kernels for that)
  if (f16) {
    a.when = 1;
    e = g.D == 128 ? launch_bwd128<128, 1, false, true>(tk16, tv, tq16, tdo, g, a, grid, st)
                   : launch_bwd128<64, 1, false, true>(tk16, tv, tq16, tdo, g, a, grid, st);
    if (e != cudaSuccess) return e;
    a.when = 2;
    a.item_counter = &status->pad[5];
  }
  if (g.D == 128) return launch_bwd128<128, 1, false>(tk, tv, tq, tdo, g, a, grid, st);
  return launch_bwd128<64, 1, false>(tk, tv, tq, tdo, g, a, grid, st);
}

}  // namespace vsa2
