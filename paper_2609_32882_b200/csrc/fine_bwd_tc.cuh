// Shared pieces of the two backward passes of the fine branch (fine_bwd_tc.cu: dQ pass, fine_bwd_dkv_tc.cu: dK/dV pass):
// shared-memory plan, barriers, the ring producer.
#pragma once
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kDqThreads = 416;    // dQ pass: 4 service warps, 2 x 4 elementwise warps, 1 more issuer warp
constexpr int kDkvThreads = 576;   // dK/dV pass: 4 service warps, 2 x 4 elementwise warps, 4 row-statistics warps, 2 issuer warps
constexpr int kRingA = 3;          // slots of the ring whose tiles are also an operand of the last product of a tile
constexpr int kRingB = 2;          // (the ring-B slot of a tile is also the index of its tensor-memory buffers)
static_assert(kRingB == 2, "ring B shares its slot index with the two accumulator buffers");

// Shared-memory plan of both passes (D = 128: 5 x 32 KB ring slots, 2 x 16 KB stationary tiles, 2 x 16 KB operand
// buffers, 2 KB of barriers and per-block vectors: exactly the 227 KB a block may use).  Ring A has 3 slots, ring B 2;
// each ring has one producing warp and fixed consuming roles.
// RA: slots of ring A; NP: 16 KB operand buffers (the dK/dV pass in its split mode trades one ring-A slot for the two
// buffers that hold the low-order parts of P and dS).
template <int D, int RA = kRingA, int NP = 2>
struct BwdTc {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLOT = 2 * DH * kSlab;   // a pair of cube tiles, [half][A | B]
  static constexpr uint32_t TILE = DH * kSlab;       // one cube tile, [half]
  static constexpr uint32_t PBYTES = 128 * 128;      // 128 rows x 64 bf16
  static constexpr uint32_t OFF_RING_B = RA * SLOT;
  static constexpr uint32_t OFF_ST0 = (RA + kRingB) * SLOT;       // stationary tile 0 (Q or K)
  static constexpr uint32_t OFF_ST1 = OFF_ST0 + TILE;             // stationary tile 1 (dO or V)
  static constexpr uint32_t OFF_P = OFF_ST1 + TILE;               // the 16 KB operand buffers
  static constexpr uint32_t OFF_MISC = OFF_P + NP * PBYTES;
  static constexpr uint32_t MISC_BYTES = 2048;
  static constexpr size_t smem_bytes = OFF_MISC + MISC_BYTES + 1024;
};

struct BwdMisc {
  uint64_t st_full, st_empty, o_full, o_empty;
  uint64_t a_full[kRingA], a_empty[kRingA], b_full[kRingB], b_empty[kRingB];
  uint64_t s_full[2], s_free[2], dp_full[2], dp_free[2];   // the two score / dP accumulators in tensor memory
  uint64_t p_ready, p_free;                                 // dK/dV pass: the P operand buffer
  uint64_t ds_ready[2], ds_free[2];                         // dS operand buffers (the dK/dV pass has one)
  uint64_t stat_full, stat_free;                            // dK/dV pass: the per-row statistics of a tile
  ItemQueue items;                                          // work items of this CTA (see tc_attn.cuh)
  uint64_t e_sync;                                          // group barrier of the 256 elementwise threads
  uint32_t tmem_base;
  int abort_flag;
  unsigned char edge[kRingA][2];   // dQ pass: edge flags of the two key cubes in each ring-A slot (written by its producer)
  // dQ pass: lse2[tb][c] = stats[tb * 64 + c], delta[tb][c] = stats[128 + tb * 64 + c]: per query column of the item with
  // parity tb, lse * log2(e) (+inf for padding) and delta.  dK/dV pass: (lse * log2(e), delta) of the 128 query rows of
  // the current tile, interleaved.
  alignas(16) float stats[256];
  int tok[2][64];
};
static_assert(sizeof(BwdMisc) <= 2048, "misc region too small");

__device__ __forceinline__ void bwd_init_barriers(BwdMisc* misc) {
  misc->abort_flag = 0;
  tc::mbar_init(&misc->st_full, 1);
  tc::mbar_init(&misc->st_empty, 2);     // both first-stage issuers
  tc::mbar_init(&misc->o_full, 1);       // re-initialised to 2 by the dK/dV pass (two last-stage issuers)
  tc::mbar_init(&misc->o_empty, 256);
  for (int s = 0; s < kRingA; ++s) {
    tc::mbar_init(&misc->a_full[s], 1);
    tc::mbar_init(&misc->a_empty[s], 1);
  }
  for (int s = 0; s < kRingB; ++s) {
    tc::mbar_init(&misc->b_full[s], 1);
    tc::mbar_init(&misc->b_empty[s], 1);
  }
  for (int s = 0; s < 2; ++s) {
    tc::mbar_init(&misc->s_full[s], 1);
    tc::mbar_init(&misc->s_free[s], 256);
    tc::mbar_init(&misc->dp_full[s], 1);
    tc::mbar_init(&misc->dp_free[s], 256);
    tc::mbar_init(&misc->ds_ready[s], 256);
    tc::mbar_init(&misc->ds_free[s], 1);
  }
  tc::mbar_init(&misc->p_ready, 256);
  tc::mbar_init(&misc->e_sync, 256);
  tc::mbar_init(&misc->p_free, 1);
  tc::mbar_init(&misc->stat_full, 128);
  tc::mbar_init(&misc->stat_free, 256);
}

// One warp streams pairs of cube tiles into a ring of NS slots: lane 0 owns the barriers, lanes 0 .. 2*DH-1 issue one
// box each (half h = lane / 2 of block lane & 1).  C3, C2, C1: box coordinates of this lane's block in map TMAP, `bh`: its head.
// `LANE0_PRE`: statement lane 0 runs once the slot is free, before the loads are armed (may use slot_).
#define VSA2_RING_LOAD(FULL, EMPTY, NS, RING_BASE, TMAP, SEQ, CT, CH, CW, BH, LANE0_PRE, WAITFN)                  \
  do {                                                                                                            \
    const uint32_t slot_ = (SEQ) % (NS), par_ = ((SEQ) / (NS)) & 1;                                               \
    int ok_ = 1;                                                                                                  \
    if (lane == 0) {                                                                                              \
      ok_ = tc::WAITFN(&(EMPTY)[slot_], par_ ^ 1, &misc->abort_flag);                                             \
      if (ok_) {                                                                                                  \
        LANE0_PRE;                                                                                                \
        tc::mbar_expect_tx(&(FULL)[slot_], C::SLOT);                                                              \
      }                                                                                                           \
    }                                                                                                             \
    if (!__shfl_sync(0xffffffffu, ok_, 0)) goto done;                                                             \
    if (lane < 2 * C::DH)                                                                                         \
      tc::tma_load_5d((RING_BASE) + slot_ * C::SLOT + (2 * (lane >> 1) + (lane & 1)) * kSlab, (TMAP), &(FULL)[slot_], \
                      (lane >> 1) * 64, (CW), (CH), (CT), (BH));                                                  \
  } while (0)

static inline cudaError_t bwd_sm_count(int* sms) {
  int dev = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  return cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
}

}  // namespace vsa2
