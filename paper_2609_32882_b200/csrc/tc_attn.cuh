// Helpers shared by the tensor-core attention kernels (forward and backward).
#pragma once
#include "common.cuh"
#include "tc05.cuh"
#include "tmap.cuh"

namespace vsa2 {

constexpr uint32_t kSlab = 8192;   // one cube x 64 channels of bf16, 64 rows of 128 bytes, 128-byte swizzled

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// 64 bf16 (32 packed words) -> one 128-byte row of a swizzled operand tile: 16-byte chunk c lands at c ^ (row & 7)
__device__ __forceinline__ void store_row_sw128(unsigned char* tile, int row, const uint32_t (&packed)[32]) {
  unsigned char* prow = tile + row * 128;
#pragma unroll
  for (int ch = 0; ch < 8; ++ch)
    *reinterpret_cast<uint4*>(prow + ((ch ^ (row & 7)) << 4)) =
        make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
}

// Issues the D/16 (K-major x K-major) instructions of  acc[128, 64] = A_pair[128, D] * B[64, D]^T.
// A_pair: slot laid out [half][block A | block B] slabs; B: tile laid out [half] slabs.
// The descriptors are built once and advanced by adding the (16-byte-unit) offset to the address field.
// (F16: both operands hold fp16 instead of bf16)
template <int D, bool F16 = false>
__device__ __forceinline__ void mma_pair_kmajor(uint32_t tm_acc, uint32_t a_slot, uint32_t b_tile) {
  constexpr uint32_t idesc = F16 ? tc::idesc_f16(128, 64, false, false) : tc::idesc_bf16(128, 64, false, false);
  const uint64_t da = tc::smem_desc_sw128(a_slot, 16, 1024), db = tc::smem_desc_sw128(b_tile, 16, 1024);
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const uint64_t oa = (uint64_t)(((ks / 4) * 2 * kSlab + (ks % 4) * 32) >> 4);
    const uint64_t ob = (uint64_t)(((ks / 4) * kSlab + (ks % 4) * 32) >> 4);
    tc::mma_ss(tm_acc, da + oa, db + ob, idesc, ks > 0);
  }
}

// Issues the 8 (MN-major x MN-major) instructions of  acc[D, 64] (+)= A_pair^T[D, 128] * B[128, 64], where A_pair is a
// slot in the [half][block A | block B] layout (rows = the 128 contraction indices) and B is a 128-row swizzled tile.
// `ksteps`: 8, or 4 to contract over the first block of the pair only.
template <int D, bool F16 = false>
__device__ __forceinline__ void mma_pairT_mnmajor(uint32_t tm_acc, uint32_t a_slot, uint32_t b_tile, bool accumulate_first,
                                                  int ksteps = 8) {
  constexpr uint32_t idesc = F16 ? tc::idesc_f16(128, 64, true, true) : tc::idesc_bf16(128, 64, true, true);
  constexpr uint32_t lbo = (D == 128) ? 2 * kSlab : 0;     // distance between the two 64-channel halves
  const uint64_t da = tc::smem_desc_sw128(a_slot, lbo, 1024), db = tc::smem_desc_sw128(b_tile, 0, 1024);
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint64_t oa = (uint64_t)(((ks / 4) * kSlab + (ks % 4) * 2048) >> 4);
    const uint64_t ob = (uint64_t)((ks * 2048) >> 4);
    if (ks < ksteps) tc::mma_ss(tm_acc, da + oa, db + ob, idesc, accumulate_first || (ks > 0));
  }
}

// The same product with 128 columns: B is two 128-row tiles side by side, `b_stride` bytes apart (columns 0..63 from the first,
// 64..127 from the second), acc[D, 128].  Used with B = [X_hi | X_lo], the bf16 rounding of X and the bf16 rounding of what
// that lost: the two column halves of the accumulator then sum to A^T X at about 16 bits of operand precision, for one
// N = 128 instruction (64 cycles) per step instead of two N = 64 instructions (2 x 48).
template <int D>
__device__ __forceinline__ void mma_pairT_mnmajor_n128(uint32_t tm_acc, uint32_t a_slot, uint32_t b_tile, uint32_t b_stride,
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

// fp32 pair -> packed fp16 pair (`lo` in the low half), values beyond the fp16 range clamped to +-65504
__device__ __forceinline__ uint32_t pack_f16x2_sat(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// max(m, |a|, |b|) in one instruction (the three-input maximum of sm_100; the absolute values fold into it)
__device__ __forceinline__ float max3_abs(float m, float a, float b) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(m), "f"(fabsf(a)), "f"(fabsf(b)));
  return r;
}
// fp32 pair -> packed fp16 pair (`lo` in the low half); a value beyond the fp16 range becomes an infinity
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// whether one of 32 accumulator values (float bits) is an infinity or not a number: x * 0 is 0 for every finite x
__device__ __forceinline__ bool any_non_finite32(const uint32_t (&v)[32]) {
  float t = 0.f;
#pragma unroll
  for (int e = 0; e < 32; ++e) t = fmaf(__uint_as_float(v[e]), 0.f, t);
  return t != t;
}
// x -> (bf16(x), bf16(x - bf16(x))) for two values, packed like pack_bf16x2
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16x2(x0, x1);
  const float h0 = __uint_as_float(hi << 16), h1 = __uint_as_float(hi & 0xffff0000u);
  lo = pack_bf16x2(x0 - h0, x1 - h1);
}

__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// Which cubes are cut by the grid boundary: bit 0 / 1 / 2 = last cube along t / h / w with a partial extent.
// In the half-cube grid of a 128-token-cube problem the last column of blocks along w may lie outside the grid
// altogether (extent <= 0, still bit 2); the column before it can then be the partial one (bit 3).
__device__ __forceinline__ unsigned cube_edge_flags_at(const Geo& g, int nt, int nh, int nw) {
  unsigned f = 0;
  if (nt == g.Nt - 1 && g.T % g.Bt) f |= 1u;
  if (nh == g.Nh - 1 && g.H % g.Bh) f |= 2u;
  if ((nw + 1) * g.Bw > g.W) f |= (nw == g.Nw - 1) ? 4u : 8u;
  return f;
}
__device__ __forceinline__ unsigned cube_edge_flags(const Geo& g, int n) {
  int nt, nh, nw;
  cube_coords(g, n, nt, nh, nw);
  return cube_edge_flags_at(g, nt, nh, nw);
}
// The same for a block of the fine kernels: a text block carries bit 7 and, in its low bits, its number of tokens - 1.
constexpr unsigned kTextBlockFlag = 0x80u;
__device__ __forceinline__ unsigned block_edge_flags(const Geo& g, int j) {
  if (j < g.Nvid) return cube_edge_flags(g, j);
  return kTextBlockFlag | (unsigned)(block_count(g, j) - 1);
}

// Position of a token inside its cube and the test "is this position inside the valid grid for a cube with edge flags f".
struct CubePos {
  int bt, bh, bw, lt, lh, lw;   // coordinates of the position; valid extents of the last cube along each axis
  int pos;                      // the position itself (text blocks: row of the block)
  __device__ __forceinline__ void init(const Geo& g, int pos_) {
    pos = pos_;
    bw = pos % g.Bw;
    int r = pos / g.Bw;
    bh = r % g.Bh;
    bt = r / g.Bh;
    lt = g.T - (g.Nt - 1) * g.Bt;
    lh = g.H - (g.Nh - 1) * g.Bh;
    lw = g.W - (g.Nw - 1) * g.Bw;
  }
  __device__ __forceinline__ bool valid(unsigned f, const Geo& g) const {
    if (f & kTextBlockFlag) return pos <= (int)(f & 0x7fu);
    return (!(f & 1u) || bt < lt) && (!(f & 2u) || bh < lh) && (!(f & 4u) || bw < lw) && (!(f & 8u) || bw < lw + g.Bw);
  }
};

// Column reduction of a 64-wide per-lane vector over the 32 lanes of a warp ("transpose reduce", 62 shuffles):
// afterwards v[0], v[1] hold the reduction over all lanes of columns warp_reduce_col(lane) and warp_reduce_col(lane) + 1.
// The order of the operations is fixed, so sums are reproducible.
template <bool IS_MAX>
__device__ __forceinline__ void warp_reduce_cols64(float (&v)[64], int lane) {
#pragma unroll
  for (int n = 32, off = 16; off >= 1; n >>= 1, off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n; ++i) {
      const float send = upper ? v[i] : v[i + n];
      const float keep = upper ? v[i + n] : v[i];
      const float recv = __shfl_xor_sync(0xffffffffu, send, off);
      v[i] = IS_MAX ? fmaxf(keep, recv) : keep + recv;
    }
  }
}
// The same for a 32-wide vector (31 shuffles): afterwards v[0] holds the reduction over all lanes of column `lane`.
template <bool IS_MAX>
__device__ __forceinline__ void warp_reduce_cols32(float (&v)[32], int lane) {
#pragma unroll
  for (int n = 16, off = 16; off >= 1; n >>= 1, off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n; ++i) {
      const float send = upper ? v[i] : v[i + n];
      const float keep = upper ? v[i + n] : v[i];
      const float recv = __shfl_xor_sync(0xffffffffu, send, off);
      v[i] = IS_MAX ? fmaxf(keep, recv) : keep + recv;
    }
  }
}
__device__ __forceinline__ int warp_reduce_col(int lane) {
  return ((lane >> 4) & 1) * 32 + ((lane >> 3) & 1) * 16 + ((lane >> 2) & 1) * 8 + ((lane >> 1) & 1) * 4 + (lane & 1) * 2;
}

// ------------------------------------------------------------------------------------------------
// Work queue of a persistent CTA.  Work items (query blocks or KV blocks) have very different list lengths, so a static
// round-robin split leaves some CTAs with up to 15 % more tiles than the average.  One thread of the CTA (the
// scheduler) draws item numbers from a global counter, a few items ahead, and publishes them through a small ring in
// shared memory; every role of the CTA reads the same sequence from the ring.  All CTAs therefore advance through the
// item sequence together (neighbouring items share operand tiles in L2) and finish together.  Item -1 ends the CTA.
constexpr int kItemSlots = 4;       // ring depth
constexpr int kItemAhead = 2;       // items published ahead of the scheduler's own position
struct ItemQueue {
  uint64_t full[kItemSlots], empty[kItemSlots];
  int item[kItemSlots];
};
// `consumers`: threads that call item_get for every sequence number (the scheduler thread included)
__device__ __forceinline__ void item_queue_init(ItemQueue* q, int consumers) {
  for (int s = 0; s < kItemSlots; ++s) {
    tc::mbar_init(&q->full[s], 1);
    tc::mbar_init(&q->empty[s], consumers);
  }
}
// scheduler: publishes every sequence number up to seq + kItemAhead that is not out yet; false on a timed-out wait
__device__ __forceinline__ bool item_publish_ahead(ItemQueue* q, uint32_t seq, uint32_t& published, int* counter, int total,
                                                   volatile int* abort_flag) {
  while (published <= seq + kItemAhead) {
    const uint32_t slot = published % kItemSlots, par = ((published / kItemSlots) & 1) ^ 1;
    if (!tc::mbar_wait_parked(&q->empty[slot], par, abort_flag)) return false;
    const int it = atomicAdd(counter, 1);
    q->item[slot] = it < total ? it : -1;
    tc::mbar_arrive(&q->full[slot]);
    ++published;
  }
  return true;
}
// consumer: item of sequence number seq, or -2 if the wait timed out
__device__ __forceinline__ int item_get(ItemQueue* q, uint32_t seq, volatile int* abort_flag) {
  const uint32_t slot = seq % kItemSlots, par = (seq / kItemSlots) & 1;
  if (!tc::mbar_wait_parked(&q->full[slot], par, abort_flag)) return -2;
  const int it = q->item[slot];
  tc::mbar_arrive(&q->empty[slot]);
  return it;
}
// loop header of a role whose threads all call it: `for (uint32_t seq = 0;; ++seq) { VSA2_NEXT_ITEM(item, seq); ... }`
#define VSA2_NEXT_ITEM(ITEM, SEQ)                                  \
  const int ITEM = item_get(&misc->items, (SEQ), &misc->abort_flag); \
  if (ITEM == -2) goto done;                                       \
  if (ITEM < 0) break

// the same for a role whose whole warp runs the loop (lane 0 takes the item, the others receive it by shuffle)
#define VSA2_NEXT_ITEM_WARP(ITEM, SEQ)                                     \
  int ITEM = 0;                                                            \
  if (lane == 0) ITEM = item_get(&misc->items, (SEQ), &misc->abort_flag);  \
  ITEM = __shfl_sync(0xffffffffu, ITEM, 0);                                \
  if (ITEM == -2) goto done;                                               \
  if (ITEM < 0) break

#define VSA2_WAIT(bar, parity)                                         \
  do {                                                                 \
    if (!tc::mbar_wait((bar), (parity), &misc->abort_flag)) goto done; \
  } while (0)
// Barrier among a fixed group of threads, built on an mbarrier (arrival count = size of the group) so that its wait is
// bounded like every other wait of these kernels: a thread parked in bar.sync could never leave once a partner had
// given up after a timed-out wait.  PHASE is a per-thread counter of the syncs done on that barrier.
#define VSA2_GROUP_SYNC(bar, PHASE)                \
  do {                                             \
    tc::mbar_arrive(bar);                          \
    VSA2_WAIT((bar), (PHASE) & 1u);                \
    ++(PHASE);                                     \
  } while (0)
// The same with the index of the sync (0, 1, 2, ... on that barrier) computed by the caller instead of counted.
#define VSA2_GROUP_SYNC_AT(bar, INDEX)             \
  do {                                             \
    tc::mbar_arrive(bar);                          \
    VSA2_WAIT((bar), (INDEX) & 1u);                \
  } while (0)

#define VSA2_WAIT_PARKED(bar, parity)                                         \
  do {                                                                        \
    if (!tc::mbar_wait_parked((bar), (parity), &misc->abort_flag)) goto done; \
  } while (0)

}  // namespace vsa2
