// Fine branch forward (paper Eq. 12) + gated merge (Eq. 14) on the Blackwell tensor cores.
//
// Formulation.  A query block has only B = 64 tokens, half of the 128 rows a tcgen05 MMA wants, so the
// products are taken transposed and two selected KV blocks are stacked per tile:
//     S^T [128 kv, 64 q] = K_pair [128, D] * Q^T          (M = 128 keys,      N = 64 queries, K = D)
//     O^T [D,      64 q] += V_pair^T [D, 128] * P^T       (M = D channels,    N = 64 queries, K = 128 keys)
// K and V tiles arrive by 5-D TMA straight from the raster tensors (one box = one cube, zero-filled outside
// the grid) into 128-byte-swizzled shared memory; the same V tile that TMA wrote row-per-key is read as an
// MN-major operand, so nothing is transposed in memory.  Accumulators live in tensor memory: two S^T
// buffers (64 columns each) and O^T (64 columns).
//
// Softmax.  One thread owns one key row of S^T, so a query's maximum would need a reduction across 128
// threads per tile.  Instead each query column keeps a fixed reference M (the exact column maximum of the
// first tile, in log2 units): P = 2^(s*scale*log2e - M).  Any reference gives the same softmax as long as
// nothing overflows; the row sums are checked at the end of the query block and a block whose sums left
// the safe range is recomputed by the exact-maximum kernel (see fine_fwd.cu).  Row sums are accumulated per
// thread and reduced across the 128 key rows once per query block, deterministically.
//
// Roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (one elected lane each), warps 2..5 =
// softmax + epilogue (each owns the tensor-memory lane quadrant warp % 4).  Every wait is bounded.
#include "tc_attn.cuh"

namespace vsa2 {

constexpr int kFwdThreads = 192;
constexpr int kFwdSlots = 5;
constexpr int kRescueCap = 16384;

template <int D>
struct FwdTc {
  static constexpr int DH = D / 64;
  static constexpr uint32_t SLAB = 8192;             // one cube x 64 channels
  static constexpr uint32_t SLOT = 2 * DH * SLAB;    // a K pair or a V pair
  static constexpr uint32_t QBYTES = DH * SLAB;
  static constexpr uint32_t PBYTES = 128 * 128;      // P^T: 128 key rows x 64 queries bf16
  static constexpr uint32_t OFF_Q = kFwdSlots * SLOT;
  static constexpr uint32_t OFF_P = OFF_Q + QBYTES;
  static constexpr uint32_t OFF_MISC = OFF_P + 2 * PBYTES;
  static constexpr uint32_t MISC_BYTES = 4096;
  static constexpr size_t smem_bytes = OFF_MISC + MISC_BYTES + 1024;
};

struct FwdMisc {
  uint64_t q_full, q_empty, o_full, o_empty;
  uint64_t kv_full[kFwdSlots], kv_empty[kFwdSlots];
  uint64_t s_full[2], p_ready[2], p_free[2];
  uint32_t tmem_base;
  int abort_flag;
  int rescue_flag;
  float m_ref[64];          // per query column: reference exponent (log2 units)
  float l_inv[64];
  int tok[2][64];           // raster token of each query position (-1 = padding), by item parity
  float gate[2][64];
};

struct FwdArgs {
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
};

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
  float* scratch = reinterpret_cast<float*>(p_tile);     // 32 KB, reused for the cross-row reductions

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_items = g.batch * g.Hq * g.N;
  const float c2 = g.scale * 1.4426950408889634f;

  if (tid == 0) {
    misc->abort_flag = 0;
    tc::mbar_init(&misc->q_full, 1);
    tc::mbar_init(&misc->q_empty, 1);
    tc::mbar_init(&misc->o_full, 1);
    tc::mbar_init(&misc->o_empty, 128);
    for (int s = 0; s < kFwdSlots; ++s) {
      tc::mbar_init(&misc->kv_full[s], 1);
      tc::mbar_init(&misc->kv_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(&misc->s_full[s], 1);
      tc::mbar_init(&misc->p_ready[s], 128);
      tc::mbar_init(&misc->p_free[s], 1);
    }
    tc::fence_barrier_init();
    tc::prefetch_tmap(&tm_q);
    tc::prefetch_tmap(&tm_k);
    tc::prefetch_tmap(&tm_v);
  }
  if (warp == 1) {
    tc::tmem_alloc(&misc->tmem_base, 256);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
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
        VSA2_WAIT(&misc->q_empty, (n_items & 1) ^ 1);
        tc::mbar_expect_tx(&misc->q_full, C::QBYTES);
        for (int h = 0; h < C::DH; ++h)
          tc::tma_load_5d(q_tile + h * C::SLAB, &tm_q, &misc->q_full, h * 64, iw_ * g.Bw, ih_ * g.Bh, it_ * g.Bt, bhq);
        ++n_items;
        const int nt = (k + 1) >> 1;
        for (int t = 0; t < nt; ++t) {
          const int ja = cols[2 * t], jb = (2 * t + 1 < k) ? cols[2 * t + 1] : ja;
          int at, ah, aw, bt, bh_, bw;
          cube_coords(g, ja, at, ah, aw);
          cube_coords(g, jb, bt, bh_, bw);
          {  // K pair: [half][A | B]
            const uint32_t slot = seq % kFwdSlots, par = (seq / kFwdSlots) & 1;
            unsigned char* dst = smem + slot * C::SLOT;
            VSA2_WAIT(&misc->kv_empty[slot], par ^ 1);
            tc::mbar_expect_tx(&misc->kv_full[slot], C::SLOT);
            for (int h = 0; h < C::DH; ++h) {
              tc::tma_load_5d(dst + (2 * h + 0) * C::SLAB, &tm_k, &misc->kv_full[slot], h * 64, aw * g.Bw, ah * g.Bh, at * g.Bt, bhk);
              tc::tma_load_5d(dst + (2 * h + 1) * C::SLAB, &tm_k, &misc->kv_full[slot], h * 64, bw * g.Bw, bh_ * g.Bh, bt * g.Bt, bhk);
            }
            ++seq;
          }
          {  // V pair: [A half0 .. | B half0 ..]
            const uint32_t slot = seq % kFwdSlots, par = (seq / kFwdSlots) & 1;
            unsigned char* dst = smem + slot * C::SLOT;
            VSA2_WAIT(&misc->kv_empty[slot], par ^ 1);
            tc::mbar_expect_tx(&misc->kv_full[slot], C::SLOT);
            for (int h = 0; h < C::DH; ++h) {
              tc::tma_load_5d(dst + (0 * C::DH + h) * C::SLAB, &tm_v, &misc->kv_full[slot], h * 64, aw * g.Bw, ah * g.Bh, at * g.Bt, bhk);
              tc::tma_load_5d(dst + (1 * C::DH + h) * C::SLAB, &tm_v, &misc->kv_full[slot], h * 64, bw * g.Bw, bh_ * g.Bh, bt * g.Bt, bhk);
            }
            ++seq;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = tc::idesc_bf16(128, 64, false, false);
      constexpr uint32_t idesc_o = tc::idesc_bf16(128, 64, true, true);
      const uint32_t q_addr = tc::smem_u32(q_tile), p_addr = tc::smem_u32(p_tile), slot0 = tc::smem_u32(smem);
      const uint32_t tm_o = tmem_base + 128;
      uint32_t seq_k = 0;       // ring sequence number of the next K pair (its V pair is seq_k + 1)
      uint32_t tt = 0;          // tiles issued so far (S buffer = tt & 1)
      uint32_t n_items = 0;
      for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const int i = item % g.N, bhq = item / g.N;
        const int beg = a.row_ptr[(size_t)bhq * (g.N + 1) + i], end = a.row_ptr[(size_t)bhq * (g.N + 1) + i + 1];
        const int k = end - beg;
        if (k == 0) continue;
        const int nt = (k + 1) >> 1;
        VSA2_WAIT(&misc->q_full, n_items & 1);
        tc::tc_fence_after();
        for (int t = 0; t <= nt; ++t) {
          if (t < nt) {   // S^T(t) = K_pair * Q^T
            const uint32_t seq = seq_k + 2 * t, slot = seq % kFwdSlots, par = (seq / kFwdSlots) & 1;
            VSA2_WAIT(&misc->kv_full[slot], par);
            tc::tc_fence_after();
            const uint32_t k_addr = slot0 + slot * C::SLOT, tm_s = tmem_base + ((tt + t) & 1) * 64;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint32_t aa = k_addr + (ks / 4) * 2 * C::SLAB + (ks % 4) * 32;
              const uint32_t bb = q_addr + (ks / 4) * C::SLAB + (ks % 4) * 32;
              tc::mma_ss(tm_s, tc::smem_desc_sw128(aa, 16, 1024), tc::smem_desc_sw128(bb, 16, 1024), idesc_s, ks > 0);
            }
            tc::mma_commit(&misc->s_full[(tt + t) & 1]);
            tc::mma_commit(&misc->kv_empty[slot]);
            if (t == nt - 1) tc::mma_commit(&misc->q_empty);
          }
          if (t >= 1) {   // O^T += V_pair^T * P^T for tile t - 1
            const uint32_t tp = tt + t - 1, buf = tp & 1;
            const uint32_t seq = seq_k + 2 * (t - 1) + 1, slot = seq % kFwdSlots, par = (seq / kFwdSlots) & 1;
            VSA2_WAIT(&misc->p_ready[buf], (tp >> 1) & 1);
            VSA2_WAIT(&misc->kv_full[slot], par);
            if (t == 1) VSA2_WAIT(&misc->o_empty, (n_items & 1) ^ 1);
            tc::tc_fence_after();
            const uint32_t v_addr = slot0 + slot * C::SLOT;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t aa = v_addr + (ks / 4) * C::DH * C::SLAB + (ks % 4) * 2048;
              const uint32_t bb = p_addr + buf * C::PBYTES + ks * 2048;
              tc::mma_ss(tm_o, tc::smem_desc_sw128(aa, C::DH == 2 ? C::SLAB : 0, 1024), tc::smem_desc_sw128(bb, 0, 1024),
                         idesc_o, (t > 1) || (ks > 0));
            }
            tc::mma_commit(&misc->kv_empty[slot]);
            tc::mma_commit(&misc->p_free[buf]);
            if (t == nt) tc::mma_commit(&misc->o_full);
          }
        }
        seq_k += 2 * nt;
        tt += nt;
        ++n_items;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (128 threads)
    const int quad = warp & 3;
    const int row = (quad << 5) | lane;          // tensor-memory lane: key row in S^T, channel in O^T
    const int sm_tid = tid - 64;                 // 0..127 inside this group
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && a.gate != nullptr;
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
        misc->gate[tb][sm_tid] = (coarse && l >= 0) ? a.gate[(size_t)bhq * g.L + l] : 0.f;
      }
      const float oc_d = (coarse && row < D) ? a.oc_hat[((size_t)bhq * g.N + i) * D + row] : 0.f;
      if (sm_tid == 0) misc->rescue_flag = 0;
      tc::named_bar_sync(1, 128);

      if (k == 0) {
        // no selected block: O = gate * O_c, lse = -inf
        if (row < D) {
          for (int qi = 0; qi < 64; ++qi) {
            const int l = misc->tok[tb][qi];
            if (l < 0) continue;
            const size_t idx = ((size_t)bhq * g.L + l) * D + row;
            const float val = misc->gate[tb][qi] * oc_d;
            store_out(a.o, idx, val, g.out_f32);
            if (a.o_res != nullptr) a.o_res[idx] = __float2bfloat16_rn(val - __bfloat162float(__float2bfloat16_rn(val)));
          }
        }
        if (sm_tid < 64 && misc->tok[tb][sm_tid] >= 0) a.lse[(size_t)bhq * g.L + misc->tok[tb][sm_tid]] = -INFINITY;
        continue;
      }

      float l_part[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) l_part[c] = 0.f;
      const int nt = (k + 1) >> 1;
      for (int t = 0; t < nt; ++t, ++tt) {
        const uint32_t buf = tt & 1, use = (tt >> 1) & 1;
        // validity of this thread's key row
        const int blk = row >> 6;
        const bool dup = (blk == 1) && (2 * t + 1 >= k);
        const int j = cols[dup ? 2 * t : 2 * t + blk];
        const bool valid = !dup && pos_valid(g, j, row & 63);
        VSA2_WAIT(&misc->s_full[buf], use);
        tc::tc_fence_after();
        uint32_t s0[32], s1[32];
        tc::tmem_ld32(lane_addr + buf * 64, s0);
        tc::tmem_ld32(lane_addr + buf * 64 + 32, s1);
        tc::tmem_ld_wait();
        if (t == 0) {
          // reference exponent of every query column = exact column maximum of the first tile
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            scratch[scratch_idx(sm_tid, c)] = valid ? __uint_as_float(s0[c]) : -INFINITY;
            scratch[scratch_idx(sm_tid, c + 32)] = valid ? __uint_as_float(s1[c]) : -INFINITY;
          }
          tc::named_bar_sync(1, 128);
          if (sm_tid < 64) {
            float mx = -INFINITY;
            for (int r = 0; r < 128; ++r) mx = fmaxf(mx, scratch[scratch_idx(r, sm_tid)]);
            misc->m_ref[sm_tid] = (mx > -INFINITY) ? mx * c2 : 0.f;
          }
          tc::named_bar_sync(1, 128);
        }
        VSA2_WAIT(&misc->p_free[buf], use ^ 1);
        uint32_t packed[32];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const float m0 = misc->m_ref[c], m1 = misc->m_ref[c + 1];
          float p0 = ex2_approx(fmaf(__uint_as_float(s0[c]), c2, -m0));
          float p1 = ex2_approx(fmaf(__uint_as_float(s0[c + 1]), c2, -m1));
          p0 = valid ? p0 : 0.f;
          p1 = valid ? p1 : 0.f;
          l_part[c] += p0;
          l_part[c + 1] += p1;
          packed[c >> 1] = pack_bf16x2(p0, p1);
        }
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          const float m0 = misc->m_ref[32 + c], m1 = misc->m_ref[33 + c];
          float p0 = ex2_approx(fmaf(__uint_as_float(s1[c]), c2, -m0));
          float p1 = ex2_approx(fmaf(__uint_as_float(s1[c + 1]), c2, -m1));
          p0 = valid ? p0 : 0.f;
          p1 = valid ? p1 : 0.f;
          l_part[32 + c] += p0;
          l_part[33 + c] += p1;
          packed[16 + (c >> 1)] = pack_bf16x2(p0, p1);
        }
        unsigned char* prow = p_tile + buf * C::PBYTES + row * 128;
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
          *reinterpret_cast<uint4*>(prow + ((ch ^ (row & 7)) << 4)) =
              make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
        tc::fence_proxy_async_smem();
        tc::tc_fence_before();
        tc::mbar_arrive(&misc->p_ready[buf]);
      }

      // ---- epilogue of the query block
      VSA2_WAIT(&misc->o_full, n_items & 1);
      tc::tc_fence_after();
#pragma unroll
      for (int c = 0; c < 64; ++c) scratch[scratch_idx(sm_tid, c)] = l_part[c];
      tc::named_bar_sync(1, 128);
      if (sm_tid < 64) {
        float l = 0.f;
        for (int r = 0; r < 128; ++r) l += scratch[scratch_idx(r, sm_tid)];
        // sums outside the safe range (overflow, NaN or total underflow): hand the block to the exact kernel
        if (!(l > 1e-30f && l < 1e30f)) misc->rescue_flag = 1;
        misc->l_inv[sm_tid] = 1.f / l;
        const int tk = misc->tok[tb][sm_tid];
        if (tk >= 0) a.lse[(size_t)bhq * g.L + tk] = (misc->m_ref[sm_tid] + __log2f(l)) * 0.6931471805599453f;
      }
      tc::named_bar_sync(1, 128);
      {
        uint32_t o0[32], o1[32];
        tc::tmem_ld32(lane_addr + 128, o0);
        tc::tmem_ld32(lane_addr + 128 + 32, o1);
        tc::tmem_ld_wait();
        tc::tc_fence_before();
        tc::mbar_arrive(&misc->o_empty);
        if (row < D) {
#pragma unroll
          for (int qi = 0; qi < 64; ++qi) {
            const int l = misc->tok[tb][qi];
            if (l < 0) continue;
            const float acc = __uint_as_float(qi < 32 ? o0[qi & 31] : o1[qi & 31]);
            const float val = fmaf(misc->gate[tb][qi], oc_d, acc * misc->l_inv[qi]);
            const size_t idx = ((size_t)bhq * g.L + l) * D + row;
            store_out(a.o, idx, val, g.out_f32);
            if (a.o_res != nullptr) a.o_res[idx] = __float2bfloat16_rn(val - __bfloat162float(__float2bfloat16_rn(val)));
          }
        }
      }
      if (sm_tid == 0 && misc->rescue_flag) {
        int slot = atomicAdd(a.rescue_count, 1);
        if (slot < kRescueCap) a.rescue_items[slot] = item;
        else atomicExch(&a.status->status, VSA2_ERR_UNSUPPORTED);
      }
      ++n_items;
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
  if (warp == 1) tc::tmem_dealloc(tmem_base, 256);
}

cudaError_t launch_fine_fwd_list(const Geo& g, const int* count, const int* items, const bf16* q, const bf16* k,
                                 const bf16* v, const float* gate, const int* row_ptr, const int* col_idx,
                                 const float* oc_hat, void* o, bf16* o_res, float* lse, cudaStream_t st);

size_t fine_fwd_tc_workspace_bytes() { return 256 + (size_t)kRescueCap * sizeof(int); }

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
  a.rescue_items = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(status) + 256);
  const int total = g.batch * g.Hq * g.N;
  const int grid = total < sms ? total : sms;
  if (g.D == 128) {
    if ((e = cudaFuncSetAttribute(fine_fwd_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FwdTc<128>::smem_bytes))) return e;
    fine_fwd_tc_kernel<128><<<grid, kFwdThreads, FwdTc<128>::smem_bytes, st>>>(tq, tk, tv, g, a);
  } else {
    if ((e = cudaFuncSetAttribute(fine_fwd_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FwdTc<64>::smem_bytes))) return e;
    fine_fwd_tc_kernel<64><<<grid, kFwdThreads, FwdTc<64>::smem_bytes, st>>>(tq, tk, tv, g, a);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // query blocks whose row sums left the safe range are redone with the exact running maximum
  return launch_fine_fwd_list(g, a.rescue_count, a.rescue_items, q, k, v, gate, row_ptr, col_idx, oc_hat, o, o_res, lse, st);
}

}  // namespace vsa2
