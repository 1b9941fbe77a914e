// Gate projection of the gated merge (paper Eq. 13): gate = tanh(X W_g), one column of W_g per query head, and its
// backward.  X [batch, L, C] are the layer's hidden states (bf16, tokens in raster order), W_g [C, Hq] bf16, gate and
// dgate [batch, Hq, L] fp32 (the layout vsa2_attn_fwd / vsa2_attn_bwd use).
//
// All three kernels are bound by one pass over X or dX (2 L C bytes per batch entry against 2 L C Hq FLOP with Hq a few
// dozen), so they are written for wide, coalesced HBM access; the products run on mma.sync m16n8k16 (bf16 in, fp32
// accumulate) because the N or K extent (the heads) is far below a tcgen05 tile.
//   forward : gate^T[l, h] = tanh(sum_c X[l, c] W[c, h])                        M = tokens,  N = heads,    K = channels
//   dX      : dX[l, c]     = sum_h dz[l, h] W[c, h],  dz = dgate (1 - gate^2)   M = tokens,  N = channels, K = heads
//   dW_g    : dW[c, h]     = sum_{b, l} X[l, c] dz[l, h]                        M = channels, N = heads,   K = tokens
// dW_g is reduced over the tokens in two deterministic steps (per-split partial sums, then a sum over the splits in a
// fixed order): no floating-point atomics.
#include "common.cuh"

namespace vsa2 {

namespace {

constexpr int kGtTok = 64;        // tokens per CTA tile
constexpr int kGtCh = 128;        // channels per chunk
constexpr int kGtThreads = 128;   // four warps
constexpr int kGtSplits = 16;     // token ranges per batch entry in the dW_g pass
constexpr int kDxCh = 64;         // channels per chunk of the dX pass (its fp32 staging tile has to fit beside the operands)

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(smem_row)));
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t& r0, uint32_t& r1, const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
               : "=r"(r0), "=r"(r1)
               : "r"((uint32_t)__cvta_generic_to_shared(smem_row)));
}
__device__ __forceinline__ uint32_t lds32(const bf16* p) { return *reinterpret_cast<const uint32_t*>(p); }

// X tile: rows l0 .. l0 + 63 of one batch entry, channels c0 .. c0 + 127 -> xs[64][LDX] (zero outside L x C)
constexpr int kLdx = kGtCh + 8;   // 272-byte rows: 16-byte aligned, and eight consecutive rows cover all 32 banks
__device__ __forceinline__ void load_x_tile(bf16* xs, const bf16* x, int l0, int L, int c0, int C) {
  for (int e = threadIdx.x; e < kGtTok * (kGtCh / 8); e += kGtThreads) {
    const int r = e / (kGtCh / 8), ch = e % (kGtCh / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (l0 + r < L && c0 + ch * 8 < C) v = __ldg(reinterpret_cast<const uint4*>(x + (size_t)(l0 + r) * C + c0 + ch * 8));
    *reinterpret_cast<uint4*>(xs + r * kLdx + ch * 8) = v;
  }
}

// dz = dgate (1 - gate^2) in bf16, once per backward, in the two layouts its products read:
//   dz_hm [batch][HP][Lp]  head-major  (HP = heads rounded up to 16, Lp = tokens rounded up to 64; zero padding)
//   dz_tm [batch][Lp][HP]  token-major
// grid (Lp / 64, batch)
__global__ void __launch_bounds__(kGtThreads) gate_dz_kernel(const float* __restrict__ gate, const float* __restrict__ dgate,
                                                             int L, int Lp, int Hq, int HP, bf16* __restrict__ dz_hm,
                                                             bf16* __restrict__ dz_tm) {
  extern __shared__ __align__(16) unsigned char gate_dz_smem[];
  bf16* tile = reinterpret_cast<bf16*>(gate_dz_smem);          // [HP][64 + 8]
  constexpr int LD = kGtTok + 8;
  const int l0 = blockIdx.x * kGtTok, b = blockIdx.y;
  const float* gb = gate + (size_t)b * Hq * L;
  const float* db = dgate + (size_t)b * Hq * L;
  for (int e = threadIdx.x; e < HP * kGtTok; e += kGtThreads) {
    const int h = e / kGtTok, tl = e % kGtTok;
    float v = 0.f;
    if (h < Hq && l0 + tl < L) {
      const float g = gb[(size_t)h * L + l0 + tl];
      v = db[(size_t)h * L + l0 + tl] * (1.f - g * g);
    }
    const bf16 vb = __float2bfloat16_rn(v);
    tile[h * LD + tl] = vb;
    dz_hm[((size_t)b * HP + h) * Lp + l0 + tl] = vb;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < kGtTok * HP; e += kGtThreads) {
    const int tl = e / HP, h = e % HP;
    dz_tm[((size_t)b * Lp + l0 + tl) * HP + h] = tile[h * LD + tl];
  }
}

// ---------------------------------------------------------------------------------------------- forward
// grid (ceil(L / 64), batch); NT = head tiles of 8
template <int NT>
__global__ void __launch_bounds__(kGtThreads) gate_fwd_kernel(const bf16* __restrict__ x, const bf16* __restrict__ w, int L,
                                                              int C, int Hq, float* __restrict__ gate) {
  constexpr int LDW = NT * 8 + 8;                           // 16-byte aligned rows, eight rows on different banks
  __shared__ __align__(16) bf16 xs[kGtTok * kLdx];
  __shared__ __align__(16) bf16 ws[kGtCh * LDW];            // W chunk as stored: [channel][head]; read by ldmatrix.trans
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int l0 = blockIdx.x * kGtTok, b = blockIdx.y;
  const bf16* xb = x + (size_t)b * L * C;
  const bool w_vec = Hq % 8 == 0 && (reinterpret_cast<uintptr_t>(w) & 15u) == 0;
  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  for (int c0 = 0; c0 < C; c0 += kGtCh) {
    __syncthreads();
    load_x_tile(xs, xb, l0, L, c0, C);
    if (w_vec && c0 + kGtCh <= C) {
      // rows of W are whole 16-byte vectors and the chunk is contiguous: copy as such, then clear the padding heads
      const int vec = Hq / 8;
      const uint4* src = reinterpret_cast<const uint4*>(w + (size_t)c0 * Hq);
      for (int e = threadIdx.x; e < kGtCh * vec; e += kGtThreads)
        *reinterpret_cast<uint4*>(ws + (e / vec) * LDW + (e % vec) * 8) = __ldg(src + e);
      for (int e = threadIdx.x; e < kGtCh * (NT * 8 - Hq); e += kGtThreads)
        ws[(e / (NT * 8 - Hq)) * LDW + Hq + e % (NT * 8 - Hq)] = __float2bfloat16_rn(0.f);
    } else {
      for (int e = threadIdx.x; e < kGtCh * NT * 8; e += kGtThreads) {
        const int c = e / (NT * 8), h = e % (NT * 8);
        ws[c * LDW + h] = (h < Hq && c0 + c < C) ? w[(size_t)(c0 + c) * Hq + h] : __float2bfloat16_rn(0.f);
      }
    }
    __syncthreads();
    const bf16* xr = xs + (warp * 16 + g) * kLdx + 2 * t;
#pragma unroll
    for (int ks = 0; ks < kGtCh / 16; ++ks) {
      uint32_t a[4] = {lds32(xr + ks * 16), lds32(xr + 8 * kLdx + ks * 16), lds32(xr + ks * 16 + 8),
                       lds32(xr + 8 * kLdx + ks * 16 + 8)};
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        // B fragment (k = channels, n = heads) from the [channel][head] tile: two stored 8 x 8 blocks, transposed
        uint32_t b0, b1;
        ldmatrix_x2_trans(b0, b1, ws + (ks * 16 + (lane & 15)) * LDW + n * 8);
        mma_bf16(acc[n], a, b0, b1);
      }
    }
  }
  float* gb = gate + (size_t)b * Hq * L;
  const int tok = l0 + warp * 16 + g;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int h = n * 8 + 2 * t;
    if (h < Hq) {
      if (tok < L) gb[(size_t)h * L + tok] = tanhf(acc[n][0]);
      if (tok + 8 < L) gb[(size_t)h * L + tok + 8] = tanhf(acc[n][2]);
    }
    if (h + 1 < Hq) {
      if (tok < L) gb[(size_t)(h + 1) * L + tok] = tanhf(acc[n][1]);
      if (tok + 8 < L) gb[(size_t)(h + 1) * L + tok + 8] = tanhf(acc[n][3]);
    }
  }
}

// ---------------------------------------------------------------------------------------------- dX
// grid (ceil(L / 64), batch); KT = head tiles of 16 (the contraction)
template <int KT>
__global__ void __launch_bounds__(kGtThreads) gate_bwd_dx_kernel(const bf16* __restrict__ w, const bf16* __restrict__ dz_tm,
                                                                 int L, int Lp, int C, int Hq, int out_f32,
                                                                 void* __restrict__ dx) {
  constexpr int LDZ = KT * 16 + 8;
  constexpr int LDO = kDxCh + 4;
  __shared__ __align__(16) bf16 az[kGtTok * LDZ];            // dz^T: [token][head]
  __shared__ __align__(16) bf16 ws[kDxCh * LDZ];             // W chunk: [channel][head]
  __shared__ __align__(16) float st[kGtTok * LDO];           // output tile, for coalesced stores
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int l0 = blockIdx.x * kGtTok, b = blockIdx.y;
  {
    // the tile's 64 rows of dz_tm are contiguous: 16-byte loads
    const uint4* src = reinterpret_cast<const uint4*>(dz_tm + ((size_t)b * Lp + l0) * (KT * 16));
    for (int e = threadIdx.x; e < kGtTok * KT * 2; e += kGtThreads) {
      const int tl = e / (KT * 2), ch = e % (KT * 2);
      *reinterpret_cast<uint4*>(az + tl * LDZ + ch * 8) = __ldg(src + e);
    }
  }
  __syncthreads();
  uint32_t a[KT][4];
  {
    const bf16* ar = az + (warp * 16 + g) * LDZ + 2 * t;
#pragma unroll
    for (int ks = 0; ks < KT; ++ks) {
      a[ks][0] = lds32(ar + ks * 16);
      a[ks][1] = lds32(ar + 8 * LDZ + ks * 16);
      a[ks][2] = lds32(ar + ks * 16 + 8);
      a[ks][3] = lds32(ar + 8 * LDZ + ks * 16 + 8);
    }
  }
  for (int c0 = 0; c0 < C; c0 += kDxCh) {
    __syncthreads();                                           // previous chunk's stores have read st, its products ws
    if (Hq % 8 == 0 && c0 + kDxCh <= C && (reinterpret_cast<uintptr_t>(w) & 15u) == 0) {
      // rows of W are whole 16-byte vectors: copy them as such, then clear the padding heads
      const int vec = Hq / 8;
      const uint4* src = reinterpret_cast<const uint4*>(w + (size_t)c0 * Hq);
      for (int e = threadIdx.x; e < kDxCh * vec; e += kGtThreads) {
        const int c = e / vec, v = e % vec;
        *reinterpret_cast<uint4*>(ws + c * LDZ + v * 8) = __ldg(src + e);
      }
      for (int e = threadIdx.x; e < kDxCh * (KT * 16 - Hq); e += kGtThreads) {
        const int c = e / (KT * 16 - Hq), h = Hq + e % (KT * 16 - Hq);
        ws[c * LDZ + h] = __float2bfloat16_rn(0.f);
      }
    } else {
      for (int e = threadIdx.x; e < kDxCh * KT * 16; e += kGtThreads) {
        const int c = e / (KT * 16), h = e % (KT * 16);
        ws[c * LDZ + h] = (h < Hq && c0 + c < C) ? w[(size_t)(c0 + c) * Hq + h] : __float2bfloat16_rn(0.f);
      }
    }
    __syncthreads();
#pragma unroll 4
    for (int n = 0; n < kDxCh / 8; ++n) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const bf16* wr = ws + (n * 8 + g) * LDZ + 2 * t;
#pragma unroll
      for (int ks = 0; ks < KT; ++ks) mma_bf16(acc, a[ks], lds32(wr + ks * 16), lds32(wr + ks * 16 + 8));
      *reinterpret_cast<float2*>(st + (warp * 16 + g) * LDO + n * 8 + 2 * t) = make_float2(acc[0], acc[1]);
      *reinterpret_cast<float2*>(st + (warp * 16 + g + 8) * LDO + n * 8 + 2 * t) = make_float2(acc[2], acc[3]);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < kGtTok * (kDxCh / 8); e += kGtThreads) {
      const int r = e / (kDxCh / 8), ch = e % (kDxCh / 8);
      if (l0 + r >= L || c0 + ch * 8 >= C) continue;
      const float4 v0 = *reinterpret_cast<const float4*>(st + r * LDO + ch * 8);
      const float4 v1 = *reinterpret_cast<const float4*>(st + r * LDO + ch * 8 + 4);
      const size_t idx = ((size_t)b * L + l0 + r) * C + c0 + ch * 8;
      if (out_f32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(dx) + idx) = v0;
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(dx) + idx + 4) = v1;
      } else {
        __nv_bfloat162 p0 = __floats2bfloat162_rn(v0.x, v0.y), p1 = __floats2bfloat162_rn(v0.z, v0.w);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(v1.x, v1.y), p3 = __floats2bfloat162_rn(v1.z, v1.w);
        uint4 o;
        o.x = *reinterpret_cast<uint32_t*>(&p0); o.y = *reinterpret_cast<uint32_t*>(&p1);
        o.z = *reinterpret_cast<uint32_t*>(&p2); o.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(dx) + idx) = o;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------- dW_g
// grid (ceil(C / 128), splits, batch): partial[(b * splits + s)][c][h] = sum over the split's tokens of X[l, c] dz[l, h]
template <int NT>
__global__ void __launch_bounds__(kGtThreads) gate_bwd_dw_kernel(const bf16* __restrict__ x, const bf16* __restrict__ dz_hm,
                                                                 int L, int Lp, int C, int Hq, int HP,
                                                                 float* __restrict__ partial) {
  constexpr int LDZ = kGtTok + 8;
  __shared__ __align__(16) bf16 xs[kGtTok * kLdx];           // [token][channel]; read transposed by ldmatrix
  __shared__ __align__(16) bf16 dz[NT * 8 * LDZ];            // [head][token]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int c0 = blockIdx.x * kGtCh, s = blockIdx.y, b = blockIdx.z, splits = gridDim.y;
  const int per = ((L + splits - 1) / splits + kGtTok - 1) / kGtTok * kGtTok;      // tokens per split, whole tiles
  const int l_beg = s * per, l_end = min(L, l_beg + per);
  const bf16* xb = x + (size_t)b * L * C;
  const bf16* zb = dz_hm + (size_t)b * HP * Lp;
  float acc[2][NT][4];                                        // this warp: channels 32 warp .. + 31 (two tiles of 16)
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;
  for (int l0 = l_beg; l0 < l_end; l0 += kGtTok) {
    __syncthreads();
    load_x_tile(xs, xb, l0, L, c0, C);
    for (int e = threadIdx.x; e < NT * 8 * (kGtTok / 8); e += kGtThreads) {
      const int h = e / (kGtTok / 8), ch = e % (kGtTok / 8);
      uint4 v = make_uint4(0, 0, 0, 0);
      if (h < HP) v = __ldg(reinterpret_cast<const uint4*>(zb + (size_t)h * Lp + l0 + ch * 8));
      *reinterpret_cast<uint4*>(dz + h * LDZ + ch * 8) = v;
    }
    __syncthreads();
#pragma unroll
    for (int ks = 0; ks < kGtTok / 16; ++ks) {
      uint32_t a[2][4];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        // four stored 8 x 8 blocks (tokens x channels) -> A fragment (rows = channels, k = tokens) of one 16 x 16 tile:
        // lanes 0-7: tokens 0-7 / channels 0-7, 8-15: tokens 0-7 / channels 8-15, 16-23 and 24-31: tokens 8-15
        const int tok = ks * 16 + (lane >> 4) * 8 + (lane & 7);
        const int ch = warp * 32 + m * 16 + ((lane >> 3) & 1) * 8;
        ldmatrix_x4_trans(a[m], xs + tok * kLdx + ch);
      }
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const bf16* zr = dz + (n * 8 + g) * LDZ + ks * 16 + 2 * t;
        const uint32_t b0 = lds32(zr), b1 = lds32(zr + 8);
        mma_bf16(acc[0][n], a[0], b0, b1);
        mma_bf16(acc[1][n], a[1], b0, b1);
      }
    }
  }
  float* out = partial + (size_t)(b * splits + s) * C * Hq;
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const int c = c0 + warp * 32 + m * 16 + g, h = n * 8 + 2 * t;
      if (c < C) {
        if (h < Hq) out[(size_t)c * Hq + h] = acc[m][n][0];
        if (h + 1 < Hq) out[(size_t)c * Hq + h + 1] = acc[m][n][1];
      }
      if (c + 8 < C) {
        if (h < Hq) out[(size_t)(c + 8) * Hq + h] = acc[m][n][2];
        if (h + 1 < Hq) out[(size_t)(c + 8) * Hq + h + 1] = acc[m][n][3];
      }
    }
}

__global__ void gate_reduce_dw_kernel(const float* __restrict__ partial, int parts, size_t n, float* __restrict__ dw) {
  const size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  float acc = 0.f;
  for (int p = 0; p < parts; ++p) acc += partial[(size_t)p * n + i];
  dw[i] = acc;
}

}  // namespace

bool gate_supported(int hidden, int heads) { return hidden > 0 && hidden % 8 == 0 && heads > 0 && heads <= 64; }

namespace {
int padded_heads(int heads) { return (heads + 15) / 16 * 16; }
int padded_tokens(int L) { return (L + kGtTok - 1) / kGtTok * kGtTok; }
size_t dz_bytes(int batch, int L, int heads) { return align_up((size_t)batch * padded_tokens(L) * padded_heads(heads) * sizeof(bf16), 256); }
}  // namespace

// [partial sums of dW_g][dz head-major][dz token-major]
size_t gate_bwd_workspace_bytes(int batch, int L, int hidden, int heads) {
  return align_up((size_t)batch * kGtSplits * hidden * heads * sizeof(float), 256) + 2 * dz_bytes(batch, L, heads);
}

cudaError_t launch_gate_fwd(int batch, int L, int C, int Hq, const bf16* x, const bf16* w, float* gate, cudaStream_t st) {
  dim3 grid((L + kGtTok - 1) / kGtTok, batch);
  const int nt = (Hq + 7) / 8;
#define VSA2_GATE_FWD(NT_) gate_fwd_kernel<NT_><<<grid, kGtThreads, 0, st>>>(x, w, L, C, Hq, gate)
  if (nt <= 1) VSA2_GATE_FWD(1);
  else if (nt <= 2) VSA2_GATE_FWD(2);
  else if (nt <= 4) VSA2_GATE_FWD(4);
  else if (nt <= 5) VSA2_GATE_FWD(5);
  else if (nt <= 6) VSA2_GATE_FWD(6);
  else VSA2_GATE_FWD(8);
#undef VSA2_GATE_FWD
  return cudaGetLastError();
}

cudaError_t launch_gate_bwd(int batch, int L, int C, int Hq, int out_f32, const bf16* x, const bf16* w, const float* gate,
                            const float* dgate, float* d_w, void* dx, void* workspace, cudaStream_t st) {
  const int HP = padded_heads(Hq), Lp = padded_tokens(L);
  float* partial = reinterpret_cast<float*>(workspace);
  unsigned char* wsb = reinterpret_cast<unsigned char*>(workspace);
  bf16* dz_hm = reinterpret_cast<bf16*>(wsb + align_up((size_t)batch * kGtSplits * C * Hq * sizeof(float), 256));
  bf16* dz_tm = reinterpret_cast<bf16*>(reinterpret_cast<unsigned char*>(dz_hm) + dz_bytes(batch, L, Hq));
  gate_dz_kernel<<<dim3(Lp / kGtTok, batch), kGtThreads, (size_t)HP * (kGtTok + 8) * sizeof(bf16), st>>>(gate, dgate, L, Lp, Hq,
                                                                                                   HP, dz_hm, dz_tm);
  {
    dim3 grid((L + kGtTok - 1) / kGtTok, batch);
    const int kt = (Hq + 15) / 16;
#define VSA2_GATE_DX(KT_) gate_bwd_dx_kernel<KT_><<<grid, kGtThreads, 0, st>>>(w, dz_tm, L, Lp, C, Hq, out_f32, dx)
    if (kt <= 1) VSA2_GATE_DX(1);
    else if (kt <= 2) VSA2_GATE_DX(2);
    else if (kt <= 3) VSA2_GATE_DX(3);
    else VSA2_GATE_DX(4);
#undef VSA2_GATE_DX
  }
  {
    dim3 grid((C + kGtCh - 1) / kGtCh, kGtSplits, batch);
    const int nt = (Hq + 7) / 8;
#define VSA2_GATE_DW(NT_) gate_bwd_dw_kernel<NT_><<<grid, kGtThreads, 0, st>>>(x, dz_hm, L, Lp, C, Hq, HP, partial)
    if (nt <= 1) VSA2_GATE_DW(1);
    else if (nt <= 2) VSA2_GATE_DW(2);
    else if (nt <= 4) VSA2_GATE_DW(4);
    else if (nt <= 5) VSA2_GATE_DW(5);
    else if (nt <= 6) VSA2_GATE_DW(6);
    else VSA2_GATE_DW(8);
#undef VSA2_GATE_DW
  }
  const size_t n = (size_t)C * Hq;
  gate_reduce_dw_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(partial, batch * kGtSplits, n, d_w);
  return cudaGetLastError();
}

}  // namespace vsa2
