// Shared device/host definitions of the VSA2 library: geometry of the latent grid, index
// maps between raster tokens and cubes (paper Sec. 2.2 "Permutation"), workspace layout.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vsa2.h"

namespace vsa2 {

typedef __nv_bfloat16 bf16;

constexpr int kBlockTokens = 64;   // tokens per block handled by the kernels (a 128-token cube runs as two)

// Everything a kernel needs to know about the problem; passed by value.
struct Geo {
  int batch, Hq, Hkv, rep, D;
  int T, H, W, L;
  int Bt, Bh, Bw, Nt, Nh, Nw, N;
  int Rt, Rh, Rw, Gt, Gh, Gw, G;
  int K;            // TopK after clamping
  int mode;         // VSA2_PER_*
  int out_f32;      // 1: outputs are fp32, 0: bf16
  int flags;
  float scale;      // softmax scale
  long long nnz_cap;
  // Text tokens (the sentence after Eq. 12): every token tensor holds S = L + Lt rows per head, the L video tokens in raster
  // order followed by Lt text tokens.  The routing and coarse kernels see the video part only (N = Nvid cubes).  The fine
  // kernels and the backward preprocess run on the BLOCK problem: N = Nvid + ceil(Lt / 64) blocks, block j < Nvid is video
  // cube j, block j >= Nvid holds text tokens 64 (j - Nvid) .. ; their maps are the block maps extended by the text blocks.
  int Nvid, Lt, S;
  // ceil(2^32 / d) for d = Nw, Nh, Bw, Bh (geo_set_magics): the index arithmetic of the kernels divides by these with one
  // multiply instead of a reciprocal, which would run on the unit the softmax exponentials need
  unsigned mNw, mNh, mBw, mBh;
};
inline unsigned div_magic(int d) { return d <= 1 ? 0u : (unsigned)((0x100000000ull + (unsigned)d - 1ull) / (unsigned)d); }
// to be called wherever Nw, Nh, Bw or Bh of a Geo are set
inline void geo_set_magics(Geo& g) {
  g.mNw = div_magic(g.Nw);
  g.mNh = div_magic(g.Nh);
  g.mBw = div_magic(g.Bw);
  g.mBh = div_magic(g.Bh);
}

// Status block at the start of every workspace.
struct StatusBlock {
  int status;       // VSA2_OK / VSA2_ERR_DEVICE_TIMEOUT / VSA2_ERR_MAP_OVERFLOW
  int detail;
  int pad[62];
};

// Brackets the launches of one kernel group: counts them and records the caller's timing events.
struct ProfScope {
  int id;
  cudaStream_t st;
  ProfScope(int kernel_id, cudaStream_t stream, int launches);
  ~ProfScope();
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// q = n / d, r = n % d for 0 <= n < 2^22 and 0 < d < 2^10 with m = ceil(2^32 / d) (0 for d = 1): floor(n m / 2^32), exact
// while n d < 2^32 -- one multiply.  The tensor-core kernels decode cube and token indices several times per tile; the
// earlier form (a reciprocal and a fix-up) runs on the special-function unit, behind the exponentials of the softmax warps,
// which cost a service warp of the 128-token backward 4000 cycles per tile.  A translation unit that defines
// VSA2_RECIPROCAL_DIVMOD before including this header keeps the reciprocal form (where that measured faster).
// (host and device: vsa2_selftest_divmod checks the multiply form on the host, exhaustively for small divisors)
__host__ __device__ __forceinline__ int mulhi_div(int n, unsigned m) {
  return m == 0u ? n : (int)(((unsigned long long)(unsigned)n * m) >> 32);
}
__device__ __forceinline__ void fast_divmod(int n, int d, unsigned m, int& q, int& r) {
#ifdef VSA2_RECIPROCAL_DIVMOD
  (void)m;
  q = __float2int_rz(__fdividef((float)n, (float)d));
  r = n - q * d;
  if (r < 0) {
    --q;
    r += d;
  } else if (r >= d) {
    ++q;
    r -= d;
  }
#else
  q = mulhi_div(n, m);
  r = n - q * d;
#endif
}

// cube n -> (nt, nh, nw);  n = (nt*Nh + nh)*Nw + nw
__device__ __forceinline__ void cube_coords(const Geo& g, int n, int& nt, int& nh, int& nw) {
  int r;
  fast_divmod(n, g.Nw, g.mNw, r, nw);
  fast_divmod(r, g.Nh, g.mNh, nt, nh);
}

// position (bt, bh, bw) inside cube (nt, nh, nw) -> raster token index, or -1 if padding
__device__ __forceinline__ int cube_token_at(const Geo& g, int nt, int nh, int nw, int bt, int bh, int bw) {
  int t = nt * g.Bt + bt, h = nh * g.Bh + bh, w = nw * g.Bw + bw;
  if (t >= g.T || h >= g.H || w >= g.W) return -1;
  return (t * g.H + h) * g.W + w;
}

// position p in [0, B) inside a cube, ordered (bt, bh, bw) -> raster token index, or -1 if padding
__device__ __forceinline__ int cube_token(const Geo& g, int nt, int nh, int nw, int p) {
  int bw, bh, bt, r;
  fast_divmod(p, g.Bw, g.mBw, r, bw);
  fast_divmod(r, g.Bh, g.mBh, bt, bh);
  return cube_token_at(g, nt, nh, nw, bt, bh, bw);
}

// number of valid tokens of cube n (0 only for the empty trailing half-cubes of a 128-token-cube problem)
__device__ __forceinline__ int cube_count(const Geo& g, int n) {
  int nt, nh, nw;
  cube_coords(g, n, nt, nh, nw);
  int ct = min(g.Bt, g.T - nt * g.Bt), ch = min(g.Bh, g.H - nh * g.Bh), cw = max(0, min(g.Bw, g.W - nw * g.Bw));
  return ct * ch * cw;
}

// router sub-cube gsub of cube n: number of valid tokens (0 = the sub-cube is padding only)
__device__ __forceinline__ int subcube_count(const Geo& g, int n, int gsub) {
  int nt, nh, nw;
  cube_coords(g, n, nt, nh, nw);
  int gw = gsub % g.Gw;
  int r = gsub / g.Gw;
  int gh = r % g.Gh;
  int gt = r / g.Gh;
  int t0 = nt * g.Bt + gt * g.Rt, h0 = nh * g.Bh + gh * g.Rh, w0 = nw * g.Bw + gw * g.Rw;
  int ct = max(0, min(g.Rt, g.T - t0)), ch = max(0, min(g.Rh, g.H - h0)), cw = max(0, min(g.Rw, g.W - w0));
  return ct * ch * cw;
}

// ---- blocks of the fine kernels: video cubes followed by text blocks ---------------------------------------------------
__device__ __forceinline__ bool block_is_text(const Geo& g, int j) { return j >= g.Nvid; }
// TMA box coordinates (dimensions 1..3 of the 5-D maps) of block j: a video cube in the raster map, or 64 rows of the text map
__device__ __forceinline__ void block_box(const Geo& g, int j, int& c1, int& c2, int& c3) {
  if (j < g.Nvid) {
    int jt, jh, jw;
    cube_coords(g, j, jt, jh, jw);
    c1 = jw * g.Bw; c2 = jh * g.Bh; c3 = jt * g.Bt;
  } else {
    c1 = (j - g.Nvid) * kBlockTokens; c2 = 0; c3 = 0;
  }
}
// position p of block j -> row of the token tensors (0 .. S-1), or -1 if padding
__device__ __forceinline__ int block_token(const Geo& g, int j, int p) {
  if (j < g.Nvid) {
    int jt, jh, jw;
    cube_coords(g, j, jt, jh, jw);
    return cube_token(g, jt, jh, jw, p);
  }
  const int t = (j - g.Nvid) * kBlockTokens + p;
  return t < g.Lt ? g.L + t : -1;
}
// valid tokens of block j
__device__ __forceinline__ int block_count(const Geo& g, int j) {
  if (j < g.Nvid) return cube_count(g, j);
  return min(kBlockTokens, g.Lt - (j - g.Nvid) * kBlockTokens);
}
// work item -> (batch * heads index, block).  With text tokens the blocks of a head are handed out in descending order, so
// that the text blocks (whose lists are the longest by far) start first and the persistent CTAs do not end on them.
__device__ __forceinline__ void item_block(const Geo& g, int item, int& bh, int& i) {
  bh = item / g.N;
  const int r = item - bh * g.N;
  i = g.Lt > 0 ? g.N - 1 - r : r;
}
__device__ __forceinline__ int block_item(const Geo& g, int bh, int i) { return bh * g.N + (g.Lt > 0 ? g.N - 1 - i : i); }

__device__ __forceinline__ void store_out(void* base, size_t idx, float v, int out_f32) {
  if (out_f32) reinterpret_cast<float*>(base)[idx] = v;
  else reinterpret_cast<bf16*>(base)[idx] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------------------------
// launchers implemented in the .cu files (all enqueue on `st`, return cudaGetLastError())
// ---------------------------------------------------------------------------------------------
cudaError_t launch_pool(const Geo& g, const bf16* x, int heads, bf16* xr, float* xc, cudaStream_t st);
cudaError_t launch_pool_router(const Geo& g, const bf16* q, const bf16* k, bf16* qr, bf16* kr, cudaStream_t st);
cudaError_t launch_pool_coarse(const Geo& g, const bf16* q, const bf16* k, const bf16* v, float* qc, float* kc, float* vc,
                               cudaStream_t st);

// raster <-> cube-major copy of a [batch, heads, L or N*B, D] bf16 tensor (pool.cu)
cudaError_t launch_permute(const Geo& g, const bf16* src, int heads, bool inverse, bf16* dst, cudaStream_t st);

cudaError_t launch_router_scores(const Geo& g, const bf16* qr, const bf16* kr, float* lse_r, float* pr,
                                 cudaStream_t st);

// tensor-core router (router_tc.cu): lse_r holds log2-domain row statistics between its two passes
bool router_tc_supported(const Geo& g);
cudaError_t launch_router_scores_tc(const Geo& g, const bf16* qr, const bf16* kr, float* lse_r, float* pr,
                                    StatusBlock* status, cudaStream_t st);

struct SelectScratch {
  unsigned* hist;        // [BH][3][2048]
  unsigned* state;       // [BH][8]
  float* row_tau;        // [BH][N]
  int* row_eq_take;      // [BH][N]
  int* row_cnt;          // [BH][N]
  int* row_gt;           // [BH][N]
  int* row_eq;           // [BH][N]
  unsigned* bitmap;      // [BH][N][words]   rows x column words
  unsigned* bitmap_t;    // [BH][N][words]   columns x row words
  int words;             // ceil(N/32)
};
cudaError_t launch_select(const Geo& g, const float* pr, const int* budgets, const SelectScratch& s,
                          int* row_ptr, int* col_idx, int* col_ptr, int* row_idx, StatusBlock* status,
                          cudaStream_t st);

// coarse branch forward on the fp32 cube means, TF32 tensor-core products with register-resident accumulators
// (coarse_fwd_mma.cu)
cudaError_t launch_coarse_fwd_mma(const Geo& g, const float* qc, const float* kc, const float* vc, float* oc_hat,
                                  float* lse_c, cudaStream_t st);

cudaError_t launch_fine_fwd(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                            const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                            float* lse, cudaStream_t st);

// coarse branch through the fine-branch kernels on the pooled grid (coarse_pooled.cu); offsets into a scratch region
struct PooledLayout {
  size_t status, q16, k16, v16, ptr, idx, do16, delta, dk_kv, dv_kv, total;
};
Geo pooled_geo(const Geo& g);
PooledLayout pooled_layout(const Geo& g, bool backward);
cudaError_t launch_coarse_fwd_pooled(const Geo& g, const float* qc, const float* kc, const float* vc, float* oc_hat,
                                     float* lse_c, void* workspace, StatusBlock* caller_status, cudaStream_t st);
cudaError_t launch_coarse_bwd_pooled(const Geo& g, const float* qc, const float* kc, const float* vc, const float* oc_hat,
                                     const float* lse_c, const float* d_oc_hat, float* dqc, float* dkc, float* dvc,
                                     void* workspace, StatusBlock* caller_status, cudaStream_t st);

// cubes of 128 tokens as pairs of 64-token half-cubes (wide_cube.cu); `narrow` is narrow_geo() of the problem
bool wide_cube(const Geo& g);
Geo narrow_geo(const Geo& g);
cudaError_t launch_fold_scores(const Geo& narrow, const float* pr64, float* pr, cudaStream_t st);
// "group head" routing: replaces every block score by the sum over the query heads of its KV group (in place)
cudaError_t launch_group_sum_scores(const Geo& g, float* pr, cudaStream_t st);
cudaError_t launch_fold_mean(const Geo& narrow, int heads, const float* x64, float* x, cudaStream_t st);
cudaError_t launch_fold_sum(const Geo& narrow, int heads, const float* x64, float* x, cudaStream_t st);
cudaError_t launch_expand_rows(const Geo& narrow, int heads, bool by_count, const float* x, float* x64,
                               cudaStream_t st);
cudaError_t launch_expand_map(const Geo& narrow, const int* ptr, const int* idx, int* ptr64, int* idx64,
                              cudaStream_t st);
// block map of the video cubes (g: the video problem) -> block map with `text_blocks` text blocks appended to every row and
// all-ones text rows; capx = capacity per (batch, head) of idxx
cudaError_t launch_extend_map(const Geo& g, int text_blocks, const int* ptr, const int* idx, int* ptrx, int* idxx, long long capx,
                              cudaStream_t st);

// gate projection and its backward (gate.cu)
bool gate_supported(int hidden, int heads);
size_t gate_bwd_workspace_bytes(int batch, int L, int hidden, int heads);
cudaError_t launch_gate_fwd(int batch, int L, int C, int Hq, const bf16* x, const bf16* w, float* gate, cudaStream_t st);
cudaError_t launch_gate_bwd(int batch, int L, int C, int Hq, int out_f32, const bf16* x, const bf16* w, const float* gate,
                            const float* dgate, float* d_w, void* dx, void* workspace, cudaStream_t st);

// tensor-core forward (fine_fwd_tc.cu); `status` heads a workspace of fine_fwd_tc_workspace_bytes()
size_t fine_fwd_tc_workspace_bytes();
int fwd_rescue_capacity();
void set_fwd_rescue_capacity(int cap);
cudaError_t launch_fine_fwd_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                               const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                               float* lse, StatusBlock* status, cudaStream_t st);

// tensor-core forward with the queries in the accumulator rows (fine_fwd_rows_tc.cu); same workspace as launch_fine_fwd_tc
bool fine_fwd_rows_supported(const Geo& g);
cudaError_t launch_fine_fwd_rows_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                                    const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                                    float* lse, StatusBlock* status, cudaStream_t st);

// tensor-core forward with two query blocks (128 rows) per tile (fine_fwd_rows2_tc.cu): the halves of a 128-token cube, or one
// block of two heads that share their map.  `g`, the map and oc_hat are those of the half-cube problem (or, with pair_heads,
// of the ordinary 64-token problem); the workspace is the one of launch_fine_fwd_tc
bool fine_fwd_rows2_supported(const Geo& g, bool pair_heads);
cudaError_t launch_fine_fwd_rows2_tc(const Geo& g, bool pair_heads, const bf16* q, const bf16* k, const bf16* v, const float* gate,
                                     const int* row_ptr, const int* col_idx, const float* oc_hat, void* o, bf16* o_res,
                                     float* lse, StatusBlock* status, cudaStream_t st);

// tensor-core backward passes for cubes of 128 tokens (fine_bwd128_tc.cu): `g` and the maps are those of the half-cube problem
bool fine_bwd128_supported(const Geo& g);
bool fine_bwd_dkv_wants_pair(const Geo& g);
cudaError_t launch_fine_bwd128_dq_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                     const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                                     const float* dqc, void* dq, StatusBlock* status, cudaStream_t st, void* q16, void* k16);
cudaError_t launch_fine_bwd128_dkv_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                      const float* lse, const float* delta, const int* col_ptr, const int* row_idx,
                                      const float* dkc, const float* dvc, void* dk, void* dv, StatusBlock* status,
                                      cudaStream_t st, const void* q16, const void* k16);

// tensor-core backward passes (fine_bwd_tc.cu)
cudaError_t launch_fine_bwd_dq_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                  const float* lse, const float* delta, const int* row_ptr, const int* col_idx,
                                  const float* dqc, void* dq, StatusBlock* status, cudaStream_t st, void* q16, void* k16);
bool fine_bwd_dq_uses_f16(const Geo& g);
// Slot of StatusBlock.pad that holds the range flag of the fp16 dQ passes (the slot behind it: the fallback launch's counter)
constexpr int kRangeFlagSlot = 8;
// fp16 copies of two bf16 tensors (element counts multiples of 8); a finite value beyond the fp16 range sets *range_flag
cudaError_t launch_cast_bf16_to_f16(const bf16* a, void* a16, size_t na, const bf16* b, void* b16, size_t nb, int* range_flag,
                                    cudaStream_t st);
cudaError_t launch_fine_bwd_dkv_tc(const Geo& g, const bf16* q, const bf16* k, const bf16* v, const bf16* d_o,
                                   const float* lse, const float* delta, const int* col_ptr, const int* row_idx,
                                   const float* dkc, const float* dvc, void* dk, void* dv, StatusBlock* status,
                                   cudaStream_t st, bool split_long_columns, int* item_list, const void* q16,
                                   const void* k16, void* v16, void* do16);
bool fine_bwd_dkv_gqa_uses_f16(const Geo& g);
bool fine_bwd_dkv_splits_long_columns(const Geo& g, bool split_long_columns);

cudaError_t launch_bwd_preprocess(const Geo& g, const bf16* d_o, const void* o, const bf16* o_res, const float* gate,
                                  const float* oc_hat, float* delta, float* dgate, float* d_oc_hat,
                                  cudaStream_t st);
}  // namespace vsa2
