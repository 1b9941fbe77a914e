// Cubes of 128 tokens (the 4 x 4 x 8 cube with 2 x 2 x 2 router pooling, G = 16) on top of the 64-token kernels.
//
// A cube of 128 tokens whose w extent is even is two 64-token half-cubes that are neighbours along w, and in the
// half-cube grid (same Nt, Nh; twice Nw) cube c is exactly the half-cubes 2c and 2c+1.  When the grid's last cube
// along w reaches no further than its first half, its second half-cube is EMPTY: it stays in the half-cube grid so
// that the 2c, 2c+1 numbering holds, has no valid token or router sub-cube, contributes zero weight to every fold,
// and the fine kernels treat it like the padding of any ragged cube (keys masked, nothing stored).  Every quantity of the
// method at cube level follows from the half-cube quantities without touching the tokens again:
//   * router (Eq. 5-7): the 2 x 2 x 2 sub-cubes of a cube are the sub-cubes of its two halves, so the router
//     softmax over all sub-cube keys is the same matrix, and the cube-level score is the mean over a 16 x 16
//     sub-block, i.e. a weighted mean of four half-cube scores (weights: valid query sub-cubes of each half);
//   * coarse branch (Eq. 1-4): the cube mean is the count-weighted mean of the two half means; the cube's
//     coarse output row is shared by both halves; gradients of the halves add;
//   * fine branch (Eq. 12): a kept (query cube, key cube) pair is the four kept half-cube pairs.
// The kernels here are these folds and expansions; all are small HBM-bound element-wise passes.
#include "common.cuh"

namespace vsa2 {

bool wide_cube(const Geo& g) { return g.Bt * g.Bh * g.Bw == 2 * kBlockTokens; }

// The half-cube geometry of a 128-token-cube problem.
Geo narrow_geo(const Geo& g) {
  Geo n = g;
  n.Bw = g.Bw / 2;
  n.Nw = g.Nw * 2;
  geo_set_magics(n);
  n.N = g.N * 2;
  n.Nvid = n.N;
  n.Gw = n.Bw / n.Rw;
  n.G = n.Gt * n.Gh * n.Gw;
  n.nnz_cap = g.nnz_cap * 4;
  n.K = g.K * 2 < n.N ? g.K * 2 : n.N;
  return n;
}

namespace {

__device__ __forceinline__ int valid_subcubes(const Geo& n, int cube) {
  int v = 0;
  for (int s = 0; s < n.G; ++s) v += subcube_count(n, cube, s) > 0;
  return v;
}

// pr [BH, 2N, 2N] half-cube scores -> out [BH, N, N].  Eq. 7 divides the sum over a cube pair's valid sub-cube
// pairs by (valid query sub-cubes of the cube) * G; a half-cube score is the same with its own counts.
__global__ void __launch_bounds__(256) fold_scores_kernel(Geo n, const float* __restrict__ pr, float* __restrict__ out) {
  const int N = n.N / 2;
  const int c = blockIdx.x;
  const size_t bh = (size_t)blockIdx.z * n.Hq + blockIdx.y;
  const int vq0 = valid_subcubes(n, 2 * c), vq1 = valid_subcubes(n, 2 * c + 1);
  const float w0 = (float)vq0 / (float)(2 * (vq0 + vq1)), w1 = (float)vq1 / (float)(2 * (vq0 + vq1));
  const float2* r0 = reinterpret_cast<const float2*>(pr + (bh * n.N + 2 * c) * (size_t)n.N);
  const float2* r1 = reinterpret_cast<const float2*>(pr + (bh * n.N + 2 * c + 1) * (size_t)n.N);
  for (int j = threadIdx.x; j < N; j += blockDim.x) {
    const float2 a = __ldg(r0 + j), b = __ldg(r1 + j);
    out[(bh * N + c) * (size_t)N + j] = w0 * (a.x + a.y) + w1 * (b.x + b.y);
  }
}

// x64 [BH, 2N, D] half-cube means -> x [BH, N, D] cube means (count-weighted)
__global__ void __launch_bounds__(256) fold_mean_kernel(Geo n, const float* __restrict__ x64, float* __restrict__ x,
                                                        size_t total) {
  const int D = n.D;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const size_t row = e / D;          // bh * N + c
    const int d = (int)(e % D);
    const int c = (int)(row % (n.N / 2));
    const float c0 = (float)cube_count(n, 2 * c), c1 = (float)cube_count(n, 2 * c + 1);
    float v = x64[(2 * row) * D + d] * c0;
    if (c1 > 0.f) v += x64[(2 * row + 1) * D + d] * c1;       // an empty second half (beyond the grid) has no mean
    x[e] = v / (c0 + c1);
  }
}

// x64 [BH, 2N, D] -> x [BH, N, D]: sum of the two halves
__global__ void __launch_bounds__(256) fold_sum_kernel(int D, const float* __restrict__ x64, float* __restrict__ x,
                                                       size_t total) {
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const size_t row = e / D;
    const int d = (int)(e % D);
    x[e] = x64[(2 * row) * D + d] + x64[(2 * row + 1) * D + d];
  }
}

// x [BH, N, D] -> x64 [BH, 2N, D]: each half gets the cube's row; with `by_count` scaled by the half's share of the
// cube's tokens (the consumer divides by the half's own count, which leaves row / cube count as Eq. 1 requires)
__global__ void __launch_bounds__(256) expand_rows_kernel(Geo n, int by_count, const float* __restrict__ x,
                                                          float* __restrict__ x64, size_t total64) {
  const int D = n.D;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total64; e += (size_t)gridDim.x * blockDim.x) {
    const size_t row64 = e / D;        // bh * 2N + i
    const int d = (int)(e % D);
    float v = x[(row64 >> 1) * D + d];
    if (by_count) {
      const int i = (int)(row64 % n.N);
      v *= (float)cube_count(n, i) / (float)(cube_count(n, i & ~1) + cube_count(n, i | 1));
    }
    x64[e] = v;
  }
}

// Compressed rows (or columns) of the cube map -> those of the half-cube map: list (c; j0, j1, ...) becomes the two
// lists (2c; 2j0, 2j0+1, 2j1, ...) and (2c+1; same).  ptr [BH, N+1], idx [BH, cap] -> ptr64 [BH, 2N+1], idx64 [BH, 4cap]
__global__ void __launch_bounds__(128) expand_map_kernel(int N, int Hq, long long cap, const int* __restrict__ ptr,
                                                         const int* __restrict__ idx, int* __restrict__ ptr64,
                                                         int* __restrict__ idx64) {
  const int c = blockIdx.x;
  const size_t bh = (size_t)blockIdx.z * Hq + blockIdx.y;
  const int* p = ptr + bh * (N + 1);
  // (a map whose selection overflowed nnz_cap has row pointers beyond the capacity: such rows are cut at `cap`)
  const int beg = (int)min((long long)p[c], cap), end = (int)min((long long)p[c + 1], cap), len = end - beg;
  const int* src = idx + bh * cap + beg;
  int* p64 = ptr64 + bh * (2 * N + 1);
  int* dst = idx64 + bh * 4 * cap + 4 * (size_t)beg;
  if (threadIdx.x == 0) {
    p64[2 * c] = 4 * beg;
    p64[2 * c + 1] = 4 * beg + 2 * len;
    if (c == N - 1) p64[2 * N] = 4 * end;
  }
  for (int e = threadIdx.x; e < len; e += blockDim.x) {
    const int j = src[e];
    const int2 v = make_int2(2 * j, 2 * j + 1);
    *reinterpret_cast<int2*>(dst + 2 * e) = v;
    *reinterpret_cast<int2*>(dst + 2 * len + 2 * e) = v;
  }
}

// Block map of the video cubes -> block map of the block problem with text tokens (Sec. 2.2, the sentence after Eq. 12): every
// video row (or column) additionally keeps all NtB text blocks, and every text row (column) keeps all Nvid + NtB blocks.
// ptr [BH, Nvid+1], idx [BH, cap] -> ptrx [BH, Nx+1], idxx [BH, capx] with Nx = Nvid + NtB, capx = cap + Nvid NtB + NtB Nx.
// The same rule serves the CSR and the CSC map (the extension is symmetric).
__global__ void __launch_bounds__(128) extend_map_kernel(int Nvid, int NtB, int Hq, long long cap, long long capx,
                                                         const int* __restrict__ ptr, const int* __restrict__ idx,
                                                         int* __restrict__ ptrx, int* __restrict__ idxx) {
  const int r = blockIdx.x, Nx = Nvid + NtB;
  const size_t bh = (size_t)blockIdx.z * Hq + blockIdx.y;
  const int* p = ptr + bh * (Nvid + 1);
  int* px = ptrx + bh * (Nx + 1);
  int* dst = idxx + bh * capx;
  if (r < Nvid) {
    const int beg = (int)min((long long)p[r], cap), end = (int)min((long long)p[r + 1], cap), len = end - beg;
    const int start = beg + r * NtB;
    if (threadIdx.x == 0) px[r] = start;
    const int* src = idx + bh * cap + beg;
    for (int e = threadIdx.x; e < len; e += blockDim.x) dst[start + e] = src[e];
    for (int e = threadIdx.x; e < NtB; e += blockDim.x) dst[start + len + e] = Nvid + e;
  } else {
    const int t = r - Nvid;
    const int start = (int)min((long long)p[Nvid], cap) + Nvid * NtB + t * Nx;
    if (threadIdx.x == 0) {
      px[r] = start;
      if (r == Nx - 1) px[Nx] = start + Nx;
    }
    for (int e = threadIdx.x; e < Nx; e += blockDim.x) dst[start + e] = e;
  }
}

// "group head" routing: the query heads of a KV group share one map.  pr [batch, Hq, N, N]: every entry is replaced by
// the sum over the heads of its group (added in head order), so the selection that follows picks the same set for each
__global__ void __launch_bounds__(256) group_sum_scores_kernel(float* __restrict__ pr, int rep, size_t per_head, size_t groups) {
  const size_t total = groups * per_head;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const size_t grp = e / per_head, off = e % per_head;
    float* base = pr + grp * rep * per_head + off;
    float sum = 0.f;
    for (int r = 0; r < rep; ++r) sum += base[(size_t)r * per_head];
    for (int r = 0; r < rep; ++r) base[(size_t)r * per_head] = sum;
  }
}

int grid_for(size_t total) {
  size_t blocks = (total + 255) / 256;
  return (int)(blocks < 148 * 16 ? (blocks ? blocks : 1) : 148 * 16);
}

}  // namespace

cudaError_t launch_group_sum_scores(const Geo& g, float* pr, cudaStream_t st) {
  const size_t per_head = (size_t)g.N * g.N, groups = (size_t)g.batch * g.Hkv;
  group_sum_scores_kernel<<<grid_for(groups * per_head), 256, 0, st>>>(pr, g.rep, per_head, groups);
  return cudaGetLastError();
}

cudaError_t launch_fold_scores(const Geo& narrow, const float* pr64, float* pr, cudaStream_t st) {
  const int N = narrow.N / 2;
  dim3 grid(N, narrow.Hq, narrow.batch);
  fold_scores_kernel<<<grid, 256, 0, st>>>(narrow, pr64, pr);
  return cudaGetLastError();
}

cudaError_t launch_fold_mean(const Geo& narrow, int heads, const float* x64, float* x, cudaStream_t st) {
  const size_t total = (size_t)narrow.batch * heads * (narrow.N / 2) * narrow.D;
  fold_mean_kernel<<<grid_for(total), 256, 0, st>>>(narrow, x64, x, total);
  return cudaGetLastError();
}

cudaError_t launch_fold_sum(const Geo& narrow, int heads, const float* x64, float* x, cudaStream_t st) {
  const size_t total = (size_t)narrow.batch * heads * (narrow.N / 2) * narrow.D;
  fold_sum_kernel<<<grid_for(total), 256, 0, st>>>(narrow.D, x64, x, total);
  return cudaGetLastError();
}

cudaError_t launch_expand_rows(const Geo& narrow, int heads, bool by_count, const float* x, float* x64,
                               cudaStream_t st) {
  const size_t total = (size_t)narrow.batch * heads * narrow.N * narrow.D;
  expand_rows_kernel<<<grid_for(total), 256, 0, st>>>(narrow, by_count ? 1 : 0, x, x64, total);
  return cudaGetLastError();
}

cudaError_t launch_expand_map(const Geo& narrow, const int* ptr, const int* idx, int* ptr64, int* idx64,
                              cudaStream_t st) {
  dim3 grid(narrow.N / 2, narrow.Hq, narrow.batch);
  expand_map_kernel<<<grid, 128, 0, st>>>(narrow.N / 2, narrow.Hq, narrow.nnz_cap / 4, ptr, idx, ptr64, idx64);
  return cudaGetLastError();
}

cudaError_t launch_extend_map(const Geo& g, int text_blocks, const int* ptr, const int* idx, int* ptrx, int* idxx, long long capx,
                              cudaStream_t st) {
  dim3 grid(g.Nvid + text_blocks, g.Hq, g.batch);
  extend_map_kernel<<<grid, 128, 0, st>>>(g.Nvid, text_blocks, g.Hq, g.nnz_cap, capx, ptr, idx, ptrx, idxx);
  return cudaGetLastError();
}

}  // namespace vsa2
