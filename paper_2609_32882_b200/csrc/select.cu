// TopK selection on the router block scores and construction of the block map
// (paper Eq. 8-9: the N*K largest of the flattened N*N scores; Sec. 2.1 for the per-row form).
// Scores are non-negative floats, so their bit patterns order like unsigned integers: the
// K-th largest value is found by a most-significant-digit radix select, ties at the threshold
// go to the lower flat index, and rows/columns are emitted in ascending order (deterministic,
// integer work only).
#include "common.cuh"

namespace vsa2 {

constexpr int kHistBins = 2048;
// digit positions of the three per-sequence passes: bits [31:21], [20:10], [9:0]
__device__ __forceinline__ int seq_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ unsigned seq_mask(int pass) { return pass == 2 ? 0x3FFu : 0x7FFu; }

// state[bh*8 + ..]: 0 prefix bits, 1 prefix mask, 2 remaining k, 3 tau bits, 4 eq_take
__global__ void sel_init_kernel(unsigned* state, unsigned* hist, int BH, unsigned keep) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < BH * 3 * kHistBins) hist[i] = 0u;
  if (i < BH) {
    state[i * 8 + 0] = 0u;
    state[i * 8 + 1] = 0u;
    state[i * 8 + 2] = keep;
    state[i * 8 + 3] = 0u;
    state[i * 8 + 4] = 0u;
  }
}

__global__ void __launch_bounds__(256) sel_hist_kernel(const float* __restrict__ pr, long long n_elems,
                                                       const unsigned* __restrict__ state, unsigned* hist, int pass) {
  __shared__ unsigned sh[kHistBins];
  const int bh = blockIdx.y;
  for (int i = threadIdx.x; i < kHistBins; i += blockDim.x) sh[i] = 0u;
  __syncthreads();
  const unsigned prefix = state[bh * 8 + 0], pmask = state[bh * 8 + 1];
  const int shift = seq_shift(pass);
  const unsigned dmask = seq_mask(pass);
  const unsigned* src = reinterpret_cast<const unsigned*>(pr) + (size_t)bh * n_elems;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x, nthr = (long long)gridDim.x * blockDim.x;
  long long done = 0;
  if ((n_elems & 3) == 0) {
    // 16-byte loads, two in flight per thread (the passes after the first count almost nothing: they are pure streaming reads)
    const uint4* src4 = reinterpret_cast<const uint4*>(src);
    const long long n4 = n_elems >> 2;
    for (long long i = tid; i < n4; i += 2 * nthr) {
      const uint4 a = __ldg(src4 + i);
      const bool two = i + nthr < n4;
      const uint4 b = two ? __ldg(src4 + i + nthr) : make_uint4(0, 0, 0, 0);
      const unsigned va[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if ((e < 4 || two) && (va[e] & pmask) == prefix) atomicAdd(&sh[(va[e] >> shift) & dmask], 1u);
    }
    done = n_elems;
  }
  for (long long i = done + tid; i < n_elems; i += nthr) {
    unsigned v = __ldg(src + i);
    if ((v & pmask) == prefix) atomicAdd(&sh[(v >> shift) & dmask], 1u);
  }
  __syncthreads();
  unsigned* dst = hist + ((size_t)bh * 3 + pass) * kHistBins;
  for (int i = threadIdx.x; i < kHistBins; i += blockDim.x)
    if (sh[i]) atomicAdd(&dst[i], sh[i]);
}

// One warp per (batch, head): finds the digit whose bin holds the `remaining`-th largest entry.  Lane l owns the bins
// [l * nb/32, (l+1) * nb/32); a suffix sum over the lanes locates the lane, a short serial walk the bin.
__global__ void __launch_bounds__(32) sel_pick_kernel(unsigned* state, const unsigned* hist, int pass) {
  const int bh = blockIdx.x, lane = threadIdx.x;
  const unsigned* hsrc = hist + ((size_t)bh * 3 + pass) * kHistBins;
  const unsigned remaining0 = state[bh * 8 + 2];
  const int nb = (int)seq_mask(pass) + 1, per = nb / 32;
  unsigned mine = 0u;
  for (int d = lane * per; d < (lane + 1) * per; ++d) mine += hsrc[d];
  // above = entries in the bins of all higher lanes
  unsigned incl = mine;
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned up = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += up;
  }
  const unsigned above = incl - mine;
  // the threshold bin lies in the highest lane whose suffix count reaches `remaining0`
  const bool here = above < remaining0 && incl >= remaining0;
  const unsigned vote = __ballot_sync(0xffffffffu, here);
  if (vote == 0u) {                    // fewer entries than requested (cannot happen for keep <= N*N): keep everything
    if (lane == 0) {
      const int shift = seq_shift(pass);
      state[bh * 8 + 1] |= seq_mask(pass) << shift;
      state[bh * 8 + 2] = remaining0 - incl;      // lane 0's inclusive suffix = all entries
      if (pass == 2) { state[bh * 8 + 3] = state[bh * 8 + 0]; state[bh * 8 + 4] = state[bh * 8 + 2]; }
    }
    return;
  }
  if (lane == 31 - __clz(vote)) {
    unsigned remaining = remaining0 - above;
    int bin = lane * per;
    for (int d = (lane + 1) * per - 1; d >= lane * per; --d) {
      const unsigned c = hsrc[d];
      if (c >= remaining) { bin = d; break; }
      remaining -= c;
    }
    const int shift = seq_shift(pass);
    const unsigned prefix = state[bh * 8 + 0] | ((unsigned)bin << shift);
    state[bh * 8 + 0] = prefix;
    state[bh * 8 + 1] |= seq_mask(pass) << shift;
    state[bh * 8 + 2] = remaining;
    if (pass == 2) {
      state[bh * 8 + 3] = prefix;      // tau: the smallest kept value
      state[bh * 8 + 4] = remaining;   // how many entries equal to tau are kept
    }
  }
}

// per-sequence, one read of P_r for both the counts and the emission: one warp per row writes the row's bitmap words of the
// entries above tau (`bits_gt`) and equal to tau (`bits_eq`) and the two counts.  grid (ceil(N/8), BH), 256 threads
__global__ void __launch_bounds__(256) sel_row_bits_kernel(const float* __restrict__ pr, int N, int words,
                                                           const unsigned* __restrict__ state, unsigned* bits_gt,
                                                           unsigned* bits_eq, int* row_gt, int* row_eq) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int bh = blockIdx.y;
  if (i >= N) return;
  const unsigned tau = state[bh * 8 + 3];
  const unsigned* src = reinterpret_cast<const unsigned*>(pr) + ((size_t)bh * N + i) * N;
  int gt = 0, eq = 0;
  constexpr int U = 8;                 // words in flight per warp (the kernel is a pure streaming read)
  for (int w0 = 0; w0 < words; w0 += U) {
    unsigned v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int j = (w0 + u) * 32 + lane;
      v[u] = j < N ? __ldg(src + j) : 0u;      // (scores are non-negative: 0 is never above tau, and equal only if tau = 0
    }                                          //  -- excluded by the j < N test below)
    unsigned mine_g = 0u, mine_e = 0u;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int j = (w0 + u) * 32 + lane;
      const unsigned gb = __ballot_sync(0xffffffffu, j < N && v[u] > tau);
      const unsigned eb = __ballot_sync(0xffffffffu, j < N && v[u] == tau);
      if (lane == u) { mine_g = gb; mine_e = eb; }
      gt += __popc(gb);
      eq += __popc(eb);
    }
    if (lane < U && w0 + lane < words) {       // lanes 0..U-1 write one word each: consecutive addresses
      bits_gt[((size_t)bh * N + i) * words + w0 + lane] = mine_g;
      bits_eq[((size_t)bh * N + i) * words + w0 + lane] = mine_e;
    }
  }
  if (lane == 0) {
    row_gt[(size_t)bh * N + i] = gt;
    row_eq[(size_t)bh * N + i] = eq;
  }
}

// inclusive prefix sum over the lanes of a warp
__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// per-sequence: ordered emission of the kept columns from the two bitmaps (`bitmap` holds the entries above tau on entry and
// the kept entries on return).  One warp per row, one LANE per bitmap word: the lanes count their bits, a warp scan gives every
// word its position in the row's list, and each lane writes its own few entries (a warp per word spent 30 instructions on
// every word, 45 words a row).  Ties at tau go to the lower column: a lane keeps the equal entries whose rank in the row is
// below the row's quota.  grid (ceil(N/8), BH), 256 threads
__global__ void __launch_bounds__(256) sel_emit_rows_bits_kernel(int N, int words, const unsigned* __restrict__ bits_eq,
                                                                 const int* __restrict__ row_eq_take,
                                                                 const int* __restrict__ row_ptr, int* col_idx,
                                                                 unsigned* bitmap, long long nnz_cap) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int bh = blockIdx.y;
  if (i >= N) return;
  const int take = row_eq_take[(size_t)bh * N + i];
  int pos = row_ptr[(size_t)bh * (N + 1) + i];
  int eq_seen = 0;
  int* out = col_idx + (size_t)bh * nnz_cap;
  const size_t base = ((size_t)bh * N + i) * words;
  for (int w0 = 0; w0 < words; w0 += 32) {
    const int w = w0 + lane;
    const unsigned gb = w < words ? bitmap[base + w] : 0u;
    unsigned eb = w < words ? __ldg(bits_eq + base + w) : 0u;
    const int ce = __popc(eb);
    const int ce_incl = warp_incl_scan(ce, lane);
    int rank = eq_seen + ce_incl - ce;             // equal entries of the row before this word
    unsigned keep = 0u;
    while (eb != 0u && rank < take) {
      keep |= eb & (0u - eb);
      eb &= eb - 1u;
      ++rank;
    }
    unsigned sel = gb | keep;
    const int c = __popc(sel);
    const int c_incl = warp_incl_scan(c, lane);
    int p = pos + c_incl - c;
    unsigned kept = 0u;                              // (entries past the capacity of the map are dropped from the bitmap too,
    while (sel != 0u) {                              //  so that the transposed map lists exactly the pairs emitted here)
      if (p < nnz_cap) {
        out[p] = w * 32 + (__ffs(sel) - 1);
        kept |= sel & (0u - sel);
      }
      sel &= sel - 1u;
      ++p;
    }
    if (w < words && kept != gb) bitmap[base + w] = kept;
    pos += __shfl_sync(0xffffffffu, c_incl, 31);
    eq_seen += __shfl_sync(0xffffffffu, ce_incl, 31);
  }
}

// per-row modes: radix select of the k_i-th largest of row i.  grid (N, BH), 256 threads
__global__ void __launch_bounds__(256) sel_row_topk_kernel(const float* __restrict__ pr, int N, int K,
                                                           const int* __restrict__ budgets, float* row_tau,
                                                           int* row_eq_take, int* row_cnt) {
  __shared__ unsigned sh[256];
  __shared__ unsigned s_prefix, s_mask, s_remaining;
  const int i = blockIdx.x, bh = blockIdx.y;
  const unsigned* src = reinterpret_cast<const unsigned*>(pr) + ((size_t)bh * N + i) * N;
  int k = budgets ? budgets[(size_t)bh * N + i] : K;
  k = max(0, min(k, N));
  const size_t o = (size_t)bh * N + i;
  if (k == 0) {
    if (threadIdx.x == 0) { row_tau[o] = INFINITY; row_eq_take[o] = 0; row_cnt[o] = 0; }
    return;
  }
  if (threadIdx.x == 0) { s_prefix = 0u; s_mask = 0u; s_remaining = (unsigned)k; }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    sh[threadIdx.x] = 0u;
    __syncthreads();
    const unsigned prefix = s_prefix, pmask = s_mask;
    for (int j = threadIdx.x; j < N; j += blockDim.x) {
      unsigned v = __ldg(src + j);
      if ((v & pmask) == prefix) atomicAdd(&sh[(v >> shift) & 0xFFu], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned remaining = s_remaining;
      int bin = 0;
      for (int d = 255; d >= 0; --d) {
        unsigned c = sh[d];
        if (c >= remaining) { bin = d; break; }
        remaining -= c;
      }
      s_prefix = prefix | ((unsigned)bin << shift);
      s_mask = pmask | (0xFFu << shift);
      s_remaining = remaining;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    row_tau[o] = __uint_as_float(s_prefix);
    row_eq_take[o] = (int)s_remaining;
    row_cnt[o] = k;
  }
}

// exclusive scan of v over the block (1024 threads); returns the prefix, total in `total`
__device__ __forceinline__ int block_excl_scan(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
    int wi = w;
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    warp_sums[lane] = wi - w;        // exclusive prefix of the warp sums
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  int res = warp_sums[warp] + incl - v;
  total = warp_sums[32];
  __syncthreads();
  return res;
}

// one block per (batch, head): per-sequence tie quota per row, then row_ptr = exclusive scan of counts
__global__ void __launch_bounds__(1024) sel_scan_rows_kernel(int N, int per_sequence, const unsigned* __restrict__ state,
                                                             const int* __restrict__ row_gt, const int* __restrict__ row_eq,
                                                             float* row_tau, int* row_eq_take, int* row_cnt, int* row_ptr,
                                                             long long nnz_cap, StatusBlock* status) {
  __shared__ int ws[33];
  const int bh = blockIdx.x;
  const size_t base = (size_t)bh * N;
  if (per_sequence) {
    const unsigned tau = state[bh * 8 + 3];
    const int quota = (int)state[bh * 8 + 4];
    int carry = 0;
    for (int i0 = 0; i0 < N; i0 += blockDim.x) {
      int i = i0 + threadIdx.x;
      int eq = i < N ? row_eq[base + i] : 0;
      int tot;
      int before = carry + block_excl_scan(eq, ws, tot);
      if (i < N) {
        int take = max(0, min(eq, quota - before));
        row_eq_take[base + i] = take;
        row_cnt[base + i] = row_gt[base + i] + take;
        row_tau[base + i] = __uint_as_float(tau);
      }
      carry += tot;
    }
    __syncthreads();
  }
  int carry = 0;
  for (int i0 = 0; i0 < N; i0 += blockDim.x) {
    int i = i0 + threadIdx.x;
    int c = i < N ? row_cnt[base + i] : 0;
    int tot;
    int pre = carry + block_excl_scan(c, ws, tot);
    // (an overflowing selection is reported below; its row pointers stop at the capacity, so that every later reader of
    // the map stays inside col_idx: rows past the capacity are empty, the row that crosses it is cut)
    if (i < N) row_ptr[(size_t)bh * (N + 1) + i] = (int)min((long long)pre, nnz_cap);
    carry += tot;
  }
  if (threadIdx.x == 0) {
    row_ptr[(size_t)bh * (N + 1) + N] = (int)min((long long)carry, nnz_cap);
    if ((long long)carry > nnz_cap) atomicExch(&status->status, VSA2_ERR_MAP_OVERFLOW);
  }
}

// one warp per row: ordered emission of the kept columns and of the row's bitmap words
__global__ void __launch_bounds__(256) sel_emit_rows_kernel(const float* __restrict__ pr, int N, int words,
                                                            const float* __restrict__ row_tau,
                                                            const int* __restrict__ row_eq_take,
                                                            const int* __restrict__ row_ptr, int* col_idx,
                                                            unsigned* bitmap, long long nnz_cap) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int bh = blockIdx.y;
  if (i >= N) return;
  const unsigned* src = reinterpret_cast<const unsigned*>(pr) + ((size_t)bh * N + i) * N;
  const unsigned tau = __float_as_uint(row_tau[(size_t)bh * N + i]);
  const int take = row_eq_take[(size_t)bh * N + i];
  int pos = row_ptr[(size_t)bh * (N + 1) + i];
  int eq_seen = 0;
  int* out = col_idx + (size_t)bh * nnz_cap;
  const unsigned lt = (1u << lane) - 1u;
  for (int w = 0; w < words; ++w) {
    int j = w * 32 + lane;
    unsigned v = j < N ? __ldg(src + j) : 0u;
    bool gt = j < N && v > tau;
    bool eq = j < N && v == tau;
    unsigned eqb = __ballot_sync(0xffffffffu, eq);
    bool sel = gt || (eq && (eq_seen + __popc(eqb & lt)) < take);
    unsigned selb = __ballot_sync(0xffffffffu, sel);
    const int p = pos + __popc(selb & lt);
    const bool emit = sel && p < nnz_cap;            // (entries past the capacity of the map are dropped from the bitmap too,
    if (emit) out[p] = j;                            //  so that the transposed map lists exactly the pairs emitted here)
    const unsigned keptb = __ballot_sync(0xffffffffu, emit);
    pos += __popc(selb);
    eq_seen += __popc(eqb);
    if (lane == 0) bitmap[((size_t)bh * N + i) * words + w] = keptb;
  }
}

// bitmap [BH][N rows][words] -> bitmap_t [BH][N columns][words] (bit i of row-word set <-> bit of column-word set):
// one warp per 32 x 32 bit tile, transposed with 32 ballots.  grid (words, ceil(words/8), BH), 256 threads
__global__ void __launch_bounds__(256) sel_transpose_bitmap_kernel(const unsigned* __restrict__ bitmap, int N, int words,
                                                                   unsigned* __restrict__ bitmap_t) {
  const int lane = threadIdx.x & 31;
  const int wj = blockIdx.x;                                   // word column of the source: columns 32 wj .. 32 wj + 31
  const int wi = blockIdx.y * 8 + (threadIdx.x >> 5);          // word row of the source: rows 32 wi .. 32 wi + 31
  const int bh = blockIdx.z;
  if (wi >= words) return;
  const int i = wi * 32 + lane;
  const unsigned v = i < N ? __ldg(bitmap + ((size_t)bh * N + i) * words + wj) : 0u;
  unsigned mine = 0u;
#pragma unroll
  for (int bit = 0; bit < 32; ++bit) {
    const unsigned col_word = __ballot_sync(0xffffffffu, (v >> bit) & 1u);   // rows 32 wi .. of column 32 wj + bit
    if (lane == bit) mine = col_word;
  }
  const int j = wj * 32 + lane;
  if (j < N) bitmap_t[((size_t)bh * N + j) * words + wi] = mine;
}

// one warp per column: number of kept rows.  grid (ceil(N/8), BH), 256 threads
__global__ void __launch_bounds__(256) sel_col_count_kernel(const unsigned* __restrict__ bitmap_t, int N, int words,
                                                            int* col_cnt) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5), bh = blockIdx.y;
  if (j >= N) return;
  const unsigned* bm = bitmap_t + ((size_t)bh * N + j) * words;
  int c = 0;
  for (int w = lane; w < words; w += 32) c += __popc(__ldg(bm + w));
  for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if (lane == 0) col_cnt[(size_t)bh * N + j] = c;
}

__global__ void __launch_bounds__(1024) sel_scan_cols_kernel(int N, const int* __restrict__ col_cnt, int* col_ptr,
                                                             long long nnz_cap) {
  __shared__ int ws[33];
  const int bh = blockIdx.x;
  int carry = 0;
  for (int j0 = 0; j0 < N; j0 += blockDim.x) {
    int j = j0 + threadIdx.x;
    int c = j < N ? col_cnt[(size_t)bh * N + j] : 0;
    int tot;
    int pre = carry + block_excl_scan(c, ws, tot);
    if (j < N) col_ptr[(size_t)bh * (N + 1) + j] = (int)min((long long)pre, nnz_cap);      // (as for the rows)
    carry += tot;
  }
  if (threadIdx.x == 0) col_ptr[(size_t)bh * (N + 1) + N] = (int)min((long long)carry, nnz_cap);
}

// one warp per column, one lane per bitmap word: ordered emission of the rows that keep it.  grid (ceil(N/8), BH), 256 threads
__global__ void __launch_bounds__(256) sel_emit_cols_kernel(const unsigned* __restrict__ bitmap_t, int N, int words,
                                                            const int* __restrict__ col_ptr, int* row_idx,
                                                            long long nnz_cap) {
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5), bh = blockIdx.y;
  if (j >= N) return;
  const unsigned* bm = bitmap_t + ((size_t)bh * N + j) * words;
  int pos = col_ptr[(size_t)bh * (N + 1) + j];
  int* out = row_idx + (size_t)bh * nnz_cap;
  for (int w0 = 0; w0 < words; w0 += 32) {
    // one lane per word, as in sel_emit_rows_bits_kernel
    unsigned word = w0 + lane < words ? __ldg(bm + w0 + lane) : 0u;
    const int c = __popc(word);
    const int c_incl = warp_incl_scan(c, lane);
    int p = pos + c_incl - c;
    while (word != 0u) {
      if (p < nnz_cap) out[p] = (w0 + lane) * 32 + (__ffs(word) - 1);
      word &= word - 1u;
      ++p;
    }
    pos += __shfl_sync(0xffffffffu, c_incl, 31);
  }
}

cudaError_t launch_select(const Geo& g, const float* pr, const int* budgets, const SelectScratch& s, int* row_ptr,
                          int* col_idx, int* col_ptr, int* row_idx, StatusBlock* status, cudaStream_t st) {
  const int BH = g.batch * g.Hq, N = g.N;
  const long long n_elems = (long long)N * N;
  if (g.mode == VSA2_PER_SEQUENCE) {
    const unsigned keep = (unsigned)((long long)N * g.K);
    int init_n = BH * 3 * kHistBins;
    sel_init_kernel<<<(init_n + 255) / 256, 256, 0, st>>>(s.state, s.hist, BH, keep);
    int chunks = (int)((n_elems + 256 * 16 - 1) / (256 * 16));
    if (chunks > 256) chunks = 256;
    for (int pass = 0; pass < 3; ++pass) {
      sel_hist_kernel<<<dim3(chunks, BH), 256, 0, st>>>(pr, n_elems, s.state, s.hist, pass);
      sel_pick_kernel<<<BH, 32, 0, st>>>(s.state, s.hist, pass);
    }
    // counts and bitmaps in one read of P_r (the bitmap of the entries equal to tau borrows the transposed bitmap's space)
    sel_row_bits_kernel<<<dim3((N + 7) / 8, BH), 256, 0, st>>>(pr, N, s.words, s.state, s.bitmap, s.bitmap_t, s.row_gt, s.row_eq);
  } else {
    sel_row_topk_kernel<<<dim3(N, BH), 256, 0, st>>>(pr, N, g.K, g.mode == VSA2_PER_QUERY_BUDGET ? budgets : nullptr,
                                                     s.row_tau, s.row_eq_take, s.row_cnt);
  }
  sel_scan_rows_kernel<<<BH, 1024, 0, st>>>(N, g.mode == VSA2_PER_SEQUENCE, s.state, s.row_gt, s.row_eq, s.row_tau,
                                            s.row_eq_take, s.row_cnt, row_ptr, g.nnz_cap, status);
  if (g.mode == VSA2_PER_SEQUENCE)
    sel_emit_rows_bits_kernel<<<dim3((N + 7) / 8, BH), 256, 0, st>>>(N, s.words, s.bitmap_t, s.row_eq_take, row_ptr, col_idx,
                                                                     s.bitmap, g.nnz_cap);
  else
    sel_emit_rows_kernel<<<dim3((N + 7) / 8, BH), 256, 0, st>>>(pr, N, s.words, s.row_tau, s.row_eq_take, row_ptr,
                                                                col_idx, s.bitmap, g.nnz_cap);
  // columns: transposed bitmap, then counts (row_gt reused as scratch), scan, ordered emission
  sel_transpose_bitmap_kernel<<<dim3(s.words, (s.words + 7) / 8, BH), 256, 0, st>>>(s.bitmap, N, s.words, s.bitmap_t);
  sel_col_count_kernel<<<dim3((N + 7) / 8, BH), 256, 0, st>>>(s.bitmap_t, N, s.words, s.row_gt);
  sel_scan_cols_kernel<<<BH, 1024, 0, st>>>(N, s.row_gt, col_ptr, g.nnz_cap);
  sel_emit_cols_kernel<<<dim3((N + 7) / 8, BH), 256, 0, st>>>(s.bitmap_t, N, s.words, col_ptr, row_idx, g.nnz_cap);
  return cudaGetLastError();
}

}  // namespace vsa2
