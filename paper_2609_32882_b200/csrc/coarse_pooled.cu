// Coarse branch (paper Eq. 2-3) and its backward on the Blackwell tensor cores, by running the fine-branch kernels on the
// POOLED grid: the N = Nt x Nh x Nw cube means form a small (Nt, Nh, Nw) token grid of their own, in raster order,
// and dense attention over them is block-sparse attention with every block selected.  The pooled fp32 means are
// rounded to bf16 (the precision of the model's other attention operands), the outputs stay fp32.
// This file holds the glue: the pooled problem's geometry, the dense block map, the casts and the launch sequence.
#include "common.cuh"

namespace vsa2 {

// geometry of the pooled problem: tokens = cubes of g, cubes of 4 x 4 x 4 pooled tokens, every block selected
Geo pooled_geo(const Geo& g) {
  Geo p = wide_cube(g) ? narrow_geo(g) : g;      // the kernels' blocks are 64 pooled tokens whatever the caller's cube
  p.T = g.Nt; p.H = g.Nh; p.W = g.Nw;
  p.L = g.N;
  p.Nt = (p.T + p.Bt - 1) / p.Bt; p.Nh = (p.H + p.Bh - 1) / p.Bh; p.Nw = (p.W + p.Bw - 1) / p.Bw;
  p.N = p.Nt * p.Nh * p.Nw;
  geo_set_magics(p);
  p.Nvid = p.N; p.Lt = 0; p.S = p.L;
  p.K = p.N;
  p.mode = VSA2_PER_QUERY;
  p.out_f32 = 1;
  p.flags = VSA2_FLAG_NO_COARSE;
  p.nnz_cap = (long long)p.N * p.N;
  return p;
}

PooledLayout pooled_layout(const Geo& g, bool backward) {
  const Geo p = pooled_geo(g);
  PooledLayout r;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t BHq = (size_t)g.batch * g.Hq, BHk = (size_t)g.batch * g.Hkv;
  r.status = take(fine_fwd_tc_workspace_bytes());
  r.q16 = take(BHq * g.N * g.D * sizeof(bf16));
  r.k16 = take(BHk * g.N * g.D * sizeof(bf16));
  r.v16 = take(BHk * g.N * g.D * sizeof(bf16));
  r.ptr = take(BHq * (p.N + 1) * sizeof(int));
  r.idx = take(BHq * (size_t)p.N * p.N * sizeof(int));
  r.do16 = r.delta = r.dk_kv = r.dv_kv = 0;
  if (backward) {
    r.do16 = take(BHq * g.N * g.D * sizeof(bf16));
    r.delta = take(BHq * g.N * sizeof(float));
    r.dk_kv = take(BHk * g.N * g.D * sizeof(float));
    r.dv_kv = take(BHk * g.N * g.D * sizeof(float));
  }
  r.total = off;
  return r;
}

__global__ void cast_f32_to_bf16_kernel(const float* __restrict__ x, bf16* __restrict__ y, size_t n4) {
  const size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4 v = __ldg(reinterpret_cast<const float4*>(x) + i);
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<uint32_t*>(&a);
  o.y = *reinterpret_cast<uint32_t*>(&b);
  reinterpret_cast<uint2*>(y)[i] = o;
}

static cudaError_t cast_to_bf16(const float* x, bf16* y, size_t n, cudaStream_t st) {
  const size_t n4 = n / 4;      // n is a multiple of the head dimension
  cast_f32_to_bf16_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(x, y, n4);
  return cudaGetLastError();
}

// dense map of np blocks for `heads` lists: ptr[h][i] = i * np, idx[h][i * np + j] = j (its transpose is the same map)
__global__ void dense_map_kernel(int* __restrict__ ptr, int* __restrict__ idx, int np, int heads) {
  const int h = blockIdx.x;
  if (h >= heads) return;
  for (int i = threadIdx.x; i <= np; i += blockDim.x) ptr[(size_t)h * (np + 1) + i] = i * np;
  for (int e = threadIdx.x; e < np * np; e += blockDim.x) idx[(size_t)h * np * np + e] = e % np;
}

// the recursive dK/dV pass returns one gradient per KV head; the epilogues of the main passes sum dK_c, dV_c over the
// query heads of a group, so the result goes to the group's first query head and zeros to the others
__global__ void spread_to_group_kernel(const float* __restrict__ x_kv, float* __restrict__ x_q, int rep, size_t per_head4,
                                       int heads_q) {
  const size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  const int hq = blockIdx.y;            // b * Hq + hq (Hq = Hkv * rep, so b * Hq + hq = (b * Hkv + hk) * rep + hh)
  if (i >= per_head4 || hq >= heads_q) return;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (hq % rep == 0) v = __ldg(reinterpret_cast<const float4*>(x_kv) + (size_t)(hq / rep) * per_head4 + i);
  reinterpret_cast<float4*>(x_q)[(size_t)hq * per_head4 + i] = v;
}

// The pooled passes count their work items in a status block of their own (inside the scratch region); a non-zero
// status word there (a bounded wait that ran out, a rescue list that overflowed) is copied into the caller's status word,
// which is the one vsa2_device_status reads.
__global__ void merge_status_kernel(const StatusBlock* __restrict__ from, StatusBlock* __restrict__ into) {
  const int s = from->status;
  if (s != 0) atomicCAS(&into->status, 0, s);
}

cudaError_t launch_coarse_fwd_pooled(const Geo& g, const float* qc, const float* kc, const float* vc, float* oc_hat,
                                     float* lse_c, void* workspace, StatusBlock* caller_status, cudaStream_t st) {
  const Geo p = pooled_geo(g);
  const PooledLayout lay = pooled_layout(g, false);
  unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
  const size_t BHq = (size_t)g.batch * g.Hq, BHk = (size_t)g.batch * g.Hkv;
  bf16* q16 = reinterpret_cast<bf16*>(ws + lay.q16);
  bf16* k16 = reinterpret_cast<bf16*>(ws + lay.k16);
  bf16* v16 = reinterpret_cast<bf16*>(ws + lay.v16);
  int* ptr = reinterpret_cast<int*>(ws + lay.ptr);
  int* idx = reinterpret_cast<int*>(ws + lay.idx);
  cudaError_t e;
  if ((e = cudaMemsetAsync(ws + lay.status, 0, sizeof(StatusBlock), st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(qc, q16, BHq * g.N * g.D, st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(kc, k16, BHk * g.N * g.D, st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(vc, v16, BHk * g.N * g.D, st)) != cudaSuccess) return e;
  dense_map_kernel<<<(unsigned)BHq, 256, 0, st>>>(ptr, idx, p.N, (int)BHq);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  if ((e = launch_fine_fwd_tc(p, q16, k16, v16, nullptr, ptr, idx, nullptr, oc_hat, nullptr, lse_c,
                              reinterpret_cast<StatusBlock*>(ws + lay.status), st)) != cudaSuccess)
    return e;
  merge_status_kernel<<<1, 1, 0, st>>>(reinterpret_cast<const StatusBlock*>(ws + lay.status), caller_status);
  return cudaGetLastError();
}

cudaError_t launch_coarse_bwd_pooled(const Geo& g, const float* qc, const float* kc, const float* vc, const float* oc_hat,
                                     const float* lse_c, const float* d_oc_hat, float* dqc, float* dkc, float* dvc,
                                     void* workspace, StatusBlock* caller_status, cudaStream_t st) {
  const Geo p = pooled_geo(g);
  const PooledLayout lay = pooled_layout(g, true);
  unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
  const size_t BHq = (size_t)g.batch * g.Hq, BHk = (size_t)g.batch * g.Hkv;
  bf16* q16 = reinterpret_cast<bf16*>(ws + lay.q16);
  bf16* k16 = reinterpret_cast<bf16*>(ws + lay.k16);
  bf16* v16 = reinterpret_cast<bf16*>(ws + lay.v16);
  bf16* do16 = reinterpret_cast<bf16*>(ws + lay.do16);
  int* ptr = reinterpret_cast<int*>(ws + lay.ptr);
  int* idx = reinterpret_cast<int*>(ws + lay.idx);
  float* delta = reinterpret_cast<float*>(ws + lay.delta);
  float* dk_kv = reinterpret_cast<float*>(ws + lay.dk_kv);
  float* dv_kv = reinterpret_cast<float*>(ws + lay.dv_kv);
  StatusBlock* status = reinterpret_cast<StatusBlock*>(ws + lay.status);
  cudaError_t e;
  if ((e = cudaMemsetAsync(status, 0, sizeof(StatusBlock), st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(qc, q16, BHq * g.N * g.D, st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(kc, k16, BHk * g.N * g.D, st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(vc, v16, BHk * g.N * g.D, st)) != cudaSuccess) return e;
  if ((e = cast_to_bf16(d_oc_hat, do16, BHq * g.N * g.D, st)) != cudaSuccess) return e;
  dense_map_kernel<<<(unsigned)BHq, 256, 0, st>>>(ptr, idx, p.N, (int)BHq);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // delta_c = rowsum(dO_c * O_c) through the preprocess kernel of the pooled problem (no gate: only delta is written)
  if ((e = launch_bwd_preprocess(p, do16, oc_hat, nullptr, nullptr, nullptr, delta, nullptr, nullptr, st)) != cudaSuccess) return e;
  if ((e = launch_fine_bwd_dq_tc(p, q16, k16, v16, do16, lse_c, delta, ptr, idx, nullptr, dqc, status, st, nullptr, nullptr)) != cudaSuccess) return e;
  const bool grouped = g.rep > 1;
  if ((e = launch_fine_bwd_dkv_tc(p, q16, k16, v16, do16, lse_c, delta, ptr, idx, nullptr, nullptr, grouped ? dk_kv : dkc,
                                  grouped ? dv_kv : dvc, status, st, false, nullptr, nullptr, nullptr, nullptr, nullptr)) != cudaSuccess)
    return e;
  if (grouped) {
    const size_t per_head4 = (size_t)g.N * g.D / 4;
    dim3 grid((unsigned)((per_head4 + 255) / 256), (unsigned)BHq);
    spread_to_group_kernel<<<grid, 256, 0, st>>>(dk_kv, dkc, g.rep, per_head4, (int)BHq);
    spread_to_group_kernel<<<grid, 256, 0, st>>>(dv_kv, dvc, g.rep, per_head4, (int)BHq);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  merge_status_kernel<<<1, 1, 0, st>>>(status, caller_status);
  return cudaGetLastError();
}

}  // namespace vsa2
