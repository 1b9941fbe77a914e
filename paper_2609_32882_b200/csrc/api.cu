// C ABI of the VSA2 library: argument checks, workspace layout, kernel sequencing.
#include <math.h>
#include <string.h>

#include <atomic>

#include "common.cuh"

using namespace vsa2;

namespace {

cudaEvent_t g_prof_start[VSA2_KERNEL_COUNT];
cudaEvent_t g_prof_stop[VSA2_KERNEL_COUNT];
std::atomic<long long> g_launches{0};

struct RouteLayout {
  size_t status, qr, kr, lse_r, pr, hist, state, row_tau, row_eq_take, row_cnt, row_gt, row_eq, bitmap, bitmap_t, total;
  int words;
};
struct BwdLayout {
  size_t status, delta, d_oc_hat, delta_c, dqc, dkc, dvc, pooled, total;
};

struct Carver {
  size_t off = 0;
  size_t take(size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  }
};

int fill_geo(const vsa2_params* p, Geo* g) {
  if (p == nullptr) return VSA2_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->heads_q <= 0 || p->heads_kv <= 0 || p->grid_t <= 0 || p->grid_h <= 0 || p->grid_w <= 0 ||
      p->cube_t <= 0 || p->cube_h <= 0 || p->cube_w <= 0 || p->rpool_t <= 0 || p->rpool_h <= 0 || p->rpool_w <= 0)
    return VSA2_ERR_INVALID_ARG;
  if (p->heads_q % p->heads_kv) return VSA2_ERR_INVALID_ARG;
  if (p->select_mode < VSA2_PER_SEQUENCE || p->select_mode > VSA2_PER_QUERY_BUDGET) return VSA2_ERR_INVALID_ARG;
  if (p->out_dtype != VSA2_BF16 && p->out_dtype != VSA2_F32) return VSA2_ERR_INVALID_ARG;
  if (p->topk < 0 || p->nnz_cap < 0 || !(p->softmax_scale >= 0.f) || p->text_len < 0) return VSA2_ERR_INVALID_ARG;
  if (p->cube_t % p->rpool_t || p->cube_h % p->rpool_h || p->cube_w % p->rpool_w) return VSA2_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return VSA2_ERR_UNSUPPORTED;
  // 64-token cubes, or 128-token cubes that split along w into two 64-token halves the router pooling respects
  const long long cube_tokens = (long long)p->cube_t * p->cube_h * p->cube_w;
  const bool wide = cube_tokens == 2 * kBlockTokens;
  if (cube_tokens != kBlockTokens && !wide) return VSA2_ERR_UNSUPPORTED;
  if (wide && (p->cube_w % 2 || (p->cube_w / 2) % p->rpool_w)) return VSA2_ERR_UNSUPPORTED;
  if (p->batch > 65535 || p->heads_q > 65535 || p->heads_q / p->heads_kv > 16) return VSA2_ERR_UNSUPPORTED;
  g->batch = p->batch; g->Hq = p->heads_q; g->Hkv = p->heads_kv; g->rep = p->heads_q / p->heads_kv; g->D = p->head_dim;
  g->T = p->grid_t; g->H = p->grid_h; g->W = p->grid_w;
  long long L = (long long)g->T * g->H * g->W;
  if (L + p->text_len > 0x7fffffffLL / 128) return VSA2_ERR_UNSUPPORTED;
  g->L = (int)L;
  g->Lt = p->text_len;
  g->S = (int)L + p->text_len;
  g->Bt = p->cube_t; g->Bh = p->cube_h; g->Bw = p->cube_w;
  g->Nt = (g->T + g->Bt - 1) / g->Bt; g->Nh = (g->H + g->Bh - 1) / g->Bh; g->Nw = (g->W + g->Bw - 1) / g->Bw;
  g->N = g->Nt * g->Nh * g->Nw;
  geo_set_magics(*g);
  g->Nvid = g->N;
  g->Rt = p->rpool_t; g->Rh = p->rpool_h; g->Rw = p->rpool_w;
  g->Gt = g->Bt / g->Rt; g->Gh = g->Bh / g->Rh; g->Gw = g->Bw / g->Rw;
  g->G = g->Gt * g->Gh * g->Gw;
  if (128 % (wide ? g->G / 2 : g->G)) return VSA2_ERR_UNSUPPORTED;
  int K = p->topk;
  if (K == 0) {
    if (!(p->keep_fraction > 0.f) || p->keep_fraction > 1.f) {
      if (p->select_mode != VSA2_PER_QUERY_BUDGET) return VSA2_ERR_INVALID_ARG;
      K = 1;
    } else {
      K = (int)lroundf(p->keep_fraction * (float)g->N);
      if (K < 1) K = 1;
    }
  }
  if (K > g->N) K = g->N;
  g->K = K;
  g->mode = p->select_mode;
  g->out_f32 = p->out_dtype == VSA2_F32;
  g->flags = p->flags;
  g->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)g->D);
  if (p->nnz_cap > 0) g->nnz_cap = p->nnz_cap;
  else if (p->select_mode == VSA2_PER_QUERY_BUDGET) return VSA2_ERR_INVALID_ARG;
  else g->nnz_cap = (long long)g->N * K;
  return VSA2_OK;
}

// Block problem of the fine kernels with text tokens: the N video cubes followed by ceil(Lt / 64) text blocks; its maps
// are the video maps with the text blocks appended to every row and one dense row per text block.
int text_blocks(const Geo& g) { return (g.Lt + kBlockTokens - 1) / kBlockTokens; }
Geo text_geo(const Geo& g) {
  Geo x = g;
  const int tb = text_blocks(g);
  x.N = g.Nvid + tb;
  x.nnz_cap = g.nnz_cap + (long long)g.Nvid * tb + (long long)tb * x.N;
  return x;
}
struct TextMapLayout {
  size_t ptr, idx, cptr, ridx, total;     // offsets behind the call's other workspace regions
};
TextMapLayout text_map_layout(const Geo& g, bool with_csc) {
  TextMapLayout r = {};
  if (g.Lt == 0) return r;
  const Geo x = text_geo(wide_cube(g) ? narrow_geo(g) : g);      // (128-token cubes: the block problem of the half-cubes)
  Carver c;
  const size_t BHq = (size_t)g.batch * g.Hq;
  r.ptr = c.take(BHq * (x.N + 1) * sizeof(int));
  r.idx = c.take(BHq * (size_t)x.nnz_cap * sizeof(int));
  if (with_csc) {
    r.cptr = c.take(BHq * (x.N + 1) * sizeof(int));
    r.ridx = c.take(BHq * (size_t)x.nnz_cap * sizeof(int));
  }
  r.total = c.off;
  return r;
}

RouteLayout route_layout(const Geo& g) {
  RouteLayout r;
  Carver c;
  const size_t BHq = (size_t)g.batch * g.Hq, BHk = (size_t)g.batch * g.Hkv, NG = (size_t)g.N * g.G;
  r.words = (g.N + 31) / 32;
  r.status = c.take(sizeof(StatusBlock));
  r.qr = c.take(BHq * NG * g.D * sizeof(bf16));
  r.kr = c.take(BHk * NG * g.D * sizeof(bf16));
  r.lse_r = c.take(BHq * NG * sizeof(float));
  r.pr = c.take(BHq * (size_t)g.N * g.N * sizeof(float));
  r.hist = c.take(BHq * 3 * 2048 * sizeof(unsigned));
  r.state = c.take(BHq * 8 * sizeof(unsigned));
  r.row_tau = c.take(BHq * g.N * sizeof(float));
  r.row_eq_take = c.take(BHq * g.N * sizeof(int));
  r.row_cnt = c.take(BHq * g.N * sizeof(int));
  r.row_gt = c.take(BHq * g.N * sizeof(int));
  r.row_eq = c.take(BHq * g.N * sizeof(int));
  r.bitmap = c.take(BHq * (size_t)g.N * r.words * sizeof(unsigned));
  r.bitmap_t = c.take(BHq * (size_t)g.N * r.words * sizeof(unsigned));
  r.total = c.off;
  return r;
}

BwdLayout bwd_layout(const Geo& g) {
  BwdLayout r;
  Carver c;
  const size_t BHq = (size_t)g.batch * g.Hq;
  r.status = c.take(sizeof(StatusBlock));
  r.delta = c.take(BHq * g.S * sizeof(float));
  r.d_oc_hat = c.take(BHq * g.N * g.D * sizeof(float));
  r.delta_c = c.take(BHq * g.N * sizeof(float));
  r.dqc = c.take(BHq * g.N * g.D * sizeof(float));
  r.dkc = c.take(BHq * g.N * g.D * sizeof(float));
  r.dvc = c.take(BHq * g.N * g.D * sizeof(float));
  r.pooled = c.take(pooled_layout(g, true).total);
  r.total = c.off;
  return r;
}

// [StatusBlock + rescue list of the fine forward][scratch of the coarse branch on the pooled grid]
size_t fwd_pooled_offset() { return align_up(fine_fwd_tc_workspace_bytes(), 256); }

// 128-token cubes: the regions above are laid out for the half-cube problem (`n` = narrow_geo), followed by what
// links the two levels: cube-level router scores, half-cube copies of the coarse tensors and of the block map.
struct WideRouteLayout {
  RouteLayout narrow;      // status, qr, kr, lse_r, pr (half-cube scores); its selection scratch is unused
  RouteLayout cube;        // selection scratch and pr at cube level, offsets relative to `cube_base`
  size_t cube_base, total;
};
WideRouteLayout wide_route_layout(const Geo& g) {
  WideRouteLayout r;
  r.narrow = route_layout(narrow_geo(g));
  r.cube = route_layout(g);
  r.cube_base = align_up(r.narrow.hist, 256);     // everything from the half-cube histograms on is not needed
  r.total = r.cube_base + r.cube.total;
  return r;
}
struct WideFwdLayout {
  size_t pooled, x64, oc_hat64, ptr64, idx64, total;
};
WideFwdLayout wide_fwd_layout(const Geo& g) {
  const Geo n = narrow_geo(g);
  WideFwdLayout r;
  Carver c;
  const size_t BHq = (size_t)g.batch * g.Hq;
  c.take(fine_fwd_tc_workspace_bytes());
  r.pooled = c.take(pooled_layout(g, false).total);
  r.x64 = c.take(BHq * n.N * n.D * sizeof(float));
  r.oc_hat64 = c.take(BHq * n.N * n.D * sizeof(float));
  r.ptr64 = c.take(BHq * (n.N + 1) * sizeof(int));
  r.idx64 = c.take(BHq * (size_t)n.nnz_cap * sizeof(int));
  r.total = c.off;
  return r;
}
struct WideBwdLayout {
  BwdLayout narrow;        // status, delta, d_oc_hat, dqc, dkc, dvc at half-cube level (delta_c and pooled unused)
  BwdLayout cube;          // d_oc_hat, delta_c, dqc, dkc, dvc, pooled at cube level, offsets relative to `cube_base`
  size_t cube_base, oc_hat64, ptr64, idx64, cptr64, ridx64, total;
};
WideBwdLayout wide_bwd_layout(const Geo& g) {
  const Geo n = narrow_geo(g);
  WideBwdLayout r;
  r.narrow = bwd_layout(n);
  r.cube = bwd_layout(g);
  r.cube_base = align_up(r.narrow.pooled, 256);
  Carver c;
  c.off = r.cube_base + r.cube.total;
  const size_t BHq = (size_t)g.batch * g.Hq;
  r.oc_hat64 = c.take(BHq * n.N * n.D * sizeof(float));
  r.ptr64 = c.take(BHq * (n.N + 1) * sizeof(int));
  r.idx64 = c.take(BHq * (size_t)n.nnz_cap * sizeof(int));
  r.cptr64 = c.take(BHq * (n.N + 1) * sizeof(int));
  r.ridx64 = c.take(BHq * (size_t)n.nnz_cap * sizeof(int));
  r.total = c.off;
  return r;
}

size_t route_workspace_bytes(const Geo& g) { return wide_cube(g) ? wide_route_layout(g).total : route_layout(g).total; }
size_t fwd_base_bytes(const Geo& g) {
  return wide_cube(g) ? wide_fwd_layout(g).total : align_up(fwd_pooled_offset() + pooled_layout(g, false).total, 256);
}
size_t bwd_base_bytes(const Geo& g) { return wide_cube(g) ? wide_bwd_layout(g).total : align_up(bwd_layout(g).total, 256); }
size_t fwd_workspace_bytes(const Geo& g) { return fwd_base_bytes(g) + text_map_layout(g, false).total; }
// fp16 copies of Q and K for the dQ pass (behind the other regions of the backward's workspace)
bool dq_pass_f16(const Geo& g) { return fine_bwd_dq_uses_f16(g); }
size_t bwd_f16_offset(const Geo& g) { return align_up(bwd_base_bytes(g) + text_map_layout(g, true).total, 256); }
size_t bwd_q16_bytes(const Geo& g) { return align_up((size_t)g.batch * g.Hq * g.S * g.D * sizeof(bf16), 256); }
size_t bwd_k16_bytes(const Geo& g) { return align_up((size_t)g.batch * g.Hkv * g.S * g.D * sizeof(bf16), 256); }
// GQA groups: fp16 copies of V and dO as well, for the all-fp16 dK/dV pass (behind the copies of Q and K)
bool dkv_pass_gqa_f16(const Geo& g) { return dq_pass_f16(g) && fine_bwd_dkv_gqa_uses_f16(g); }
size_t bwd_workspace_bytes(const Geo& g) {
  if (!dq_pass_f16(g)) return bwd_base_bytes(g) + text_map_layout(g, true).total;
  size_t n = bwd_f16_offset(g) + bwd_q16_bytes(g) + bwd_k16_bytes(g);
  if (dkv_pass_gqa_f16(g)) n += bwd_k16_bytes(g) + bwd_q16_bytes(g);      // V like K, dO like Q
  return n;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

// The kernels are built for sm_100a only.
int check_device() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return VSA2_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return VSA2_ERR_CUDA;
  return major == 10 ? VSA2_OK : VSA2_ERR_UNSUPPORTED;
}

template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(reinterpret_cast<unsigned char*>(ws) + off); }

cudaError_t g_last_cuda_error = cudaSuccess;

#define VSA2_CUDA(call)                              \
  do {                                               \
    cudaError_t e_ = (call);                         \
    if (e_ != cudaSuccess) {                         \
      g_last_cuda_error = e_;                        \
      return VSA2_ERR_CUDA;                          \
    }                                                \
  } while (0)

}  // namespace

namespace vsa2 {
ProfScope::ProfScope(int kernel_id, cudaStream_t stream, int launches) : id(kernel_id), st(stream) {
  g_launches += launches;
  if (g_prof_start[id] != nullptr) cudaEventRecord(g_prof_start[id], st);
}
ProfScope::~ProfScope() {
  if (g_prof_stop[id] != nullptr) cudaEventRecord(g_prof_stop[id], st);
}
}  // namespace vsa2

extern "C" {

int vsa2_profile_events(int32_t kernel_id, void* start_event, void* stop_event) {
  if (kernel_id < 0 || kernel_id >= VSA2_KERNEL_COUNT) return VSA2_ERR_INVALID_ARG;
  g_prof_start[kernel_id] = reinterpret_cast<cudaEvent_t>(start_event);
  g_prof_stop[kernel_id] = reinterpret_cast<cudaEvent_t>(stop_event);
  return VSA2_OK;
}

int64_t vsa2_launch_count(void) { return g_launches.load(); }

int32_t vsa2_debug_rescue_capacity(int32_t capacity) {
  set_fwd_rescue_capacity(capacity);
  return fwd_rescue_capacity();
}

const char* vsa2_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

int vsa2_query_sizes(const vsa2_params* p, vsa2_sizes* out) {
  if (out == nullptr) return VSA2_ERR_INVALID_ARG;
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  memset(out, 0, sizeof(*out));
  out->n_cubes = g.N;
  out->n_subcubes = g.G;
  out->block_tokens = g.Bt * g.Bh * g.Bw;
  out->topk_eff = g.K;
  out->seq_len = g.L;
  out->nnz_cap = g.nnz_cap;
  const long long BHq = (long long)g.batch * g.Hq, BHk = (long long)g.batch * g.Hkv;
  out->ptr_elems = BHq * (g.N + 1);
  out->idx_elems = BHq * g.nnz_cap;
  out->pooled_q_elems = BHq * g.N * g.D;
  out->pooled_kv_elems = BHk * g.N * g.D;
  out->lse_c_elems = BHq * g.N;
  out->o_res_elems = g.out_f32 ? 0 : BHq * (long long)g.S * g.D;
  out->tokens_per_head = g.S;
  out->text_blocks = text_blocks(g);
  out->route_workspace_bytes = route_workspace_bytes(g);
  out->fwd_workspace_bytes = fwd_workspace_bytes(g);
  out->bwd_workspace_bytes = bwd_workspace_bytes(g);
  return VSA2_OK;
}

int vsa2_route(const vsa2_params* p, const void* q, const void* k, const int32_t* budgets, const vsa2_map* map,
               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  if (!q || !k || !map || !workspace || !map->row_ptr || !map->col_idx || !map->col_ptr || !map->row_idx)
    return VSA2_ERR_INVALID_ARG;
  if (g.mode == VSA2_PER_QUERY_BUDGET && budgets == nullptr) return VSA2_ERR_INVALID_ARG;
  if (g.mode == VSA2_PER_QUERY_BUDGET && (g.flags & VSA2_FLAG_GROUP_ROUTING)) return VSA2_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(k) || !aligned256(workspace)) return VSA2_ERR_MISALIGNED;
  if (workspace_bytes < route_workspace_bytes(g)) return VSA2_ERR_WORKSPACE_TOO_SMALL;
  if ((rc = check_device()) != VSA2_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // 128-token cubes: sub-cube means and router scores at half-cube level (`r`), folded to cube scores; the
  // selection then runs on the cube-level matrix
  const bool wide = wide_cube(g);
  const Geo r = wide ? narrow_geo(g) : g;
  const RouteLayout rl = route_layout(r);
  RouteLayout lay = rl;
  unsigned char* sel_base = reinterpret_cast<unsigned char*>(workspace);
  if (wide) {
    const WideRouteLayout wl = wide_route_layout(g);
    lay = wl.cube;
    sel_base += wl.cube_base;
  }
  StatusBlock* status = at<StatusBlock>(workspace, rl.status);
  VSA2_CUDA(cudaMemsetAsync(status, 0, sizeof(StatusBlock), st));
  bf16* qr = at<bf16>(workspace, rl.qr);
  bf16* kr = at<bf16>(workspace, rl.kr);
  {
    ProfScope ps(VSA2_KERNEL_POOL_ROUTER, st, 1);
    VSA2_CUDA(launch_pool_router(r, reinterpret_cast<const bf16*>(q), reinterpret_cast<const bf16*>(k), qr, kr, st));
  }
  float* pr = at<float>(workspace, rl.pr);
  if (router_tc_supported(r))
    VSA2_CUDA(launch_router_scores_tc(r, qr, kr, at<float>(workspace, rl.lse_r), pr, status, st));
  else   // sub-cube counts the tensor-core kernel has no layout for (G = 1 is the VSA router of Sec. 2.1)
    VSA2_CUDA(launch_router_scores(r, qr, kr, at<float>(workspace, rl.lse_r), pr, st));
  if (wide) {
    g_launches += 1;
    float* pr_cube = at<float>(sel_base, lay.pr);
    VSA2_CUDA(launch_fold_scores(r, pr, pr_cube, st));
    pr = pr_cube;
  }
  if ((g.flags & VSA2_FLAG_GROUP_ROUTING) && g.rep > 1) {
    g_launches += 1;
    VSA2_CUDA(launch_group_sum_scores(g, pr, st));
  }
  workspace = sel_base;
  SelectScratch s;
  s.hist = at<unsigned>(workspace, lay.hist);
  s.state = at<unsigned>(workspace, lay.state);
  s.row_tau = at<float>(workspace, lay.row_tau);
  s.row_eq_take = at<int>(workspace, lay.row_eq_take);
  s.row_cnt = at<int>(workspace, lay.row_cnt);
  s.row_gt = at<int>(workspace, lay.row_gt);
  s.row_eq = at<int>(workspace, lay.row_eq);
  s.bitmap = at<unsigned>(workspace, lay.bitmap);
  s.bitmap_t = at<unsigned>(workspace, lay.bitmap_t);
  s.words = lay.words;
  {
    ProfScope ps(VSA2_KERNEL_SELECT, st, g.mode == VSA2_PER_SEQUENCE ? 14 : 7);
    VSA2_CUDA(launch_select(g, pr, budgets, s, map->row_ptr, map->col_idx, map->col_ptr, map->row_idx, status, st));
  }
  return VSA2_OK;
}

const float* vsa2_route_scores(const vsa2_params* p, const void* workspace) {
  Geo g;
  if (workspace == nullptr || fill_geo(p, &g) != VSA2_OK) return nullptr;
  size_t off = route_layout(g).pr;
  if (wide_cube(g)) {
    const WideRouteLayout wl = wide_route_layout(g);
    off = wl.cube_base + wl.cube.pr;
  }
  return reinterpret_cast<const float*>(reinterpret_cast<const unsigned char*>(workspace) + off);
}

int vsa2_attn_fwd(const vsa2_params* p, const void* q, const void* k, const void* v, const float* gate,
                  const vsa2_map* map, void* o, float* lse, const vsa2_saved* saved, void* workspace,
                  size_t workspace_bytes, void* cuda_stream) {
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  if (!q || !k || !v || !map || !o || !lse || !workspace || !map->row_ptr || !map->col_idx) return VSA2_ERR_INVALID_ARG;
  const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE);
  if (coarse && (!saved || !saved->qc || !saved->kc || !saved->vc || !saved->oc_hat || !saved->lse_c))
    return VSA2_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned256(workspace))
    return VSA2_ERR_MISALIGNED;
  if (saved != nullptr && !g.out_f32 && saved->o_res != nullptr && !aligned16(saved->o_res)) return VSA2_ERR_MISALIGNED;
  if (workspace_bytes < fwd_workspace_bytes(g)) return VSA2_ERR_WORKSPACE_TOO_SMALL;
  if ((rc = check_device()) != VSA2_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  VSA2_CUDA(cudaMemsetAsync(workspace, 0, sizeof(StatusBlock), st));
  const bf16* qb = reinterpret_cast<const bf16*>(q);
  const bf16* kb = reinterpret_cast<const bf16*>(k);
  const bf16* vb = reinterpret_cast<const bf16*>(v);
  // 128-token cubes: the fine kernels run on the half-cube problem `n` with the expanded map; the coarse branch
  // runs at cube level from folded half-cube means
  const bool wide = wide_cube(g);
  const Geo n = wide ? narrow_geo(g) : g;
  const WideFwdLayout wl = wide ? wide_fwd_layout(g) : WideFwdLayout();
  const size_t pooled_off = wide ? wl.pooled : fwd_pooled_offset();
  const int* row_ptr = map->row_ptr;
  const int* col_idx = map->col_idx;
  const float* oc_hat = coarse ? saved->oc_hat : nullptr;
  if (coarse) {
    {
      ProfScope ps(VSA2_KERNEL_POOL, st, wide ? 6 : 1);
      if (!wide) {
        VSA2_CUDA(launch_pool_coarse(g, qb, kb, vb, saved->qc, saved->kc, saved->vc, st));
      } else {
        float* x64 = at<float>(workspace, wl.x64);
        VSA2_CUDA(launch_pool(n, qb, n.Hq, nullptr, x64, st));
        VSA2_CUDA(launch_fold_mean(n, n.Hq, x64, saved->qc, st));
        VSA2_CUDA(launch_pool(n, kb, n.Hkv, nullptr, x64, st));
        VSA2_CUDA(launch_fold_mean(n, n.Hkv, x64, saved->kc, st));
        VSA2_CUDA(launch_pool(n, vb, n.Hkv, nullptr, x64, st));
        VSA2_CUDA(launch_fold_mean(n, n.Hkv, x64, saved->vc, st));
      }
    }
    {
      ProfScope ps(VSA2_KERNEL_COARSE_FWD, st, ((g.flags & VSA2_FLAG_BF16_COARSE_FWD) ? 7 : 1) + (wide ? 1 : 0));
      if (!(g.flags & VSA2_FLAG_BF16_COARSE_FWD))
        VSA2_CUDA(launch_coarse_fwd_mma(g, saved->qc, saved->kc, saved->vc, saved->oc_hat, saved->lse_c, st));
      else
        VSA2_CUDA(launch_coarse_fwd_pooled(g, saved->qc, saved->kc, saved->vc, saved->oc_hat, saved->lse_c,
                                           at<unsigned char>(workspace, pooled_off),
                                           reinterpret_cast<StatusBlock*>(workspace), st));
      if (wide) {
        VSA2_CUDA(launch_expand_rows(n, n.Hq, false, saved->oc_hat, at<float>(workspace, wl.oc_hat64), st));
        oc_hat = at<float>(workspace, wl.oc_hat64);
      }
    }
  }
  if (wide) {
    g_launches += 1;
    VSA2_CUDA(launch_expand_map(n, map->row_ptr, map->col_idx, at<int>(workspace, wl.ptr64), at<int>(workspace, wl.idx64), st));
    row_ptr = at<int>(workspace, wl.ptr64);
    col_idx = at<int>(workspace, wl.idx64);
  }
  bf16* o_res = (saved != nullptr && !g.out_f32) ? reinterpret_cast<bf16*>(saved->o_res) : nullptr;
  Geo fx = n;                                   // geometry of the fine kernels' block problem
  if (g.Lt > 0) {
    // text tokens: append the text blocks to the map (in the workspace) and run the kernels on the block problem
    // (with 128-token cubes the half-cube map built above is what gets extended, and the 64-token kernels run)
    const TextMapLayout tl = text_map_layout(g, false);
    unsigned char* tbase = at<unsigned char>(workspace, fwd_base_bytes(g));
    fx = text_geo(n);
    if (!fine_fwd_rows_supported(fx)) return VSA2_ERR_UNSUPPORTED;
    g_launches += 1;
    VSA2_CUDA(launch_extend_map(n, text_blocks(g), row_ptr, col_idx, at<int>(tbase, tl.ptr), at<int>(tbase, tl.idx),
                                fx.nnz_cap, st));
    row_ptr = at<int>(tbase, tl.ptr);
    col_idx = at<int>(tbase, tl.idx);
  }
  {
    ProfScope ps(VSA2_KERNEL_FINE_FWD, st, (g.flags & VSA2_FLAG_EXACT_MAX_FWD) ? 1 : 2);
    if (g.flags & VSA2_FLAG_EXACT_MAX_FWD)
      VSA2_CUDA(launch_fine_fwd(fx, qb, kb, vb, coarse ? gate : nullptr, row_ptr, col_idx, oc_hat, o, o_res, lse, st));
    else if ((wide || (g.flags & VSA2_FLAG_GROUP_ROUTING)) && fine_fwd_rows2_supported(n, !wide))
      // 128 query rows per tile: the halves of a 128-token cube, or two heads of a group that share their map
      VSA2_CUDA(launch_fine_fwd_rows2_tc(n, !wide, qb, kb, vb, coarse ? gate : nullptr, row_ptr, col_idx, oc_hat, o, o_res, lse,
                                         reinterpret_cast<StatusBlock*>(workspace), st));
    else if (fine_fwd_rows_supported(fx))
      VSA2_CUDA(launch_fine_fwd_rows_tc(fx, qb, kb, vb, coarse ? gate : nullptr, row_ptr, col_idx, oc_hat, o, o_res, lse,
                                        reinterpret_cast<StatusBlock*>(workspace), st));
    else
      VSA2_CUDA(launch_fine_fwd_tc(n, qb, kb, vb, coarse ? gate : nullptr, row_ptr, col_idx, oc_hat, o, o_res, lse,
                                   reinterpret_cast<StatusBlock*>(workspace), st));
  }
  return VSA2_OK;
}

int vsa2_attn_bwd(const vsa2_params* p, const void* q, const void* k, const void* v, const float* gate,
                  const vsa2_map* map, const void* o, const float* lse, const vsa2_saved* saved, const void* d_o,
                  void* dq, void* dk, void* dv, float* dgate, void* workspace, size_t workspace_bytes,
                  void* cuda_stream) {
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  if (!q || !k || !v || !map || !o || !lse || !d_o || !dq || !dk || !dv || !workspace || !map->row_ptr ||
      !map->col_idx || !map->col_ptr || !map->row_idx)
    return VSA2_ERR_INVALID_ARG;
  const bool coarse = !(g.flags & VSA2_FLAG_NO_COARSE) && gate != nullptr;
  if (coarse && (!saved || !saved->qc || !saved->kc || !saved->vc || !saved->oc_hat || !saved->lse_c))
    return VSA2_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv) || !aligned256(workspace))
    return VSA2_ERR_MISALIGNED;
  if (workspace_bytes < bwd_workspace_bytes(g)) return VSA2_ERR_WORKSPACE_TOO_SMALL;
  if ((rc = check_device()) != VSA2_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  VSA2_CUDA(cudaMemsetAsync(workspace, 0, sizeof(StatusBlock), st));
  // 128-token cubes: preprocess and the fine passes run on the half-cube problem `n` (regions `lay`), the coarse
  // backward at cube level (regions `cl` behind `cube_ws`); folds and expansions link the two
  const bool wide = wide_cube(g);
  const Geo n = wide ? narrow_geo(g) : g;
  const WideBwdLayout wl = wide ? wide_bwd_layout(g) : WideBwdLayout();
  const BwdLayout lay = wide ? wl.narrow : bwd_layout(g);
  const BwdLayout cl = wide ? wl.cube : lay;
  void* cube_ws = wide ? at<unsigned char>(workspace, wl.cube_base) : workspace;
  const bf16* qb = reinterpret_cast<const bf16*>(q);
  const bf16* kb = reinterpret_cast<const bf16*>(k);
  const bf16* vb = reinterpret_cast<const bf16*>(v);
  const bf16* dob = reinterpret_cast<const bf16*>(d_o);
  float* delta = at<float>(workspace, lay.delta);
  float* d_oc_hat = at<float>(workspace, lay.d_oc_hat);
  float* dqc = at<float>(workspace, lay.dqc);
  float* dkc = at<float>(workspace, lay.dkc);
  float* dvc = at<float>(workspace, lay.dvc);
  float* d_oc_hat_cube = at<float>(cube_ws, cl.d_oc_hat);
  float* dqc_cube = at<float>(cube_ws, cl.dqc);
  float* dkc_cube = at<float>(cube_ws, cl.dkc);
  float* dvc_cube = at<float>(cube_ws, cl.dvc);
  const int* row_ptr = map->row_ptr;
  const int* col_idx = map->col_idx;
  const int* col_ptr = map->col_ptr;
  const int* row_idx = map->row_idx;
  const float* oc_hat = coarse ? saved->oc_hat : nullptr;
  if (wide) {
    g_launches += 2;
    VSA2_CUDA(launch_expand_map(n, map->row_ptr, map->col_idx, at<int>(workspace, wl.ptr64), at<int>(workspace, wl.idx64), st));
    VSA2_CUDA(launch_expand_map(n, map->col_ptr, map->row_idx, at<int>(workspace, wl.cptr64), at<int>(workspace, wl.ridx64), st));
    row_ptr = at<int>(workspace, wl.ptr64);
    col_idx = at<int>(workspace, wl.idx64);
    col_ptr = at<int>(workspace, wl.cptr64);
    row_idx = at<int>(workspace, wl.ridx64);
    if (coarse) {
      g_launches += 1;
      VSA2_CUDA(launch_expand_rows(n, n.Hq, false, saved->oc_hat, at<float>(workspace, wl.oc_hat64), st));
      oc_hat = at<float>(workspace, wl.oc_hat64);
    }
  }
  Geo fx = n;                                   // geometry of the fine kernels' block problem
  if (g.Lt > 0) {
    const TextMapLayout tl = text_map_layout(g, true);
    unsigned char* tbase = at<unsigned char>(workspace, bwd_base_bytes(g));
    fx = text_geo(n);
    g_launches += 2;
    VSA2_CUDA(launch_extend_map(n, text_blocks(g), row_ptr, col_idx, at<int>(tbase, tl.ptr), at<int>(tbase, tl.idx),
                                fx.nnz_cap, st));
    VSA2_CUDA(launch_extend_map(n, text_blocks(g), col_ptr, row_idx, at<int>(tbase, tl.cptr), at<int>(tbase, tl.ridx),
                                fx.nnz_cap, st));
    row_ptr = at<int>(tbase, tl.ptr);
    col_idx = at<int>(tbase, tl.idx);
    col_ptr = at<int>(tbase, tl.cptr);
    row_idx = at<int>(tbase, tl.ridx);
  }
  if (!coarse && dgate != nullptr)
    VSA2_CUDA(cudaMemsetAsync(dgate, 0, (size_t)g.batch * g.Hq * g.L * sizeof(float), st));
  const bf16* o_res = (saved != nullptr && !g.out_f32) ? reinterpret_cast<const bf16*>(saved->o_res) : nullptr;
  {
    ProfScope ps(VSA2_KERNEL_BWD_PRE, st, 1);
    VSA2_CUDA(launch_bwd_preprocess(fx, dob, o, o_res, coarse ? gate : nullptr, oc_hat, delta, coarse ? dgate : nullptr,
                                    d_oc_hat, st));
  }
  if (coarse) {
    // pooled grid: four casts, the dense map, the pooled preprocess, dQ, dK/dV (+ two group spreads)
    ProfScope ps(VSA2_KERNEL_COARSE_BWD, st, 9 + (g.rep > 1 ? 2 : 0) + (wide ? 4 : 0));
    if (wide) VSA2_CUDA(launch_fold_sum(n, n.Hq, d_oc_hat, d_oc_hat_cube, st));
    VSA2_CUDA(launch_coarse_bwd_pooled(g, saved->qc, saved->kc, saved->vc, saved->oc_hat, saved->lse_c, d_oc_hat_cube,
                                       dqc_cube, dkc_cube, dvc_cube, at<unsigned char>(cube_ws, cl.pooled),
                                       reinterpret_cast<StatusBlock*>(workspace), st));
    if (wide) {
      VSA2_CUDA(launch_expand_rows(n, n.Hq, true, dqc_cube, dqc, st));
      VSA2_CUDA(launch_expand_rows(n, n.Hq, true, dkc_cube, dkc, st));
      VSA2_CUDA(launch_expand_rows(n, n.Hq, true, dvc_cube, dvc, st));
    }
  }
  // cubes of 128 tokens: both passes on 128 x 128 tiles
  const bool wide128 = wide && g.Lt == 0 && fine_bwd128_supported(n);
  {
    const bool f16 = dq_pass_f16(g);     // the copy, the fp16 form, the (idle) fallback
    ProfScope ps(VSA2_KERNEL_FINE_BWD_DQ, st, f16 ? 3 : 1);
    if (wide128)
      VSA2_CUDA(launch_fine_bwd128_dq_tc(n, qb, kb, vb, dob, lse, delta, row_ptr, col_idx, coarse ? dqc : nullptr, dq,
                                         reinterpret_cast<StatusBlock*>(workspace), st,
                                         f16 ? at<unsigned char>(workspace, bwd_f16_offset(g)) : nullptr,
                                         f16 ? at<unsigned char>(workspace, bwd_f16_offset(g) + bwd_q16_bytes(g)) : nullptr));
    else
      VSA2_CUDA(launch_fine_bwd_dq_tc(fx, qb, kb, vb, dob, lse, delta, row_ptr, col_idx, coarse ? dqc : nullptr, dq,
                                      reinterpret_cast<StatusBlock*>(workspace), st,
                                      f16 ? at<unsigned char>(workspace, bwd_f16_offset(g)) : nullptr,
                                      f16 ? at<unsigned char>(workspace, bwd_f16_offset(g) + bwd_q16_bytes(g)) : nullptr));
  }
  {
    const bool dkv128 = wide128 && !fine_bwd_dkv_wants_pair(n);
    // scratch for the list of the long column lists (two-launch form): d_oc_hat is dead once the coarse backward has run
    const size_t list_need = (size_t)fx.batch * fx.Hkv * fx.N + 1, list_have = (size_t)n.batch * n.Hq * n.N * n.D;
    int* item_list = list_need <= list_have ? reinterpret_cast<int*>(d_oc_hat) : nullptr;
    const bool two = !dkv128 && fine_bwd_dkv_splits_long_columns(fx, true);
    const bool gqa16 = !dkv128 && dkv_pass_gqa_f16(g);    // (the copy of V and dO, the all-fp16 form, the pair form as its fallback)
    const bool f16 = (two || gqa16) && dq_pass_f16(g);              // the dQ pass has left fp16 copies of Q and K
    ProfScope ps(VSA2_KERNEL_FINE_BWD_DKV, st, dkv128 ? (dq_pass_f16(g) ? 2 : 1)
                                                      : two ? (item_list ? 3 : 2) + (f16 ? 1 : 0) : (gqa16 ? 3 : 1));
    unsigned char* v16 = gqa16 ? at<unsigned char>(workspace, bwd_f16_offset(g) + bwd_q16_bytes(g) + bwd_k16_bytes(g)) : nullptr;
    if (dkv128)
      VSA2_CUDA(launch_fine_bwd128_dkv_tc(n, qb, kb, vb, dob, lse, delta, col_ptr, row_idx, coarse ? dkc : nullptr,
                                          coarse ? dvc : nullptr, dk, dv, reinterpret_cast<StatusBlock*>(workspace), st,
                                          dq_pass_f16(g) ? at<unsigned char>(workspace, bwd_f16_offset(g)) : nullptr,
                                          dq_pass_f16(g) ? at<unsigned char>(workspace, bwd_f16_offset(g) + bwd_q16_bytes(g)) : nullptr));
    else
      VSA2_CUDA(launch_fine_bwd_dkv_tc(fx, qb, kb, vb, dob, lse, delta, col_ptr, row_idx, coarse ? dkc : nullptr,
                                       coarse ? dvc : nullptr, dk, dv, reinterpret_cast<StatusBlock*>(workspace), st, true,
                                       item_list, f16 ? at<unsigned char>(workspace, bwd_f16_offset(g)) : nullptr,
                                       f16 ? at<unsigned char>(workspace, bwd_f16_offset(g) + bwd_q16_bytes(g)) : nullptr, v16,
                                       gqa16 ? v16 + bwd_k16_bytes(g) : nullptr));
  }
  return VSA2_OK;
}

int vsa2_permute_cube_major(const vsa2_params* p, int32_t heads, int32_t inverse, const void* src, void* dst,
                            void* cuda_stream) {
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  if (!src || !dst || heads <= 0 || heads > 65535) return VSA2_ERR_INVALID_ARG;
  if (!aligned16(src) || !aligned16(dst)) return VSA2_ERR_MISALIGNED;
  if ((rc = check_device()) != VSA2_OK) return rc;
  g_launches += 1;
  VSA2_CUDA(launch_permute(g, reinterpret_cast<const bf16*>(src), heads, inverse != 0, reinterpret_cast<bf16*>(dst),
                           reinterpret_cast<cudaStream_t>(cuda_stream)));
  return VSA2_OK;
}

int vsa2_gate_fwd(const vsa2_params* p, int32_t hidden, const void* x, const void* w_g, float* gate, void* cuda_stream) {
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  if (!x || !w_g || !gate) return VSA2_ERR_INVALID_ARG;
  if (!gate_supported(hidden, g.Hq)) return VSA2_ERR_UNSUPPORTED;
  if (!aligned16(x)) return VSA2_ERR_MISALIGNED;
  if ((rc = check_device()) != VSA2_OK) return rc;
  g_launches += 1;
  VSA2_CUDA(launch_gate_fwd(g.batch, g.L, hidden, g.Hq, reinterpret_cast<const bf16*>(x), reinterpret_cast<const bf16*>(w_g),
                            gate, reinterpret_cast<cudaStream_t>(cuda_stream)));
  return VSA2_OK;
}

size_t vsa2_gate_bwd_workspace_bytes(const vsa2_params* p, int32_t hidden) {
  Geo g;
  if (fill_geo(p, &g) != VSA2_OK || !gate_supported(hidden, g.Hq)) return 0;
  return gate_bwd_workspace_bytes(g.batch, g.L, hidden, g.Hq);
}

int vsa2_gate_bwd(const vsa2_params* p, int32_t hidden, const void* x, const void* w_g, const float* gate,
                  const float* dgate, float* d_w_g, void* dx, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  Geo g;
  int rc = fill_geo(p, &g);
  if (rc != VSA2_OK) return rc;
  if (!x || !w_g || !gate || !dgate || !d_w_g || !dx || !workspace) return VSA2_ERR_INVALID_ARG;
  if (!gate_supported(hidden, g.Hq)) return VSA2_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(dx) || !aligned256(workspace)) return VSA2_ERR_MISALIGNED;
  if (workspace_bytes < gate_bwd_workspace_bytes(g.batch, g.L, hidden, g.Hq)) return VSA2_ERR_WORKSPACE_TOO_SMALL;
  if ((rc = check_device()) != VSA2_OK) return rc;
  g_launches += 4;
  VSA2_CUDA(launch_gate_bwd(g.batch, g.L, hidden, g.Hq, g.out_f32, reinterpret_cast<const bf16*>(x),
                            reinterpret_cast<const bf16*>(w_g), gate, dgate, d_w_g, dx, workspace,
                            reinterpret_cast<cudaStream_t>(cuda_stream)));
  return VSA2_OK;
}

int vsa2_device_status(const void* workspace, void* cuda_stream, int32_t* status_out) {
  if (workspace == nullptr || status_out == nullptr) return VSA2_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  VSA2_CUDA(cudaStreamSynchronize(st));
  int s = 0;
  VSA2_CUDA(cudaMemcpy(&s, workspace, sizeof(int), cudaMemcpyDeviceToHost));
  *status_out = s;
  return VSA2_OK;
}

const char* vsa2_strerror(int code) {
  switch (code) {
    case VSA2_OK: return "ok";
    case VSA2_ERR_INVALID_ARG: return "invalid argument";
    case VSA2_ERR_UNSUPPORTED: return "unsupported shape, dtype or device (needs sm_100)";
    case VSA2_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case VSA2_ERR_MISALIGNED: return "pointer not aligned (16 bytes for tensors, 256 bytes for workspaces)";
    case VSA2_ERR_CUDA: return "CUDA call or kernel launch failed";
    case VSA2_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case VSA2_ERR_MAP_OVERFLOW: return "more selected blocks than nnz_cap";
    case VSA2_ERR_STATIC_SCRATCH: return "problem needs more scratch than the library's built-in 8 MiB buffer (use vsa2_route)";
    default: return "unknown vsa2 error";
  }
}

}  // extern "C"
