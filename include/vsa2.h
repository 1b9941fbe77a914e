/*
 * vsa2.h -- C ABI of the B200 (sm_100a) library for VSA2 routed block-sparse attention.
 *
 * The operator (paper Sec. 2.2) works on the tokens of a video latent grid (T, H, W), tiled
 * into cubes of B = Bt*Bh*Bw tokens (N = Nt*Nh*Nw cubes after padding each dimension up to a
 * whole number of cubes):
 *
 *   coarse branch  Q_c,K_c,V_c = MeanPool_B(Q,K,V); P_c = softmax(Q_c K_c^T * scale);
 *                  O_c = Repeat_B(P_c V_c)                                       (Eq. 1-4)
 *   router         Q_r,K_r = MeanPool_R(Q,K); P^_r = softmax(Q_r K_r^T * scale);
 *                  P_r = MeanPool_{GxG}(P^_r), G = B/R                           (Eq. 5-7)
 *   selection      keep the N*K largest of the N*N entries of P_r                (Eq. 8-9)
 *   fine branch    O_f = BlockSparseAttn(Q,K,V; M)                               (Eq. 12)
 *   merge          O = gate * O_c + O_f                                          (Eq. 14)
 *
 * Conventions shared by every entry point
 *   - All tensor pointers are DEVICE pointers on the current CUDA device unless a comment says
 *     "host".  Structs (params, map, saved, sizes) live in HOST memory and are read during
 *     the call only.  The library never allocates or frees device memory in the four entry
 *     points vsa2_route / vsa2_attn_fwd / vsa2_attn_bwd / vsa2_device_status: every buffer
 *     is caller-owned.
 *   - Q is [batch, heads_q, L, D], K and V are [batch, heads_kv, L, D], bf16, contiguous,
 *     tokens in raster order l = (t*H + h)*W + w of the VALID grid (padding is never
 *     materialised), L = T*H*W.  Query head hq uses KV head hq / (heads_q / heads_kv).
 *   - Tensor base pointers must be 16-byte aligned (workspaces 256-byte aligned).
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default stream);
 *     no entry point synchronises the stream except vsa2_device_status.
 *   - Return value: VSA2_OK or a negative vsa2 error code; nothing is enqueued when an
 *     argument check fails.  There is no CPU fallback.
 */
#ifndef VSA2_H_
#define VSA2_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  VSA2_OK = 0,
  VSA2_ERR_INVALID_ARG = -1,          /* null pointer, non-positive size, bad enum, heads_q % heads_kv != 0 ... */
  VSA2_ERR_UNSUPPORTED = -2,          /* shape outside what the kernels implement, or device is not sm_100 */
  VSA2_ERR_WORKSPACE_TOO_SMALL = -3,
  VSA2_ERR_MISALIGNED = -4,
  VSA2_ERR_CUDA = -5,                 /* a CUDA runtime/driver call or a launch failed */
  VSA2_ERR_DEVICE_TIMEOUT = -6,       /* a bounded device-side wait ran out (reported by vsa2_device_status) */
  VSA2_ERR_MAP_OVERFLOW = -7,         /* more selected blocks than nnz_cap (reported by vsa2_device_status) */
  VSA2_ERR_STATIC_SCRATCH = -8        /* vsa2_route_noalloc: the problem needs more scratch than the built-in buffer */
};

enum { VSA2_PER_SEQUENCE = 0,         /* Eq. 8-9: the N*K largest entries of the flattened P_r per (batch, query head) */
       VSA2_PER_QUERY = 1,            /* Sec. 2.1 (VSA form): the K largest per query block */
       VSA2_PER_QUERY_BUDGET = 2 };   /* query block i keeps its own k_i largest (k_i from `budgets`) */

enum { VSA2_BF16 = 0, VSA2_F32 = 1 };

enum { VSA2_FLAG_NO_COARSE = 1,       /* skip the coarse branch: O = O_f (the gate = 0 case, Sec. 2.3) */
       VSA2_FLAG_EXACT_MAX_FWD = 2 }; /* validation aid: run the whole fine forward with the slow kernel that tracks
                                         the exact running row maximum (the tensor-core kernel falls back to it only
                                         for query blocks whose softmax sums leave the safe range) */
/* Coarse branch (Eq. 2-3).  Default: forward with TF32 tensor-core tiles on the fp32 cube means (O_c feeds dGate, which
 * needs that precision); backward by running the tcgen05 fine-branch kernels on the pooled grid with the means rounded
 * to bf16 (its results enter dQ, dK, dV divided by the cube size, where bf16 operand rounding is far below the error
 * bounds). */
enum { VSA2_FLAG_BF16_COARSE_FWD = 64 }; /* forward of the coarse branch on the pooled grid with bf16 operands as well
                                         (about 8x faster; O_c then carries bf16 operand rounding: O stays within the
                                         output bound, dGate of a later backward may exceed 2e-2 by about 2x) */
/* Precision of the backward passes.  P and dS are 16-bit operands of the dV, dK and dQ products; rounded once to bf16 (2^-9
 * relative) they alone push the worst elements of large gradients (|g| > 5) past max abs err 2e-2 (720p sample, fp32 outputs:
 * dQ 2.5e-2; with one query head per KV head the KV blocks that nearly every query keeps reach |dK| = 15 and 1.5 - 2.7e-2).
 * Default: the dQ pass works on fp16 copies of Q and K that it makes in the workspace (every bf16 value inside the fp16
 * range has an exact fp16 image, so S is unchanged) and rounds dS to fp16, 11 significant bits instead of 8, at the speed
 * of the once-rounded form; with one query head per KV head the dK/dV pass does the same for S, dS and its dK product (P and
 * the dV product stay bf16: |dV| is small).  Measured against the oracle (fp32 outputs, 720p sample): dQ 8.7e-3, dK 3.5e-3.
 * A range flag guards the fp16 forms: a finite |Q| or |K| of 65520 or more, or a dS beyond the largest fp16 value, and the passes are
 * redone by the bf16-pair kernels described next (launched behind the fp16 ones, they return at once while the flag is clear).
 * GQA groups (a KV block sums the query blocks of several heads) with TopK >= 8: the dK/dV pass makes fp16 copies of V and dO
 * as well and runs all four products in fp16, P included (480p sample: dK 9.4e-3, dV 2.7e-3; once-rounded bf16 2.2e-2 and
 * 1.4e-2), about 30 % faster than the pair form.
 * The pair form carries X as the bf16 value and the bf16 rounding of what that lost, in one product of twice the width: the
 * dK/dV pass of GQA groups uses it when rows keep fewer than 8 blocks or have per-row budgets (sharply peaked weights, where
 * 11 bits do not do), and as its fallback; the fallback of the one-head-per-KV-head case uses it for the KV blocks kept by more
 * than 256 query blocks.
 * With cubes of 128 tokens both passes have the same fp16 forms on 128 x 128 tiles (the pair form of the dQ pass, its fallback,
 * travels along the contraction; the fallback of the dK/dV pass is its bf16 form); a dK/dV pass for GQA groups or with
 * VSA2_FLAG_PRECISE_BWD runs on the 64-token halves. */
enum { VSA2_FLAG_FAST_BWD = 4 };      /* round P and dS once to bf16 everywhere, no fp16 copies (saves the 0.5 ms copy at 720p; GQA
                                         dK/dV pass about 30 % faster) */
enum { VSA2_FLAG_PRECISE_BWD = 8 };   /* bf16 pairs in the dQ pass and in the dK/dV pass, for MHA as well (dQ pass about 15 %, dK/dV
                                         pass about 35 % slower): for maps that keep only a few blocks per row, where the softmax is
                                         sharply peaked and P itself needs the extra bits */
enum { VSA2_FLAG_GROUP_ROUTING = 256 };/* vsa2_route: the query heads of one KV group share one block map ("group head", Sec. 4
                                         ablation): the block scores of the group's heads are added before the TopK, so
                                         the maps written for those heads are identical.  Not with VSA2_PER_QUERY_BUDGET
                                         (budgets belong to single heads): VSA2_ERR_UNSUPPORTED.
                                         vsa2_attn_fwd with this flag RELIES on that: with an even number of query heads per
                                         KV head it stacks pairs of heads in the 128 rows of one tile (the same K/V tiles
                                         serve both) and reads the map of the first head of each pair only */

/* Problem statement (host struct). */
typedef struct vsa2_params {
  int32_t batch, heads_q, heads_kv, head_dim;  /* head_dim in {64, 128}; heads_q % heads_kv == 0, ratio <= 16 */
  int32_t grid_t, grid_h, grid_w;              /* valid latent grid */
  int32_t cube_t, cube_h, cube_w;              /* cube (block) shape: 64 tokens (e.g. 4,4,4), or 128 tokens with cube_w even
                                                  and rpool_w dividing cube_w/2 (the paper's 4,4,8 with R = 2,2,2: G = 16);
                                                  N, K, budgets and the block map are then in cubes of 128 tokens, and the
                                                  library routes and pools on the cube's two 64-token halves along w
                                                  and runs the fine branch on 128 x 128 tiles
                                                  (Sec. 2.2 "Permutation", Eq. 5-7, Eq. 12) */
  int32_t rpool_t, rpool_h, rpool_w;           /* router pooling R, each divides the cube dimension */
  int32_t select_mode;                         /* VSA2_PER_* */
  int32_t topk;                                /* K in blocks (clamped to N); if 0, K = max(1, round(keep_fraction*N)) */
  float   keep_fraction;                       /* 1 - block sparsity, used only when topk == 0 */
  float   softmax_scale;                       /* 0 => 1/sqrt(head_dim); used by coarse, router and fine alike */
  int32_t out_dtype;                           /* VSA2_BF16 or VSA2_F32: dtype of O, dQ, dK, dV */
  int32_t flags;                               /* VSA2_FLAG_* */
  int32_t text_len;                            /* Lt >= 0: text tokens that share the attention space (Sec. 2.2, the sentence
                                                  after Eq. 12; MMDiT).  With Lt > 0 every token tensor (q, k, v, o, d_o, dq, dk,
                                                  dv: [batch, heads, L + Lt, D]; lse: [batch, heads_q, L + Lt]) holds the L video
                                                  tokens in raster order followed by the Lt text tokens.  The block map, the router
                                                  and the coarse branch cover the video tokens only; gate and dgate stay
                                                  [batch, heads_q, L].  With cubes of 128 tokens the fine branch then runs on the
                                                  64-token halves (the text blocks are 64 tokens). */
  int64_t nnz_cap;                             /* capacity of col_idx/row_idx per (batch, query head); 0 => N*K.
                                                  PER_QUERY_BUDGET requires it (>= sum_i min(k_i, N)). */
} vsa2_params;

/* Derived sizes (host struct, filled by vsa2_query_sizes).  Element counts are totals over batch and heads. */
typedef struct vsa2_sizes {
  int32_t n_cubes;            /* N */
  int32_t n_subcubes;         /* G */
  int32_t block_tokens;       /* B */
  int32_t topk_eff;           /* K after clamping / keep_fraction */
  int64_t seq_len;            /* L */
  int64_t nnz_cap;            /* per (batch, query head) */
  int64_t ptr_elems;          /* int32 elements of row_ptr and of col_ptr: batch*heads_q*(N+1) */
  int64_t idx_elems;          /* int32 elements of col_idx and of row_idx: batch*heads_q*nnz_cap */
  int64_t pooled_q_elems;     /* float elements of saved.qc and saved.oc_hat: batch*heads_q*N*D */
  int64_t pooled_kv_elems;    /* float elements of saved.kc and of saved.vc: batch*heads_kv*N*D */
  int64_t lse_c_elems;        /* float elements of saved.lse_c: batch*heads_q*N */
  int64_t o_res_elems;        /* bf16 elements of saved.o_res: batch*heads_q*(L + Lt)*D (0 when out_dtype is fp32) */
  size_t  route_workspace_bytes;
  size_t  fwd_workspace_bytes;
  size_t  bwd_workspace_bytes;
  int64_t tokens_per_head;    /* L + Lt: rows per head of every token tensor */
  int32_t text_blocks;        /* ceil(Lt / 64): blocks the fine kernels append to the N video cubes */
  int32_t reserved;
} vsa2_sizes;

/* Block map of the selected (query block, KV block) pairs (host struct of device pointers).
 * CSR: query block i of (b, hq) owns col_idx[(b*Hq+hq)*nnz_cap + row_ptr[(b*Hq+hq)*(N+1) + i ...+ i+1)],
 * KV block indices ascending.  CSC is the transpose (KV block j -> ascending query blocks), used by
 * the dK/dV pass. */
typedef struct vsa2_map {
  int32_t* row_ptr;   /* [batch, heads_q, N+1] */
  int32_t* col_idx;   /* [batch, heads_q, nnz_cap] */
  int32_t* col_ptr;   /* [batch, heads_q, N+1] */
  int32_t* row_idx;   /* [batch, heads_q, nnz_cap] */
} vsa2_map;

/* State the forward pass leaves for the backward pass (host struct of device pointers, fp32). */
typedef struct vsa2_saved {
  float* qc;       /* [batch, heads_q,  N, D]  Eq. 1 */
  float* kc;       /* [batch, heads_kv, N, D] */
  float* vc;       /* [batch, heads_kv, N, D] */
  float* oc_hat;   /* [batch, heads_q,  N, D]  Eq. 3 */
  float* lse_c;    /* [batch, heads_q,  N]     log-sum-exp of the coarse scores */
  void*  o_res;    /* bf16 [batch, heads_q, L, D], optional (may be NULL), used only when out_dtype is bf16:
                      the rounding residual bf16(O_fp32 - O_bf16) of the forward output.  The backward adds it
                      back to O when it forms delta = rowsum(dO * O_f), which removes the bf16 storage noise of O
                      from dQ and dK. */
} vsa2_saved;

/* Validates `p` and fills `out`.  Pure host arithmetic; no CUDA call. */
int vsa2_query_sizes(const vsa2_params* p, vsa2_sizes* out);

/* Router + selection (Eq. 5-9).  Reads q, k; writes the CSR and CSC maps.
 *   budgets: device int32 [batch, heads_q, N], only for VSA2_PER_QUERY_BUDGET (else may be NULL).
 *   workspace: >= sizes.route_workspace_bytes; holds the pooled bf16 operands, the router
 *   log-sum-exp, P_r [batch, heads_q, N, N] fp32 and selection scratch.  Its first word is the
 *   device status word read by vsa2_device_status.
 * Pooled router operands are the bf16 rounding of the fp32 mean (sum taken along w, then h, then
 * t; valid tokens only).  Ties in the TopK go to the lower flat index i*N + j.  No gradient is
 * defined through this call (Sec. 2.1). */
int vsa2_route(const vsa2_params* p, const void* q, const void* k, const int32_t* budgets,
               const vsa2_map* map_out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Allocation-free variant of vsa2_route (the paper has no counterpart).
 *
 * For callers that cannot allocate device memory where they need a block map: code running where cudaMalloc is
 * forbidden or would stall (an allocator lock is held, a latency-critical loop sized up front, a plug-in that is
 * handed no allocator) or a process whose memory budget is fixed at start-up.  Same inputs, outputs, readings and
 * error codes as vsa2_route, but the workspace is a device array built into the library: 8 MiB
 * (VSA2_ROUTE_NOALLOC_MAX_BYTES) that every GPU loading the library holds until the process exits.
 *   - A problem whose sizes.route_workspace_bytes exceeds 8 MiB is rejected with VSA2_ERR_STATIC_SCRATCH before
 *     anything is enqueued (roughly: up to ~2k tokens x 12 heads fits; the 480p and 720p shapes do not).
 *   - device_status: optional device int32; if not NULL the status word of this call (VSA2_OK,
 *     VSA2_ERR_MAP_OVERFLOW, VSA2_ERR_DEVICE_TIMEOUT) is copied there on the stream, after the kernels.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *     current); make that first call at start-up, outside any stream capture: with CUDA's lazy module loading it is
 *     also the moment the driver loads the library's device code and backs the 8 MiB array, so it is the one call
 *     that can fail for lack of memory.  No call uses cudaMalloc, cudaFree or any allocating routine.
 *   - All calls on one device share the one array, and it keeps the last call's contents: the call clears what
 *     must start at zero itself, but two calls that overlap on the GPU (different streams, no ordering) race;
 *     order them on one stream or with events.  The address look-up is guarded by a mutex; the library's launch
 *     counter is atomic; the profiling hooks (vsa2_profile_events) are not thread-safe. */
#define VSA2_ROUTE_NOALLOC_MAX_BYTES (8u << 20)
int vsa2_route_noalloc(const vsa2_params* p, const void* q, const void* k, const int32_t* budgets,
                       const vsa2_map* map_out, int32_t* device_status, void* cuda_stream);

/* Read-only access to the block scores P_r [batch, heads_q, N, N] (fp32) that the last vsa2_route
 * call on `workspace` left there; valid until the workspace is reused.  Returns NULL on bad input. */
const float* vsa2_route_scores(const vsa2_params* p, const void* workspace);

/* Text tokens (p->text_len > 0; Sec. 2.2, the sentence after Eq. 12).  Reading taken: one softmax per query row over its whole
 * key set.  A video query of cube i attends the kept video cubes of row i of the map and ALL text keys; a text query attends
 * all video keys and all text keys.  Text queries take no part in the coarse branch or the gate (their output is the fine
 * branch's), text keys none in the router.  vsa2_route is unchanged (it reads the video rows of q and k); vsa2_attn_fwd and
 * vsa2_attn_bwd append the text blocks to the map inside their workspace and run the same kernels on the longer lists. */

/* Coarse branch (Eq. 1-4), fine branch (Eq. 12) and merge (Eq. 14).
 *   gate: fp32 [batch, heads_q, L] (the caller's tanh(X W_g), Eq. 13); NULL means gate = 0.
 *   o:    [batch, heads_q, L, D] in p->out_dtype;  lse: fp32 [batch, heads_q, L], natural log of the
 *         fine branch's softmax denominator (scaled scores); -inf and O_f = 0 for a query block
 *         with no selected KV block.
 *   saved: filled for vsa2_attn_bwd (ignored, may be NULL, with VSA2_FLAG_NO_COARSE).
 *   workspace: >= sizes.fwd_workspace_bytes.
 * Every argument check, including the alignment of saved->o_res, runs before the first kernel is enqueued.
 * A map whose vsa2_route ended with VSA2_ERR_MAP_OVERFLOW holds truncated rows: forward and backward on it read at most
 * nnz_cap entries per (batch, query head) and compute the attention of that truncated map. */
int vsa2_attn_fwd(const vsa2_params* p, const void* q, const void* k, const void* v, const float* gate,
                  const vsa2_map* map, void* o, float* lse, const vsa2_saved* saved,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Backward of vsa2_attn_fwd for a fixed map (the map carries no gradient, Sec. 2.1).
 *   o, lse, saved: as written by the forward call;  d_o: bf16 [batch, heads_q, L, D].
 *   dq [batch, heads_q, L, D], dk, dv [batch, heads_kv, L, D] in p->out_dtype (dk, dv summed over the
 *   query heads of a group); dgate fp32 [batch, heads_q, L] (may be NULL).
 *   workspace: >= sizes.bwd_workspace_bytes (without a precision flag this includes fp16 copies of Q and K, for GQA groups
 *   also of V and dO: 2 bytes per element of those tensors).  No floating-point atomics are used: results are bitwise reproducible run to run. */
int vsa2_attn_bwd(const vsa2_params* p, const void* q, const void* k, const void* v, const float* gate,
                  const vsa2_map* map, const void* o, const float* lse, const vsa2_saved* saved,
                  const void* d_o, void* dq, void* dk, void* dv, float* dgate,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Cube-major copy of a tensor (Sec. 2.2 "Permutation": (T, H, W) -> (N_t N_h N_w) x (B_t B_h B_w)), for callers whose
 * surrounding code works in that layout; the entry points above take the raster layout and never need it.
 *   inverse == 0: src [batch, heads, L, D] raster -> dst [batch, heads, N * B, D]; cube n occupies rows n*B .. n*B+B-1, its
 *                 tokens in (b_t, b_h, b_w) order, positions outside the grid are written as zero
 *   inverse != 0: src [batch, heads, N * B, D] -> dst [batch, heads, L, D] (positions outside the grid are dropped)
 * Both bf16, device, 16-byte aligned; `heads` is heads_q or heads_kv of `p`; N and B as in vsa2_query_sizes.  Allocates
 * nothing; enqueues on `cuda_stream`. */
int vsa2_permute_cube_major(const vsa2_params* p, int32_t heads, int32_t inverse, const void* src, void* dst,
                            void* cuda_stream);

/* Gate projection of the gated merge (Sec. 2.2 "Gated Merge", Eq. 13): gate[b, h, l] = tanh(sum_c x[b, l, c] * w_g[c, h]),
 * one column of W_g per query head.  The layer that owns the hidden states calls this before vsa2_attn_fwd (which takes
 * the gate as an input) and vsa2_gate_bwd after vsa2_attn_bwd (which returns dgate).
 *   x     [batch, L, hidden]      bf16, device, 16-byte aligned; tokens in raster order, L = grid_t * grid_h * grid_w
 *   w_g   [hidden, heads_q]       bf16, device
 *   gate  [batch, heads_q, L]     fp32, device (written)
 * hidden must be a positive multiple of 8 and heads_q <= 64, else VSA2_ERR_UNSUPPORTED.  Only batch, heads_q and the grid of
 * `p` are used.  Allocates nothing; enqueues on `cuda_stream`. */
int vsa2_gate_fwd(const vsa2_params* p, int32_t hidden, const void* x, const void* w_g, float* gate, void* cuda_stream);

/* Backward of vsa2_gate_fwd.  With dz = dgate * (1 - gate^2):
 *   d_w_g [hidden, heads_q]       fp32, device (written): sum over batch and tokens of x[b, l, c] * dz[b, h, l]
 *   dx    [batch, L, hidden]      p->out_dtype, device, 16-byte aligned (written): sum_h dz[b, h, l] * w_g[c, h]
 *   gate, dgate [batch, heads_q, L] fp32, device: the output of vsa2_gate_fwd and the dgate of vsa2_attn_bwd
 *   workspace: device, 256-byte aligned, at least vsa2_gate_bwd_workspace_bytes(p, hidden) (dz in bf16 and the
 *   partial sums of d_w_g, which are added in a fixed order: results are bitwise reproducible).  Errors as for vsa2_gate_fwd, plus
 *   VSA2_ERR_WORKSPACE_TOO_SMALL / VSA2_ERR_MISALIGNED. */
size_t vsa2_gate_bwd_workspace_bytes(const vsa2_params* p, int32_t hidden);
int vsa2_gate_bwd(const vsa2_params* p, int32_t hidden, const void* x, const void* w_g, const float* gate,
                  const float* dgate, float* d_w_g, void* dx, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Synchronises `cuda_stream`, reads the status word at the start of `workspace` and stores it in
 * *status_out (host): VSA2_OK, VSA2_ERR_DEVICE_TIMEOUT or VSA2_ERR_MAP_OVERFLOW. */
int vsa2_device_status(const void* workspace, void* cuda_stream, int32_t* status_out);

/* Kernel groups, for timing from outside (e.g. a benchmark) without a profiler. */
enum {
  VSA2_KERNEL_POOL = 0,         /* vsa2_attn_fwd: cube means of Q, K, V (Eq. 1) */
  VSA2_KERNEL_ROUTER_LSE = 1,   /* router pass 1: row log-sum-exp (Eq. 6) */
  VSA2_KERNEL_ROUTER_POOL = 2,  /* router pass 2: softmax + G x G pooling (Eq. 6-7) */
  VSA2_KERNEL_SELECT = 3,       /* TopK + CSR/CSC (Eq. 8-9) */
  VSA2_KERNEL_COARSE_FWD = 4,   /* Eq. 2-3 */
  VSA2_KERNEL_FINE_FWD = 5,     /* Eq. 12 + Eq. 14 */
  VSA2_KERNEL_BWD_PRE = 6,      /* delta, dGate, dO_c_hat */
  VSA2_KERNEL_COARSE_BWD = 7,
  VSA2_KERNEL_FINE_BWD_DQ = 8,
  VSA2_KERNEL_FINE_BWD_DKV = 9,
  VSA2_KERNEL_POOL_ROUTER = 10, /* vsa2_route: sub-cube means of Q, K (Eq. 5) */
  VSA2_KERNEL_COUNT = 11
};

/* Asks the library to record `start_event` before and `stop_event` after the launches of one kernel
 * group (cudaEvent_t handles passed as void*, recorded on the stream of the call that launches them) in
 * every later call, until cleared by passing NULL events.  The paper has no counterpart: this is a
 * measurement hook.  Process-global and not thread-safe. */
int vsa2_profile_events(int32_t kernel_id, void* start_event, void* stop_event);

/* Number of kernels this library has launched in this process so far. */
int64_t vsa2_launch_count(void);

/* Diagnostic: runs, in one CTA, the two tensor-core products the attention kernels are built from, on
 * real cube tiles of batch 0 / head 0 fetched by TMA: S^T = K_pair Q^T (fp32 [128, 64]; K_pair = the 64-token
 * tiles of cubes cube_a and cube_b stacked) and O^T = V_pair^T P^T (fp32 [128, 64]; rows are head channels, with
 * head_dim 64 rows 64..127 repeat rows 0..63), where p_t is a bf16 [128, 64] matrix supplied by the caller.
 * k_tile_dump receives the raw shared-memory image of the K pair (2 * head_dim/64 * 8 KB).  `status` is a device
 * int32 set to VSA2_ERR_DEVICE_TIMEOUT if a bounded wait ran out.  The paper has no counterpart. */
int vsa2_selftest_umma(const vsa2_params* p, const void* q, const void* k, const void* v, int32_t cube_q,
                       int32_t cube_a, int32_t cube_b, const void* p_t, float* s_t_out, float* o_t_out,
                       void* k_tile_dump, int32_t* status, void* cuda_stream);

/* Diagnostic of the bounded-wait discipline (the paper has no counterpart).  Every device-side wait of the attention
 * kernels gives up after a time limit: the CTA raises an abort flag, all its roles leave, the status word becomes
 * VSA2_ERR_DEVICE_TIMEOUT and tensor memory is released.  This call runs that path alone, in one CTA: one thread waits
 * `limit_us` microseconds (1 .. 100000) on a barrier nothing arrives at, a second thread waits on another barrier with the
 * kernels' own 2 s limit and must be released by the first one's abort flag.  `status` (device int32, caller-zeroed)
 * receives VSA2_ERR_DEVICE_TIMEOUT; `waited_ns` (device uint64, may be NULL) the time the first wait took.  No GPU fault,
 * trap or hang is involved and the context stays usable. */
int vsa2_selftest_timeout(uint32_t limit_us, int32_t* status, uint64_t* waited_ns, void* cuda_stream);

/* Host-only diagnostic (no GPU, no CUDA call; the paper has no counterpart): the kernels decode cube and token indices with
 * q = floor(n * ceil(2^32 / d) / 2^32) instead of a division.  Checks that quotient against n / d for every 0 <= n <= n_max
 * and every divisor d_min .. d_exhaustive, and for the divisors up to d_max at every multiple of d and its two neighbours.
 * Returns the number of wrong quotients (0 for n_max * d_max < 2^32; the library's n stay below 2^22, its d below 2^10). */
int64_t vsa2_selftest_divmod(int32_t n_max, int32_t d_min, int32_t d_exhaustive, int32_t d_max);

/* Test hook (the paper has no counterpart): number of query blocks the forward kernels may hand to the exact-maximum
 * fall-back per call, 1 .. 16384 (default 16384, which also sizes the workspace).  When more blocks than that leave the
 * safe range of the fixed-reference softmax, the surplus is not recomputed, the status word becomes VSA2_ERR_UNSUPPORTED
 * and nothing outside the list is read or written.  Process-global; returns the value now in force. */
int32_t vsa2_debug_rescue_capacity(int32_t capacity);

/* Text of the CUDA error behind the most recent VSA2_ERR_CUDA returned in this process ("no error" if none). */
const char* vsa2_last_cuda_error(void);

/* Static string for an error code. */
const char* vsa2_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* VSA2_H_ */
