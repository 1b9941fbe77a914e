"""CPU oracle for VSA2 routed block-sparse attention (forward and backward).

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64 numpy
restatement of what the paper defines, written to be checked against the paper
by eye.  It shares no code with the CUDA path and neither imports the other.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it.

What the paper fixes and where (section / equation of the VSA2 paper):

* dense attention S = Q K^T / sqrt(D), P = softmax(S + M), O = P V      -- Sec. 2.1
* block mask M with one value per (B, B) tile                            -- Sec. 2.1
* cube-major token order, cube index n = (n_t N_h + n_h) N_w + n_w       -- Sec. 2.2 "Permutation"
* coarse branch: mean-pool over cubes, N x N softmax attention, repeat   -- Sec. 2.2 Eq. 1-4
* router: mean-pool over R sub-cubes, softmax, G x G mean-pool           -- Sec. 2.2 Eq. 5-7
* per-sequence TopK over the flattened N*N scores, N*K blocks kept       -- Sec. 2.2 Eq. 8-9
* fine branch: block-sparse attention over the kept pairs                -- Sec. 2.2 Eq. 12
* gated merge O = G * O_c + O_f, gate G = tanh(X W_g)                    -- Sec. 2.2 Eq. 13-14
* padding to whole cubes, padded tokens masked                           -- Sec. 2.2 "Kernel Implementation"
* the routing decision carries no gradient                               -- Sec. 2.1 (last paragraph)

Readings taken where the paper is silent.  The paper cannot confirm them; what the
tests pin is that each function computes exactly the reading stated here:

* padding: every mean runs over valid tokens only; padded keys and empty key
  sub-cubes are excluded from every softmax; the router's G x G mean divides by
  (valid query sub-cubes of the cube) x (full G).  Pinned on padded grids by
  library pooling of a zero-padded volume and of a volume of ones, and by a
  brute-force softmax with an explicit -inf mask.
* router operands: the pooled Q_r, K_r are rounded to bf16 (round to nearest
  even) after an fp32 sum taken in a fixed order (along w, then h, then t) and
  an fp32 division by the valid count.  Pinned by torch's bf16 cast and by a
  constructed case in which the order of the sum decides the result.
* ties in TopK go to the lower flat index i*N + j.  Pinned by Python's sort.
* a query block with no selected KV block gets O_f = 0 and lse = -inf.  Pinned by
  the dense masked restatement with an empty mask row.
* gate projection: X [L, C] are the layer's hidden states (C = model width) and
  W_g has one column per query head, W_g [C, H_q], so that G [H_q, L] holds the
  per-token per-head gate of Eq. 13 (the paper writes one head: W_g in R^{D x 1}).
* text tokens (Sec. 2.2, the sentence after Eq. 12): one softmax per row over the kept video blocks plus all text
  keys (video queries) or over everything (text queries); see `joint_*` below.  Pinned by SDPA over the
  concatenated sequence, by the log-sum-exp merge identity and by autograd.
Every function here is pinned by tests/test_oracle_pins.py.
"""
from __future__ import annotations

import numpy as np

PER_SEQUENCE = 0       # Eq. 8-9: N*K largest of the flattened N*N scores
PER_QUERY = 1          # Sec. 2.1 (VSA form): K largest per query block (row)
PER_QUERY_BUDGET = 2   # row i keeps its own k_i largest


# ----------------------------------------------------------------------------
# bf16 helpers (the inputs of the method are bf16 bit patterns)
# ----------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def round_f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 value (ties to even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


# ----------------------------------------------------------------------------
# geometry of the latent grid (Table 1 of the paper: T,H,W / B / N / R / G)
# ----------------------------------------------------------------------------
class Geometry:
    """Index maps between raster token order l = (t*H + h)*W + w and cubes.

    cube index    n = (n_t*N_h + n_h)*N_w + n_w            (Sec. 2.2 "Permutation")
    sub-cube idx  g = (g_t*G_h + g_h)*G_w + g_w inside a cube, G_x = B_x / R_x
    The grid is padded up to whole cubes; only valid tokens exist in the arrays.
    """

    def __init__(self, grid, cube=(4, 4, 4), rpool=(2, 2, 2)):
        self.T, self.H, self.W = (int(v) for v in grid)
        self.Bt, self.Bh, self.Bw = (int(v) for v in cube)
        self.Rt, self.Rh, self.Rw = (int(v) for v in rpool)
        for b, r in zip(cube, rpool):
            if b % r:
                raise ValueError("router pool must divide the cube")
        self.L = self.T * self.H * self.W
        self.B = self.Bt * self.Bh * self.Bw
        self.Nt = -(-self.T // self.Bt)
        self.Nh = -(-self.H // self.Bh)
        self.Nw = -(-self.W // self.Bw)
        self.N = self.Nt * self.Nh * self.Nw
        self.Gt, self.Gh, self.Gw = self.Bt // self.Rt, self.Bh // self.Rh, self.Bw // self.Rw
        self.G = self.Gt * self.Gh * self.Gw
        l = np.arange(self.L)
        t, h, w = l // (self.H * self.W), (l // self.W) % self.H, l % self.W
        self.cube_of = ((t // self.Bt) * self.Nh + (h // self.Bh)) * self.Nw + (w // self.Bw)
        bt, bh, bw = t % self.Bt, h % self.Bh, w % self.Bw
        self.sub_of = ((bt // self.Rt) * self.Gh + (bh // self.Rh)) * self.Gw + (bw // self.Rw)
        # raster indices of the valid tokens of each cube, in (b_t, b_h, b_w) order
        pos = (bt * self.Bh + bh) * self.Bw + bw
        order = np.lexsort((pos, self.cube_of))
        counts = np.bincount(self.cube_of, minlength=self.N)
        self.cube_count = counts
        starts = np.concatenate(([0], np.cumsum(counts)))
        self.cube_tokens = [order[starts[n]:starts[n + 1]] for n in range(self.N)]
        self.sub_count = np.zeros((self.N, self.G), dtype=np.int64)
        np.add.at(self.sub_count, (self.cube_of, self.sub_of), 1)

    def raster_index(self, t, h, w):
        return (t * self.H + h) * self.W + w


# ----------------------------------------------------------------------------
# Sec. 2.2 "Permutation": cube-major token order
# ----------------------------------------------------------------------------
def to_cube_major(X: np.ndarray, geo: Geometry, fill=0.0) -> np.ndarray:
    """X [L, D] in raster order -> [N * B, D]: cube n occupies rows n*B .. n*B + B - 1, its tokens in (b_t, b_h, b_w)
    order; positions outside the grid hold `fill`."""
    Y = np.full((geo.N * geo.B, X.shape[1]), fill, dtype=X.dtype)
    l = np.arange(geo.L)
    t, h, w = l // (geo.H * geo.W), (l // geo.W) % geo.H, l % geo.W
    pos = ((t % geo.Bt) * geo.Bh + (h % geo.Bh)) * geo.Bw + (w % geo.Bw)
    Y[geo.cube_of * geo.B + pos] = X
    return Y


def from_cube_major(Y: np.ndarray, geo: Geometry) -> np.ndarray:
    """Inverse of to_cube_major on the valid tokens: [N * B, D] -> [L, D]."""
    l = np.arange(geo.L)
    t, h, w = l // (geo.H * geo.W), (l // geo.W) % geo.H, l % geo.W
    pos = ((t % geo.Bt) * geo.Bh + (h % geo.Bh)) * geo.Bw + (w % geo.Bw)
    return Y[geo.cube_of * geo.B + pos]


# ----------------------------------------------------------------------------
# Eq. 1: coarse mean pooling over cubes
# ----------------------------------------------------------------------------
def mean_pool_cube(X: np.ndarray, geo: Geometry) -> np.ndarray:
    """X [L, D] -> X_c [N, D]: mean over the valid tokens of each cube."""
    Xc = np.zeros((geo.N, X.shape[1]), dtype=np.float64)
    for n in range(geo.N):
        Xc[n] = X[geo.cube_tokens[n]].sum(axis=0) / geo.cube_count[n]
    return Xc


# ----------------------------------------------------------------------------
# Eq. 5: router mean pooling over R sub-cubes (bf16 operands, fixed fp32 order)
# ----------------------------------------------------------------------------
def mean_pool_router(X: np.ndarray, geo: Geometry):
    """X [L, D] (bf16-exact values) -> (X_r [N, G, D] float64 holding bf16 values,
    valid [N, G] bool).

    The sum over a sub-cube runs in float32: first along w left to right, then
    along h, then along t; tokens outside the grid add +0.  The float32 sum is
    divided (IEEE float32 division) by the number of valid tokens and rounded
    to bf16, ties to even.
    """
    D = X.shape[1]
    X32 = X.astype(np.float32)
    # scatter into a zero-padded [T_pad, H_pad, W_pad, D] volume
    Tp, Hp, Wp = geo.Nt * geo.Bt, geo.Nh * geo.Bh, geo.Nw * geo.Bw
    vol = np.zeros((Tp, Hp, Wp, D), dtype=np.float32)
    vol[:geo.T, :geo.H, :geo.W] = X32.reshape(geo.T, geo.H, geo.W, D)
    ones = np.zeros((Tp, Hp, Wp), dtype=np.int64)
    ones[:geo.T, :geo.H, :geo.W] = 1
    # reduce along w, then h, then t, each left to right, all in float32
    v = vol.reshape(Tp, Hp, Wp // geo.Rw, geo.Rw, D)
    acc = v[:, :, :, 0]
    for i in range(1, geo.Rw):
        acc = acc + v[:, :, :, i]
    v = acc.reshape(Tp, Hp // geo.Rh, geo.Rh, Wp // geo.Rw, D)
    acc = v[:, :, 0]
    for i in range(1, geo.Rh):
        acc = acc + v[:, :, i]
    v = acc.reshape(Tp // geo.Rt, geo.Rt, Hp // geo.Rh, Wp // geo.Rw, D)
    acc = v[:, 0]
    for i in range(1, geo.Rt):
        acc = acc + v[:, i]
    assert acc.dtype == np.float32
    cnt = ones.reshape(Tp // geo.Rt, geo.Rt, Hp // geo.Rh, geo.Rh, Wp // geo.Rw, geo.Rw).sum(axis=(1, 3, 5))
    with np.errstate(invalid="ignore", divide="ignore"):
        mean = acc / cnt.astype(np.float32)[..., None]
    mean = np.where(cnt[..., None] > 0, mean, np.float32(0)).astype(np.float32)
    mean = round_f32_to_bf16(mean)
    # [Nt*Gt, Nh*Gh, Nw*Gw, D] -> [N, G, D]
    m = mean.reshape(geo.Nt, geo.Gt, geo.Nh, geo.Gh, geo.Nw, geo.Gw, D)
    m = m.transpose(0, 2, 4, 1, 3, 5, 6).reshape(geo.N, geo.G, D)
    c = cnt.reshape(geo.Nt, geo.Gt, geo.Nh, geo.Gh, geo.Nw, geo.Gw)
    c = c.transpose(0, 2, 4, 1, 3, 5).reshape(geo.N, geo.G)
    assert np.array_equal(c, geo.sub_count)
    return m.astype(np.float64), c > 0


# ----------------------------------------------------------------------------
# Eq. 6-7: pool - softmax - pool router scores
# ----------------------------------------------------------------------------
def router_block_scores(Qr, Kr, q_valid, k_valid, scale) -> np.ndarray:
    """Q_r, K_r [N, G, D], validity [N, G] -> P_r [N, N].

    p_hat = row softmax of Q_r K_r^T * scale over all valid router keys of the
    sequence (Eq. 6); P_r[i, j] is its mean over the G x G sub-block of cube
    pair (i, j) (Eq. 7): sum over valid query and key sub-cubes divided by
    (number of valid query sub-cubes of cube i) * G.
    """
    N, G, D = Qr.shape
    q = Qr.reshape(N * G, D)
    k = Kr.reshape(N * G, D)
    s = (q @ k.T) * scale
    s[:, ~k_valid.reshape(-1)] = -np.inf
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    p_hat = e / e.sum(axis=1, keepdims=True)
    p_hat[~q_valid.reshape(-1), :] = 0.0
    block_sum = p_hat.reshape(N, G, N, G).sum(axis=(1, 3))
    g_i = q_valid.sum(axis=1).astype(np.float64)
    return block_sum / (g_i[:, None] * G)


# ----------------------------------------------------------------------------
# Eq. 8-9 (and the per-row VSA form): TopK -> boolean block mask
# ----------------------------------------------------------------------------
def select_blocks(P_r, mode, topk=0, budgets=None) -> np.ndarray:
    """P_r [N, N] -> bool mask [N, N] (True = block pair kept).

    The decision is taken on float32 scores (the kernel's precision); among
    equal scores the lower flat index i*N + j wins.  K is clamped to N.
    """
    N = P_r.shape[0]
    p = P_r.astype(np.float32)
    mask = np.zeros((N, N), dtype=bool)
    if mode == PER_SEQUENCE:
        keep = N * min(int(topk), N)
        order = np.argsort(-p.reshape(-1), kind="stable")[:keep]
        mask.reshape(-1)[order] = True
    elif mode in (PER_QUERY, PER_QUERY_BUDGET):
        for i in range(N):
            k_i = int(topk) if mode == PER_QUERY else int(budgets[i])
            k_i = max(0, min(k_i, N))
            order = np.argsort(-p[i], kind="stable")[:k_i]
            mask[i, order] = True
    else:
        raise ValueError("unknown selection mode")
    return mask


def mask_to_csr(mask):
    """bool [N, N] -> (row_ptr [N+1], col_idx [nnz]), columns ascending per row."""
    N = mask.shape[0]
    counts = mask.sum(axis=1)
    row_ptr = np.concatenate(([0], np.cumsum(counts))).astype(np.int32)
    col_idx = np.concatenate([np.nonzero(mask[i])[0] for i in range(N)] + [np.zeros(0, np.int64)])
    return row_ptr, col_idx.astype(np.int32)


def mask_to_csc(mask):
    """bool [N, N] -> (col_ptr [N+1], row_idx [nnz]), rows ascending per column."""
    return mask_to_csr(mask.T)


# ----------------------------------------------------------------------------
# Eq. 2-3: coarse branch attention on the pooled tokens
# ----------------------------------------------------------------------------
def coarse_attention(Qc, Kc, Vc, scale):
    """[N, D] pooled tensors -> (O_c_hat [N, D], lse_c [N])."""
    s = (Qc @ Kc.T) * scale
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    return (e / l) @ Vc, (m + np.log(l))[:, 0]


# ----------------------------------------------------------------------------
# Eq. 12: fine branch, block-sparse attention over the kept block pairs
# ----------------------------------------------------------------------------
def fine_attention(Q, K, V, mask, geo: Geometry, scale, rows=None):
    """Q, K, V [L, D], mask [N, N] -> (O_f [L, D], lse [L]).

    Query tokens of cube i attend the valid tokens of every cube j with
    mask[i, j]; softmax at token level over exactly those keys.  A cube with
    no kept block gets O_f = 0 and lse = -inf.  `rows` restricts the work to
    some query cubes (the others stay 0 / -inf).
    """
    L, D = Q.shape
    O_f = np.zeros((L, D), dtype=np.float64)
    lse = np.full(L, -np.inf, dtype=np.float64)
    for i in (range(geo.N) if rows is None else rows):
        cols = np.nonzero(mask[i])[0]
        if cols.size == 0:
            continue
        qt = geo.cube_tokens[i]
        kt = np.concatenate([geo.cube_tokens[j] for j in cols])
        s = (Q[qt] @ K[kt].T) * scale
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        l = e.sum(axis=1, keepdims=True)
        O_f[qt] = (e / l) @ V[kt]
        lse[qt] = (m + np.log(l))[:, 0]
    return O_f, lse


# ----------------------------------------------------------------------------
# Sec. 2.2 "Fine Branch", the sentence after Eq. 12: text tokens (MMDiT)
# ----------------------------------------------------------------------------
# Video and text tokens share one attention space.  Reading taken (the paper gives one sentence): the block map M
# covers video-video pairs only; every video query additionally attends ALL text keys, and every text query attends
# all video keys and all text keys, each row with ONE softmax over its whole key set.  Text tokens take no part in
# the coarse branch, the router or the gate: a text query's output is its fine-branch output.
def joint_fine_attention(Q, K, V, Qt, Kt, Vt, mask, geo: Geometry, scale, rows=None, text_rows=None):
    """Video Q, K, V [L, D], text Qt, Kt, Vt [Lt, D], mask [N, N] -> (O_f [L, D], lse [L], O_t [Lt, D], lse_t [Lt]).

    Video queries of cube i: softmax over the valid tokens of the kept cubes of row i followed by all text tokens.
    Text queries: softmax over all video tokens followed by all text tokens.  `rows` / `text_rows` restrict the work to
    some video query cubes / text query tokens (the others stay 0 / -inf).
    """
    L, D = Q.shape
    Lt = Qt.shape[0]
    O_f = np.zeros((L, D), dtype=np.float64)
    lse = np.full(L, -np.inf, dtype=np.float64)
    for i in (range(geo.N) if rows is None else rows):
        cols = np.nonzero(mask[i])[0]
        qt = geo.cube_tokens[i]
        kt = np.concatenate([geo.cube_tokens[j] for j in cols] + [np.zeros(0, np.int64)]).astype(np.int64)
        Kk = np.concatenate([K[kt], Kt])
        Vv = np.concatenate([V[kt], Vt])
        if Kk.shape[0] == 0:
            continue
        s = (Q[qt] @ Kk.T) * scale
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        l = e.sum(axis=1, keepdims=True)
        O_f[qt] = (e / l) @ Vv
        lse[qt] = (m + np.log(l))[:, 0]
    O_t = np.zeros((Lt, D), dtype=np.float64)
    lse_t = np.full(Lt, -np.inf, dtype=np.float64)
    tr = np.arange(Lt) if text_rows is None else np.asarray(text_rows, dtype=np.int64)
    if tr.size:
        Kk = np.concatenate([K, Kt])
        Vv = np.concatenate([V, Vt])
        s = (Qt[tr] @ Kk.T) * scale
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        l = e.sum(axis=1, keepdims=True)
        O_t[tr] = (e / l) @ Vv
        lse_t[tr] = (m + np.log(l))[:, 0]
    return O_f, lse, O_t, lse_t


def joint_fine_backward(Q, K, V, Qt, Kt, Vt, mask, geo: Geometry, scale, dO, dOt, lse, O_f, lse_t, O_t,
                        rows=None, text_rows=None):
    """Backward of joint_fine_attention for the video query cubes in `rows` and the text queries in `text_rows` (all if
    None).  Same formulas as fine_backward, over each row's whole key set.  Returns dQ, dK, dV [L, D] and dQt, dKt, dVt
    [Lt, D] (the key / value gradients hold only the contributions of the visited queries)."""
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    dQt, dKt, dVt = np.zeros_like(Qt), np.zeros_like(Kt), np.zeros_like(Vt)
    delta = (dO * O_f).sum(axis=1)
    for i in (range(geo.N) if rows is None else rows):
        cols = np.nonzero(mask[i])[0]
        qt = geo.cube_tokens[i]
        kt = np.concatenate([geo.cube_tokens[j] for j in cols] + [np.zeros(0, np.int64)]).astype(np.int64)
        nv = kt.size
        Kk = np.concatenate([K[kt], Kt])
        Vv = np.concatenate([V[kt], Vt])
        if Kk.shape[0] == 0:
            continue
        s = (Q[qt] @ Kk.T) * scale
        P = np.exp(s - lse[qt][:, None])
        dVv = P.T @ dO[qt]
        dP = dO[qt] @ Vv.T
        dS = P * (dP - delta[qt][:, None])
        dQ[qt] += (dS @ Kk) * scale
        dKk = (dS.T @ Q[qt]) * scale
        dK[kt] += dKk[:nv]
        dV[kt] += dVv[:nv]
        dKt += dKk[nv:]
        dVt += dVv[nv:]
    tr = np.arange(Qt.shape[0]) if text_rows is None else np.asarray(text_rows, dtype=np.int64)
    if tr.size:
        L = K.shape[0]
        Kk = np.concatenate([K, Kt])
        Vv = np.concatenate([V, Vt])
        delta_t = (dOt[tr] * O_t[tr]).sum(axis=1)
        s = (Qt[tr] @ Kk.T) * scale
        P = np.exp(s - lse_t[tr][:, None])
        dVv = P.T @ dOt[tr]
        dP = dOt[tr] @ Vv.T
        dS = P * (dP - delta_t[:, None])
        dQt[tr] += (dS @ Kk) * scale
        dKk = (dS.T @ Qt[tr]) * scale
        dK += dKk[:L]
        dV += dVv[:L]
        dKt += dKk[L:]
        dVt += dVv[L:]
    return dQ, dK, dV, dQt, dKt, dVt


def joint_head_forward(Q, K, V, Qt, Kt, Vt, gate, mask, geo: Geometry, scale):
    """The whole operator with text tokens for one head: coarse branch and merge on the video tokens as in head_forward
    (Eq. 1-4, 14), fine branch by joint_fine_attention.  Returns the dict of head_forward plus O_t, lse_t."""
    Qc, Kc, Vc = mean_pool_cube(Q, geo), mean_pool_cube(K, geo), mean_pool_cube(V, geo)
    Oc_hat, lse_c = coarse_attention(Qc, Kc, Vc, scale)
    O_f, lse, O_t, lse_t = joint_fine_attention(Q, K, V, Qt, Kt, Vt, mask, geo, scale)
    O = gate[:, None] * Oc_hat[geo.cube_of] + O_f
    return dict(O=O, O_f=O_f, lse=lse, O_t=O_t, lse_t=lse_t, Oc_hat=Oc_hat, lse_c=lse_c, Qc=Qc, Kc=Kc, Vc=Vc)


def joint_head_backward(Q, K, V, Qt, Kt, Vt, gate, mask, geo: Geometry, scale, dO, dOt, fwd=None):
    """Gradients of sum(O * dO) + sum(O_t * dOt) for one head given the block mask: coarse path as in head_backward,
    fine path by joint_fine_backward.  Returns dQ, dK, dV, dGate (video) and dQt, dKt, dVt (text)."""
    if fwd is None:
        fwd = joint_head_forward(Q, K, V, Qt, Kt, Vt, gate, mask, geo, scale)
    c = coarse_path_backward(Q, K, V, gate, geo, scale, dO, fwd)
    fq, fk, fv, tq, tk, tv = joint_fine_backward(Q, K, V, Qt, Kt, Vt, mask, geo, scale, dO, dOt, fwd["lse"], fwd["O_f"],
                                                 fwd["lse_t"], fwd["O_t"])
    return dict(dQ=c["dQ"] + fq, dK=c["dK"] + fk, dV=c["dV"] + fv, dGate=c["dGate"], dQt=tq, dKt=tk, dVt=tv)


# ----------------------------------------------------------------------------
# whole operator, one (batch, query head): Eq. 1-4, 12, 14
# ----------------------------------------------------------------------------
def head_forward(Q, K, V, gate, mask, geo: Geometry, scale):
    """Returns dict with O, O_f, lse, O_c_hat, lse_c, Q_c, K_c, V_c for one head."""
    Qc, Kc, Vc = mean_pool_cube(Q, geo), mean_pool_cube(K, geo), mean_pool_cube(V, geo)
    Oc_hat, lse_c = coarse_attention(Qc, Kc, Vc, scale)                  # Eq. 2-3
    O_f, lse = fine_attention(Q, K, V, mask, geo, scale)                 # Eq. 12
    O_c = Oc_hat[geo.cube_of]                                            # Eq. 4 (Repeat_B)
    O = gate[:, None] * O_c + O_f                                        # Eq. 14
    return dict(O=O, O_f=O_f, lse=lse, Oc_hat=Oc_hat, lse_c=lse_c, Qc=Qc, Kc=Kc, Vc=Vc)


def coarse_path_backward(Q, K, V, gate, geo: Geometry, scale, dO, fwd):
    """Backward of the merge, repeat, coarse attention and cube pooling (Eq. 14, 4, 3, 2, 1).

    Returns dGate [L] and the coarse branch's contribution to dQ, dK, dV [L, D].
    """
    Oc_hat, Qc, Kc, Vc = fwd["Oc_hat"], fwd["Qc"], fwd["Kc"], fwd["Vc"]
    # merge (Eq. 14) and repeat (Eq. 4)
    dGate = (dO * Oc_hat[geo.cube_of]).sum(axis=1)
    dOc_hat = np.zeros_like(Oc_hat)
    np.add.at(dOc_hat, geo.cube_of, gate[:, None] * dO)
    # coarse attention backward (Eq. 2-3): dense softmax attention on N tokens
    s = (Qc @ Kc.T) * scale
    Pc = np.exp(s - fwd["lse_c"][:, None])
    dVc = Pc.T @ dOc_hat
    dPc = dOc_hat @ Vc.T
    delta_c = (dOc_hat * Oc_hat).sum(axis=1, keepdims=True)
    dSc = Pc * (dPc - delta_c)
    dQc = (dSc @ Kc) * scale
    dKc = (dSc.T @ Qc) * scale
    # mean-pool backward (Eq. 1): every valid token gets grad / count of its cube
    inv = 1.0 / geo.cube_count[geo.cube_of][:, None]
    return dict(dGate=dGate, dQ=dQc[geo.cube_of] * inv, dK=dKc[geo.cube_of] * inv, dV=dVc[geo.cube_of] * inv)


def fine_backward(Q, K, V, mask, geo: Geometry, scale, dO, lse, O_f, rows=None):
    """Backward of Eq. 12 for the query cubes in `rows` (all if None).

    With P = exp(S - lse), delta = rowsum(dO * O_f), dP = dO V^T, dS = P * (dP - delta):
    dQ = dS K * scale, dK = dS^T Q * scale, dV = P^T dO.  Returns the three [L, D] arrays
    (dK and dV hold only the contributions of the visited query cubes).
    """
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    delta = (dO * O_f).sum(axis=1)
    for i in (range(geo.N) if rows is None else rows):
        cols = np.nonzero(mask[i])[0]
        if cols.size == 0:
            continue
        qt = geo.cube_tokens[i]
        kt = np.concatenate([geo.cube_tokens[j] for j in cols])
        s = (Q[qt] @ K[kt].T) * scale
        P = np.exp(s - lse[qt][:, None])
        dV[kt] += P.T @ dO[qt]
        dP = dO[qt] @ V[kt].T
        dS = P * (dP - delta[qt][:, None])
        dQ[qt] += (dS @ K[kt]) * scale
        dK[kt] += (dS.T @ Q[qt]) * scale
    return dQ, dK, dV


def fine_backward_kv_cubes(Q, K, V, mask, geo: Geometry, scale, dO, kv_cubes):
    """Fine-branch dK, dV restricted to the tokens of the KV cubes in `kv_cubes`.

    Visits every query cube that keeps one of those KV cubes, runs its forward (over all of its
    kept blocks, to get lse and delta) and adds its gradient contribution to the requested
    cubes only.  Same formulas as fine_backward; used where the full backward is too slow.
    """
    dK, dV = np.zeros_like(K), np.zeros_like(V)
    kv_cubes = list(kv_cubes)
    rows = np.nonzero(mask[:, kv_cubes].any(axis=1))[0]
    O_f, lse = fine_attention(Q, K, V, mask, geo, scale, rows=rows)
    delta = (dO * O_f).sum(axis=1)
    for i in rows:
        qt = geo.cube_tokens[i]
        for j in kv_cubes:
            if not mask[i, j]:
                continue
            kt = geo.cube_tokens[j]
            s = (Q[qt] @ K[kt].T) * scale
            P = np.exp(s - lse[qt][:, None])
            dV[kt] += P.T @ dO[qt]
            dP = dO[qt] @ V[kt].T
            dS = P * (dP - delta[qt][:, None])
            dK[kt] += (dS.T @ Q[qt]) * scale
    return dK, dV


def head_backward(Q, K, V, gate, mask, geo: Geometry, scale, dO, fwd=None):
    """Gradients of sum(O * dO) for one (batch, query head) given the block mask.

    Chain rule on Eq. 14, 4, 3, 2, 1 (coarse path) and on Eq. 12 (fine path).
    The mask is a constant: nothing flows through Eq. 5-9.
    Returns dQ, dK, dV [L, D] (dK, dV are this query head's contribution) and dGate [L].
    """
    if fwd is None:
        fwd = head_forward(Q, K, V, gate, mask, geo, scale)
    c = coarse_path_backward(Q, K, V, gate, geo, scale, dO, fwd)
    fq, fk, fv = fine_backward(Q, K, V, mask, geo, scale, dO, fwd["lse"], fwd["O_f"])
    return dict(dQ=c["dQ"] + fq, dK=c["dK"] + fk, dV=c["dV"] + fv, dGate=c["dGate"])


# ----------------------------------------------------------------------------
# multi-head wrappers ([B, H, L, D] arrays; query head hq uses KV head hq // (Hq/Hkv))
# ----------------------------------------------------------------------------
def route(Q, K, geo: Geometry, scale, mode, topk=0, budgets=None, return_scores=False, share_group=False):
    """Q [B, Hq, L, D], K [B, Hkv, L, D] -> mask [B, Hq, N, N] (and P_r if asked).

    Each query head routes on its own against its KV head's pooled keys; the
    budget N*K holds per (batch, query head).

    share_group: the "group head" pattern of the ablation in Sec. 4 -- the query
    heads of one KV group share one map.  The block scores of the group's heads
    are added (the paper does not say how the heads are combined; the sum, or
    equivalently the mean, is the reading taken) and the TopK runs once per
    group; the scores returned are then the group sums, repeated per head.
    """
    Bn, Hq = Q.shape[:2]
    rep = Hq // K.shape[1]
    masks = np.zeros((Bn, Hq, geo.N, geo.N), dtype=bool)
    scores = np.zeros((Bn, Hq, geo.N, geo.N), dtype=np.float64)
    for b in range(Bn):
        kr_cache = {}
        for hq in range(Hq):
            hk = hq // rep
            if hk not in kr_cache:
                kr_cache[hk] = mean_pool_router(K[b, hk], geo)
            Kr, kv = kr_cache[hk]
            Qr, qv = mean_pool_router(Q[b, hq], geo)
            scores[b, hq] = router_block_scores(Qr, Kr, qv, kv, scale)
        if share_group:
            if budgets is not None:
                raise ValueError("per-row budgets belong to single heads: not defined for shared maps")
            for hk in range(Hq // rep):
                grp = slice(hk * rep, (hk + 1) * rep)
                scores[b, grp] = scores[b, grp].sum(axis=0, keepdims=True)
        for hq in range(Hq):
            bud = None if budgets is None else budgets[b, hq]
            masks[b, hq] = select_blocks(scores[b, hq], mode, topk, bud)
    return (masks, scores) if return_scores else masks


def forward(Q, K, V, gate, masks, geo: Geometry, scale):
    """[B, H, L, D] inputs, gate [B, Hq, L], masks [B, Hq, N, N] -> O [B,Hq,L,D], lse [B,Hq,L]."""
    Bn, Hq, L, D = Q.shape
    rep = Hq // K.shape[1]
    O = np.zeros((Bn, Hq, L, D))
    lse = np.zeros((Bn, Hq, L))
    for b in range(Bn):
        for hq in range(Hq):
            r = head_forward(Q[b, hq], K[b, hq // rep], V[b, hq // rep], gate[b, hq], masks[b, hq], geo, scale)
            O[b, hq], lse[b, hq] = r["O"], r["lse"]
    return O, lse


def backward(Q, K, V, gate, masks, geo: Geometry, scale, dO):
    """Gradients w.r.t. Q, K, V, gate; dK and dV are summed over the query heads of a group."""
    Bn, Hq, L, D = Q.shape
    rep = Hq // K.shape[1]
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    dGate = np.zeros((Bn, Hq, L))
    for b in range(Bn):
        for hq in range(Hq):
            hk = hq // rep
            g = head_backward(Q[b, hq], K[b, hk], V[b, hk], gate[b, hq], masks[b, hq], geo, scale, dO[b, hq])
            dQ[b, hq] = g["dQ"]
            dK[b, hk] += g["dK"]
            dV[b, hk] += g["dV"]
            dGate[b, hq] = g["dGate"]
    return dQ, dK, dV, dGate


# ----------------------------------------------------------------------------
# Appendix "Sparsity Computation", Eq. 15-16
# ----------------------------------------------------------------------------
# ----------------------------------------------------------------------------
# Eq. 13: the gate projection and its backward
# ----------------------------------------------------------------------------
def gate_forward(X: np.ndarray, Wg: np.ndarray) -> np.ndarray:
    """X [L, C] hidden states, W_g [C, H] -> gate [H, L] = tanh(X W_g)^T (Eq. 13, one column of W_g per head)."""
    return np.tanh(X @ Wg).T


def gate_backward(X: np.ndarray, Wg: np.ndarray, dgate: np.ndarray):
    """dgate [H, L] -> (dX [L, C], dW_g [C, H]).  With z = X W_g and gate = tanh(z): dz = dgate * (1 - gate^2),
    dX = dz W_g^T, dW_g = X^T dz."""
    gate = np.tanh(X @ Wg)                 # [L, H]
    dz = dgate.T * (1.0 - gate * gate)     # [L, H]
    return dz @ Wg.T, X.T @ dz


def fine_cost_fraction(K, B, L):
    """Fine-branch cost relative to dense attention: N K B^2 / L^2 = K B / L (Eq. 15)."""
    return K * B / L


def sparsity(K, B, R, L):
    """1 - (1/R^2 + K B / L)  (Eq. 16)."""
    return 1.0 - (1.0 / R ** 2 + K * B / L)
