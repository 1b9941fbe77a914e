"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types an oracle formula: every expected value comes from a
library routine (torch softmax / scaled_dot_product_attention / avg_pool / autograd /
bf16 cast, Python's sort), from a closed form, from a value printed in the paper, or
from brute force on a tiny case.
"""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import inputs as syn

torch.set_num_threads(max(1, os.cpu_count() or 1))
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# independent helpers: layout by reshape/permute (never the oracle's index formula)
# ---------------------------------------------------------------------------
def pad_volume(x, grid, cube, fill=0.0):
    """x [L, ...] raster -> padded volume [Tp, Hp, Wp, ...]."""
    T, H, W = grid
    Tp, Hp, Wp = (-(-g // c) * c for g, c in zip(grid, cube))
    vol = np.full((Tp, Hp, Wp) + x.shape[1:], fill, dtype=x.dtype)
    vol[:T, :H, :W] = x.reshape((T, H, W) + x.shape[1:])
    return vol


def to_cube_major(vol, cube):
    """[Tp, Hp, Wp, ...] -> [N, B, ...] : R^{THW} = R^{Nt Nh Nw x Bt Bh Bw} (Sec. 2.2 Permutation)."""
    Tp, Hp, Wp = vol.shape[:3]
    Bt, Bh, Bw = cube
    rest = vol.shape[3:]
    v = vol.reshape((Tp // Bt, Bt, Hp // Bh, Bh, Wp // Bw, Bw) + rest)
    perm = (0, 2, 4, 1, 3, 5) + tuple(range(6, 6 + len(rest)))
    v = v.transpose(perm)
    return v.reshape((-1, Bt * Bh * Bw) + rest)


def dense_restatement(Q, K, V, gate, mask, grid, cube, scale):
    """O = gate * Repeat(softmax(Qc Kc^T) Vc) + softmax(Q K^T scale + M_token) V in torch fp64.

    Q, K, V: torch [L, D] (may require grad); mask: bool ndarray [N, N].
    Tokens are laid out cube-major with reshape/permute; padded slots are masked keys.
    """
    L, D = Q.shape
    B = cube[0] * cube[1] * cube[2]
    idx = to_cube_major(pad_volume(np.arange(L), grid, cube, fill=-1), cube)      # [N, B]
    N = idx.shape[0]
    flat = torch.from_numpy(idx.reshape(-1))
    valid = flat >= 0
    gather = flat.clamp(min=0)
    Qp, Kp, Vp = Q[gather], K[gather], V[gather]                                   # [N*B, D]
    token_mask = torch.from_numpy(np.kron(mask, np.ones((B, B), dtype=bool))) & valid[None, :]
    s = (Qp @ Kp.T) * scale
    s = s.masked_fill(~token_mask, float("-inf"))
    row_any = token_mask.any(dim=1, keepdim=True)
    p = torch.softmax(torch.where(row_any, s, torch.zeros_like(s)), dim=1) * row_any
    O_f = p @ Vp
    lse = torch.where(row_any[:, 0], torch.logsumexp(s, dim=1), torch.full((N * B,), float("-inf"), dtype=s.dtype))
    # coarse branch: library average pooling over cubes, valid tokens only
    w = valid.to(Q.dtype).reshape(N, B, 1)
    def pool(Xp):
        return (Xp.reshape(N, B, D) * w).sum(1) / w.sum(1)
    Qc, Kc, Vc = pool(Qp), pool(Kp), pool(Vp)
    Oc_hat = F.scaled_dot_product_attention(Qc[None], Kc[None], Vc[None], scale=scale)[0]
    O_c = Oc_hat.repeat_interleave(B, dim=0)
    gp = gate[gather]
    O_p = gp[:, None] * O_c + O_f
    # back to raster order (valid slots only)
    O = torch.zeros(L, D, dtype=Q.dtype).index_put((flat[valid],), O_p[valid])
    lse_r = torch.zeros(L, dtype=Q.dtype).index_put((flat[valid],), lse[valid])
    return O, lse_r, dict(Qc=Qc, Oc_hat=Oc_hat)


def rand_problem(grid, D, seed, cube=(4, 4, 4), density=0.5):
    rng = np.random.default_rng(seed)
    L = grid[0] * grid[1] * grid[2]
    bits = [syn.f32_to_bf16_bits(rng.standard_normal((L, D), dtype=np.float32)) for _ in range(4)]
    Q, K, V, dO = (orc.bf16_bits_to_f64(b) for b in bits)
    gate = np.tanh(rng.standard_normal(L))
    geo = orc.Geometry(grid, cube)
    mask = rng.random((geo.N, geo.N)) < density
    return Q, K, V, dO, gate, geo, mask


# ---------------------------------------------------------------------------
# bf16 helpers against torch's cast
# ---------------------------------------------------------------------------
def test_bf16_rounding_matches_torch_cast():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32) * 37.0,
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38, 1e-40], dtype=np.float32)])
    ours = orc.round_f32_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))
    bits = (ours.view(np.uint32) >> 16).astype(np.uint16)
    assert np.array_equal(orc.bf16_bits_to_f64(bits), ref.astype(np.float64))
    assert np.array_equal(syn.f32_to_bf16_bits(x), bits)
    assert np.array_equal(syn.bf16_bits_to_f32(bits), ref)


# ---------------------------------------------------------------------------
# Sec. 2.1: with every block kept the fine branch is dense softmax attention
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("grid", [(4, 8, 8), (5, 6, 7)])
def test_fine_equals_dense_attention_when_all_blocks_kept(grid):
    Q, K, V, dO, gate, geo, _ = rand_problem(grid, 32, 1)
    scale = 1.0 / np.sqrt(32)
    mask = np.ones((geo.N, geo.N), dtype=bool)
    O_f, lse = orc.fine_attention(Q, K, V, mask, geo, scale)
    tq, tk, tv = (torch.from_numpy(a) for a in (Q, K, V))
    ref = F.scaled_dot_product_attention(tq[None], tk[None], tv[None])[0].numpy()   # default scale 1/sqrt(D)
    assert np.abs(O_f - ref).max() < 1e-12
    ref_lse = torch.logsumexp(tq @ tk.T / np.sqrt(32), dim=1).numpy()
    assert np.abs(lse - ref_lse).max() < 1e-12
    # textbook three-liner (Sec. 2.1)
    S = Q @ K.T / np.sqrt(32)
    P = np.exp(S - S.max(1, keepdims=True)); P /= P.sum(1, keepdims=True)
    assert np.abs(O_f - P @ V).max() < 1e-12
    assert np.allclose(P.sum(1), 1.0)


# ---------------------------------------------------------------------------
# Eq. 12 + Eq. 1-4 + Eq. 14 against the dense masked restatement (layout by reshape)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("grid,cube", [((4, 8, 8), (4, 4, 4)), ((5, 6, 9), (4, 4, 4)), ((3, 5, 8), (2, 4, 4))])
def test_forward_equals_dense_masked_restatement(grid, cube):
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, 16, 2, cube=cube)
    mask[0, :] = False                      # an empty row: O_f = 0, lse = -inf
    scale = 0.3
    r = orc.head_forward(Q, K, V, gate, mask, geo, scale)
    O, lse, aux = dense_restatement(*(torch.from_numpy(a) for a in (Q, K, V, gate)), mask, grid, cube, scale)
    assert np.abs(r["O"] - O.numpy()).max() < 1e-12
    fin = np.isfinite(lse.numpy())
    assert np.array_equal(fin, np.isfinite(r["lse"]))
    assert np.abs(r["lse"][fin] - lse.numpy()[fin]).max() < 1e-12
    assert np.abs(r["Oc_hat"] - aux["Oc_hat"].numpy()).max() < 1e-12
    assert np.abs(r["Qc"] - aux["Qc"].numpy()).max() < 1e-13
    # rows of cube 0 got nothing from the fine branch
    assert np.all(r["O_f"][geo.cube_tokens[0]] == 0) and np.all(np.isneginf(r["lse"][geo.cube_tokens[0]]))


def test_coarse_pool_matches_library_avg_pool_and_is_convex():
    grid, D = (8, 8, 12), 8
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, D, 3)
    vol = torch.from_numpy(V.reshape(grid + (D,))).permute(3, 0, 1, 2)[None]       # [1, D, T, H, W]
    ref = F.avg_pool3d(vol, kernel_size=4)[0].permute(1, 2, 3, 0).reshape(-1, D).numpy()
    Vc = orc.mean_pool_cube(V, geo)
    assert np.abs(Vc - ref).max() < 1e-14
    Qc, Kc = orc.mean_pool_cube(Q, geo), orc.mean_pool_cube(K, geo)
    Oc, lse_c = orc.coarse_attention(Qc, Kc, Vc, 0.25)
    ref = F.scaled_dot_product_attention(*(torch.from_numpy(a)[None] for a in (Qc, Kc, Vc)), scale=0.25)[0].numpy()
    assert np.abs(Oc - ref).max() < 1e-13
    assert np.all(Oc.max(0) <= Vc.max(0) + 1e-12) and np.all(Oc.min(0) >= Vc.min(0) - 1e-12)
    assert np.abs(lse_c - torch.logsumexp(torch.from_numpy(Qc @ Kc.T * 0.25), 1).numpy()).max() < 1e-12


def test_gate_zero_gives_fine_only_and_output_is_linear_in_gate():
    Q, K, V, dO, gate, geo, mask = rand_problem((4, 8, 8), 16, 4)
    r0 = orc.head_forward(Q, K, V, np.zeros_like(gate), mask, geo, 0.25)
    assert np.array_equal(r0["O"], r0["O_f"])                                       # W_g = 0 init => O = O_f
    r1 = orc.head_forward(Q, K, V, gate, mask, geo, 0.25)
    r2 = orc.head_forward(Q, K, V, 2 * gate, mask, geo, 0.25)
    assert np.abs((r2["O"] - r1["O"]) - (r1["O"] - r0["O"])).max() < 1e-12


# ---------------------------------------------------------------------------
# Eq. 5-7 router: brute force, special cases R = B and R = 1, invariants
# ---------------------------------------------------------------------------
def _pool_lib(X, grid, k, D):
    """average pooling with kernel k over an unpadded grid via torch, float32, -> [T/k0, H/k1, W/k2, D]."""
    vol = torch.from_numpy(X.astype(np.float32).reshape(grid + (D,))).permute(3, 0, 1, 2)[None]
    return F.avg_pool3d(vol, kernel_size=k)[0].permute(1, 2, 3, 0)


def test_router_pool_is_bf16_of_the_mean():
    grid, D = (4, 8, 8), 32
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, D, 5)
    Qr, valid = orc.mean_pool_router(Q, geo)
    assert valid.all()
    lib = _pool_lib(Q, grid, (2, 2, 2), D).to(torch.bfloat16).to(torch.float64).numpy()   # [2,4,4,D]
    lib = to_cube_major(lib, (2, 2, 2))                                                     # [N, G, D]
    # identical up to the (rare) last-bit effect of the fp32 summation order
    diff = Qr != lib
    assert diff.mean() < 2e-3
    assert np.abs(Qr - lib).max() <= np.abs(lib).max() * 2.0 ** -7
    # values whose fp32 sums are exact must agree bit for bit
    Xi = np.round(Q * 4) / 4
    Qi, _ = orc.mean_pool_router(Xi, geo)
    libi = to_cube_major(_pool_lib(Xi, grid, (2, 2, 2), D).to(torch.bfloat16).to(torch.float64).numpy(), (2, 2, 2))
    assert np.array_equal(Qi, libi)


def test_router_pool_fixed_summation_order():
    """A case where the float32 summation order decides the bf16 result.

    Tokens (t,h,w): x000 = 8, x001 = 2^-5, x010 = x011 = 2^-21, the rest 0 (all bf16-exact).
    Along w first: (8 + 2^-5) is exact and (2^-21 + 2^-21) = 2^-20 is one float32 ulp of 8, so the
    float32 sum is 8 + 2^-5 + 2^-20; divided by 8 it lies just above the bf16 tie 1 + 2^-8 and rounds
    up to 1 + 2^-7.  Adding the eight values left to right, or pairing along t first, loses both
    2^-21 terms (each is half an ulp, ties to even), lands exactly on the tie and rounds to 1.0.
    """
    geo = orc.Geometry((2, 2, 2), cube=(2, 2, 2), rpool=(2, 2, 2))
    X = np.zeros((8, 1))
    X[0, 0], X[1, 0], X[2, 0], X[3, 0] = 8.0, 2.0 ** -5, 2.0 ** -21, 2.0 ** -21
    Xr, valid = orc.mean_pool_router(X, geo)
    assert valid.all() and Xr.shape == (1, 1, 1)
    assert Xr[0, 0, 0] == 1.0 + 2.0 ** -7
    lr = np.float32(0)
    for v in X[:, 0]:
        lr = np.float32(lr + np.float32(v))
    assert torch.tensor(float(lr / np.float32(8))).to(torch.bfloat16).item() == 1.0


def test_router_scores_brute_force_and_row_sums():
    grid, D = (4, 8, 8), 16
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, D, 6)
    scale = 1 / np.sqrt(D)
    Qr, qv = orc.mean_pool_router(Q, geo)
    Kr, kv = orc.mean_pool_router(K, geo)
    P_r = orc.router_block_scores(Qr, Kr, qv, kv, scale)
    # brute force: library pooling + bf16 cast, full (N G)^2 softmax, library 2-D average pooling
    q = to_cube_major(_pool_lib(Q, grid, (2, 2, 2), D).to(torch.bfloat16).to(torch.float64).numpy(), (2, 2, 2))
    k = to_cube_major(_pool_lib(K, grid, (2, 2, 2), D).to(torch.bfloat16).to(torch.float64).numpy(), (2, 2, 2))
    G = 8
    p_hat = torch.softmax(torch.from_numpy(q.reshape(-1, D) @ k.reshape(-1, D).T * scale), dim=1)
    ref = F.avg_pool2d(p_hat[None, None], kernel_size=G)[0, 0].numpy()
    assert P_r.shape == (geo.N, geo.N)
    assert np.abs(P_r - ref).max() < 2e-3 * ref.max()        # pooled operands differ only by rare last-bit flips
    # exact agreement when fed the oracle's own pooled operands
    p_hat = torch.softmax(torch.from_numpy(Qr.reshape(-1, D) @ Kr.reshape(-1, D).T * scale), dim=1)
    ref = F.avg_pool2d(p_hat[None, None], kernel_size=G)[0, 0].numpy()
    assert np.abs(P_r - ref).max() < 1e-15
    assert np.allclose(P_r.sum(axis=1), 1.0 / G, rtol=0, atol=1e-14)  # rows of p_hat sum to 1


def test_router_with_R_equal_B_is_the_coarse_score_and_R_1_is_the_token_level_score():
    grid, D = (4, 4, 8), 16
    Q, K, V, dO, gate, _, _ = rand_problem(grid, D, 7)
    scale = 1 / np.sqrt(D)
    # R = B (G = 1): P_r is the softmax of pooled-cube scores, i.e. the VSA router / P_c (Sec. 2.1)
    geo = orc.Geometry(grid, (4, 4, 4), (4, 4, 4))
    Qr, qv = orc.mean_pool_router(Q, geo)
    Kr, kv = orc.mean_pool_router(K, geo)
    P_r = orc.router_block_scores(Qr, Kr, qv, kv, scale)
    P_c = torch.softmax(torch.from_numpy(Qr[:, 0] @ Kr[:, 0].T * scale), dim=1).numpy()
    assert np.abs(P_r - P_c).max() < 1e-15
    # and the pooled operands are the bf16-rounded cube means
    assert np.abs(Qr[:, 0] - orc.mean_pool_cube(Q, geo)).max() <= np.abs(Qr).max() * 2.0 ** -8
    # R = 1 (G = B): token-level softmax, then B x B mean pooling (Eq. 10-11)
    geo1 = orc.Geometry(grid, (4, 4, 4), (1, 1, 1))
    Qr, qv = orc.mean_pool_router(Q, geo1)
    Kr, kv = orc.mean_pool_router(K, geo1)
    P_r = orc.router_block_scores(Qr, Kr, qv, kv, scale)
    Qp, Kp = to_cube_major(Q.reshape(grid + (D,)), (4, 4, 4)), to_cube_major(K.reshape(grid + (D,)), (4, 4, 4))
    P = torch.softmax(torch.from_numpy(Qp.reshape(-1, D) @ Kp.reshape(-1, D).T * scale), dim=1)
    P_oracle = F.avg_pool2d(P[None, None], kernel_size=64)[0, 0].numpy()
    assert np.abs(P_r - P_oracle).max() < 1e-15


def test_router_padding_reading_rows_sum_to_one_over_G():
    geo = orc.Geometry((3, 5, 8))
    rng = np.random.default_rng(8)
    X = orc.bf16_bits_to_f64(syn.f32_to_bf16_bits(rng.standard_normal((geo.L, 8), dtype=np.float32)))
    Xr, valid = orc.mean_pool_router(X, geo)
    assert valid.sum() == 2 * 3 * 4 and not valid.all()
    # a sub-cube with a single valid token keeps that token's value
    l = geo.raster_index(2, 4, 6)
    n, g = geo.cube_of[l], geo.sub_of[l]
    assert geo.sub_count[n, g] == 2      # (t=2 only, h=4 only, w=6..7)
    P_r = orc.router_block_scores(Xr, Xr, valid, valid, 0.3)
    assert np.allclose(P_r.sum(axis=1), 1.0 / geo.G, atol=1e-14)
    assert (P_r >= 0).all()


def _masked_subcube_mean_lib(X, grid, cube, rpool):
    """Masked mean over router sub-cubes of a padded grid from library pooling only: the zero-padded value volume and a
    padded volume of ones both go through torch avg_pool3d; their ratio is sum / (number of valid tokens).
    Returns (mean [Tp/Rt, Hp/Rh, Wp/Rw, D] float32 with 0 where nothing is valid, count of the same leading shape)."""
    D = X.shape[1]
    vol = torch.from_numpy(pad_volume(X.astype(np.float32), grid, cube)).permute(3, 0, 1, 2)[None]
    ones = torch.from_numpy(pad_volume(np.ones((X.shape[0], 1), np.float32), grid, cube)).permute(3, 0, 1, 2)[None]
    s = F.avg_pool3d(vol, kernel_size=rpool)[0].permute(1, 2, 3, 0)
    c = F.avg_pool3d(ones, kernel_size=rpool)[0].permute(1, 2, 3, 0)
    mean = torch.where(c > 0, s / c.clamp(min=1e-9), torch.zeros_like(s))
    count = torch.round(c[..., 0] * (rpool[0] * rpool[1] * rpool[2])).to(torch.int64)
    return mean, count


@pytest.mark.parametrize("grid", [(3, 5, 8), (5, 6, 9), (3, 5, 9)])
def test_router_pool_on_a_padded_grid_divides_by_the_valid_count(grid):
    """Padding reading of Eq. 5: the mean of a cut sub-cube runs over its valid tokens only.  Dividing by the full
    sub-cube size R (or by any other count) fails the bitwise comparison below."""
    cube, rpool, D = (4, 4, 4), (2, 2, 2), 8
    geo = orc.Geometry(grid, cube, rpool)
    rng = np.random.default_rng(31)
    # few mantissa bits and power-of-two counts: every fp32 sum and division is exact, so the library's masked mean and
    # the oracle's must agree bit for bit whatever the order of the additions
    X = np.round(rng.standard_normal((geo.L, D)) * 4) / 4
    Xr, valid = orc.mean_pool_router(X, geo)
    mean, count = _masked_subcube_mean_lib(X, grid, cube, rpool)
    lib = to_cube_major(mean.to(torch.bfloat16).to(torch.float64).numpy(), (geo.Gt, geo.Gh, geo.Gw))      # [N, G, D]
    cnt = to_cube_major(count.numpy(), (geo.Gt, geo.Gh, geo.Gw))                                            # [N, G]
    assert set(np.unique(cnt)) <= {0, 1, 2, 4, 8} and (cnt == 0).any() and (cnt < 8).any()
    assert np.array_equal(valid, cnt > 0)
    assert np.array_equal(Xr, lib)
    assert (Xr[~valid] == 0).all()
    # literal special case: a sub-cube with one valid token holds that token's value, one with two holds their mean
    T, H, W = grid
    l = geo.raster_index(T - 1, H - 1, W - 1)
    n, g = geo.cube_of[l], geo.sub_of[l]
    members = np.nonzero((geo.cube_of == n) & (geo.sub_of == g))[0]
    assert len(members) == cnt[n, g]
    assert np.array_equal(Xr[n, g], orc.round_f32_to_bf16(X[members].mean(axis=0).astype(np.float32)).astype(np.float64))
    if grid == (3, 5, 9):
        assert len(members) == 1 and np.array_equal(Xr[n, g], X[l])
    # general values: same means up to the last bf16 bit (fp32 summation order)
    Y = orc.bf16_bits_to_f64(syn.f32_to_bf16_bits(rng.standard_normal((geo.L, D), dtype=np.float32)))
    Yr, _ = orc.mean_pool_router(Y, geo)
    meany, _ = _masked_subcube_mean_lib(Y, grid, cube, rpool)
    liby = to_cube_major(meany.to(torch.bfloat16).to(torch.float64).numpy(), (geo.Gt, geo.Gh, geo.Gw))
    assert (Yr != liby).mean() < 5e-3 and np.abs(Yr - liby).max() <= np.abs(liby).max() * 2.0 ** -7
    # R = B: the router operand is the bf16 rounding of the cube mean of Eq. 1 (which the dense restatement pins under
    # padding); cube counts such as 3*4*4 are not powers of two, so allow the last bf16 bit
    geo_b = orc.Geometry(grid, cube, cube)
    Zr, zv = orc.mean_pool_router(Y, geo_b)
    Zc = orc.round_f32_to_bf16(orc.mean_pool_cube(Y, geo_b).astype(np.float32)).astype(np.float64)
    assert zv.all() and (Zr[:, 0] != Zc).mean() < 5e-3 and np.abs(Zr[:, 0] - Zc).max() <= np.abs(Zc).max() * 2.0 ** -7


@pytest.mark.parametrize("grid", [(3, 5, 8), (3, 5, 9)])
def test_router_scores_on_a_padded_grid_match_brute_force_with_an_explicit_mask(grid):
    """Padding reading of Eq. 6-7 against brute force: every pooled query row takes a softmax over ALL pooled keys with
    -inf written on the key sub-cubes that hold no valid token; P_r[i, j] adds the G x G sub-block over valid query
    sub-cubes and divides by (valid query sub-cubes of cube i) * G.  Not masking the empty keys, masking by cube instead
    of by sub-cube, or dividing by G * G all fail."""
    cube, rpool, D = (4, 4, 4), (2, 2, 2), 16
    geo = orc.Geometry(grid, cube, rpool)
    rng = np.random.default_rng(32)
    Q = np.round(rng.standard_normal((geo.L, D)) * 4) / 4
    K = np.round(rng.standard_normal((geo.L, D)) * 4) / 4
    scale = 0.35
    Qr, qv = orc.mean_pool_router(Q, geo)
    Kr, kv = orc.mean_pool_router(K, geo)
    P_r = orc.router_block_scores(Qr, Kr, qv, kv, scale)
    # independent operands and validity, laid out [N, G, .] by reshape
    G3 = (geo.Gt, geo.Gh, geo.Gw)
    qm, qc = _masked_subcube_mean_lib(Q, grid, cube, rpool)
    km, kc = _masked_subcube_mean_lib(K, grid, cube, rpool)
    q = torch.from_numpy(to_cube_major(qm.to(torch.bfloat16).to(torch.float64).numpy(), G3)).reshape(-1, D)
    k = torch.from_numpy(to_cube_major(km.to(torch.bfloat16).to(torch.float64).numpy(), G3)).reshape(-1, D)
    q_ok = torch.from_numpy(to_cube_major(qc.numpy(), G3) > 0)                   # [N, G]
    k_ok = torch.from_numpy(to_cube_major(kc.numpy(), G3) > 0).reshape(-1)       # [N G]
    assert (~k_ok).any() and (~q_ok).any()
    s = (q @ k.T) * scale
    s = s.masked_fill(~k_ok[None, :], float("-inf"))
    p_hat = torch.softmax(s, dim=1) * q_ok.reshape(-1, 1)
    N, G = geo.N, geo.G
    ref = torch.zeros(N, N, dtype=torch.float64)
    for i in range(N):
        for j in range(N):
            ref[i, j] = p_hat[i * G:(i + 1) * G, j * G:(j + 1) * G].sum() / (q_ok[i].sum() * G)
    assert np.abs(P_r - ref.numpy()).max() < 1e-15
    assert np.allclose(P_r.sum(axis=1), 1.0 / G, atol=1e-14)
    # a cube pair whose key cube has fewer valid sub-cubes holds less mass than the same scores would give unmasked
    empty_keys = np.nonzero(~k_ok.numpy())[0]
    p_unmasked = torch.softmax((q @ k.T) * scale, dim=1)
    assert (p_unmasked[:, empty_keys] > 0).all() and (p_hat[:, empty_keys] == 0).all()


def test_router_map_invariant_to_permuting_tokens_inside_a_sub_cube():
    grid, D = (4, 8, 8), 16
    rng = np.random.default_rng(9)
    # few mantissa bits: every fp32 partial sum is exact, so the order of the sum cannot matter
    Q = np.round(rng.standard_normal((256, D)) * 8) / 8
    K = np.round(rng.standard_normal((256, D)) * 8) / 8
    geo = orc.Geometry(grid)
    perm = np.arange(256)
    for n, g in itertools.product(range(geo.N), range(geo.G)):
        idx = np.nonzero((geo.cube_of == n) & (geo.sub_of == g))[0]
        perm[idx] = rng.permutation(idx)
    m1 = orc.route(Q[None, None], K[None, None], geo, 0.25, orc.PER_SEQUENCE, topk=2)
    m2 = orc.route(Q[perm][None, None], K[perm][None, None], geo, 0.25, orc.PER_SEQUENCE, topk=2)
    assert np.array_equal(m1, m2)


# ---------------------------------------------------------------------------
# Eq. 8-9 selection: brute-force sort, invariants, ties
# ---------------------------------------------------------------------------
def _brute_topk(flat_scores, keep):
    order = sorted(range(len(flat_scores)), key=lambda i: (-float(np.float32(flat_scores[i])), i))
    return set(order[:keep])


@pytest.mark.parametrize("N,K", [(4, 2), (13, 3), (32, 8), (7, 9)])
def test_selection_matches_brute_force_sort(N, K):
    rng = np.random.default_rng(10 + N)
    P = rng.random((N, N)) ** 4
    P[rng.random((N, N)) < 0.2] = 0.125                     # ties
    Ke = min(K, N)
    m = orc.select_blocks(P, orc.PER_SEQUENCE, topk=K)
    assert m.sum() == N * Ke                                 # exactly N K blocks per sequence (Eq. 9)
    assert set(np.nonzero(m.reshape(-1))[0]) == _brute_topk(P.reshape(-1), N * Ke)
    if Ke < N:
        assert np.float32(P[m].min()) >= np.float32(P[~m].max())
    mq = orc.select_blocks(P, orc.PER_QUERY, topk=K)
    assert (mq.sum(axis=1) == Ke).all()
    for i in range(N):
        assert set(np.nonzero(mq[i])[0]) == _brute_topk(P[i], Ke)
    budgets = rng.integers(0, N + 3, size=N)
    mb = orc.select_blocks(P, orc.PER_QUERY_BUDGET, budgets=budgets)
    assert (mb.sum(axis=1) == np.minimum(budgets, N)).all()
    for i in range(N):
        assert set(np.nonzero(mb[i])[0]) == _brute_topk(P[i], min(int(budgets[i]), N))


def test_selection_per_sequence_gives_variable_rows_and_handles_ties():
    P = np.array([[0.9, 0.8, 0.7], [0.1, 0.1, 0.1], [0.6, 0.1, 0.1]])
    m = orc.select_blocks(P, orc.PER_SEQUENCE, topk=1)       # keep 3 of 9
    assert np.array_equal(m, np.array([[1, 1, 1], [0, 0, 0], [0, 0, 0]], dtype=bool))
    m = orc.select_blocks(P, orc.PER_SEQUENCE, topk=2)       # keep 6: 0.9 .8 .7 .6 then two 0.1 at lowest flat index
    assert np.array_equal(m, np.array([[1, 1, 1], [1, 1, 0], [1, 0, 0]], dtype=bool))
    mq = orc.select_blocks(P, orc.PER_QUERY, topk=1)
    assert np.array_equal(mq, np.array([[1, 0, 0], [1, 0, 0], [1, 0, 0]], dtype=bool))


def test_csr_csc_describe_the_same_set():
    rng = np.random.default_rng(11)
    mask = rng.random((17, 17)) < 0.3
    mask[5] = False
    rp, ci = orc.mask_to_csr(mask)
    cp, ri = orc.mask_to_csc(mask)
    a = {(i, int(j)) for i in range(17) for j in ci[rp[i]:rp[i + 1]]}
    b = {(int(i), j) for j in range(17) for i in ri[cp[j]:cp[j + 1]]}
    assert a == b == {(i, j) for i in range(17) for j in range(17) if mask[i, j]}
    assert rp[-1] == cp[-1] == mask.sum()
    for i in range(17):
        assert np.all(np.diff(ci[rp[i]:rp[i + 1]]) > 0) and np.all(np.diff(ri[cp[i]:cp[i + 1]]) > 0)


# ---------------------------------------------------------------------------
# backward: autograd of the dense restatement, finite differences, GQA sum
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("grid,cube", [((4, 8, 8), (4, 4, 4)), ((5, 6, 9), (4, 4, 4))])
def test_backward_matches_autograd_of_dense_restatement(grid, cube):
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, 16, 12, cube=cube)
    mask[1, :] = False
    scale = 0.2
    g = orc.head_backward(Q, K, V, gate, mask, geo, scale, dO)
    tq, tk, tv, tg = (torch.from_numpy(a).requires_grad_(True) for a in (Q, K, V, gate))
    O, _, _ = dense_restatement(tq, tk, tv, tg, mask, grid, cube, scale)
    (O * torch.from_numpy(dO)).sum().backward()
    for name, t in (("dQ", tq), ("dK", tk), ("dV", tv), ("dGate", tg)):
        err = np.abs(g[name] - t.grad.numpy()).max()
        assert err < 1e-11, (name, err)


@pytest.mark.parametrize("kv_cubes", [(0, 5), (3, 7, 11)])
def test_fine_backward_restricted_to_kv_cubes_matches_the_full_backward_and_autograd(kv_cubes):
    """fine_backward_kv_cubes must return exactly the rows of the full fine-branch dK, dV that belong to the requested KV
    cubes: the softmax statistics (lse, delta) come from ALL kept blocks of a query row, not from the requested ones."""
    grid, cube = (5, 6, 9), (4, 4, 4)
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, 16, 21, cube=cube)
    mask[2, :] = False                                  # an empty query row
    mask[:, kv_cubes[0]] |= np.arange(geo.N) % 2 == 0   # the first requested cube is kept by many rows
    assert geo.N == 12 and (geo.cube_count < 64).any()
    scale = 0.2
    dK, dV = orc.fine_backward_kv_cubes(Q, K, V, mask, geo, scale, dO, kv_cubes)
    tok = np.concatenate([geo.cube_tokens[j] for j in kv_cubes])
    rest = np.setdiff1d(np.arange(geo.L), tok)
    assert (dK[rest] == 0).all() and (dV[rest] == 0).all()
    # (1) the full oracle backward of the fine branch
    O_f, lse = orc.fine_attention(Q, K, V, mask, geo, scale)
    _, fk, fv = orc.fine_backward(Q, K, V, mask, geo, scale, dO, lse, O_f)
    assert np.abs(dK[tok] - fk[tok]).max() < 1e-12 and np.abs(dV[tok] - fv[tok]).max() < 1e-12
    # (2) autograd of the dense masked restatement with the gate at zero (O = O_f)
    tq, tk, tv = (torch.from_numpy(a).requires_grad_(True) for a in (Q, K, V))
    O, _, _ = dense_restatement(tq, tk, tv, torch.zeros(geo.L, dtype=torch.float64), mask, grid, cube, scale)
    (O * torch.from_numpy(dO)).sum().backward()
    assert np.abs(dK[tok] - tk.grad.numpy()[tok]).max() < 1e-11
    assert np.abs(dV[tok] - tv.grad.numpy()[tok]).max() < 1e-11
    assert np.abs(tk.grad.numpy()[tok]).max() > 1e-3


def test_backward_matches_central_finite_differences_on_config0():
    wl = syn.CONFIGS[0]
    data = syn.make_inputs(wl, threads=1)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    Q, K, V, dO = (orc.bf16_bits_to_f64(data[k][0, 0]) for k in ("q", "k", "v", "do"))
    gate = data["gate"][0, 0].astype(np.float64)
    scale = 1 / np.sqrt(wl.head_dim)
    mask = orc.route(Q[None, None], K[None, None], geo, scale, wl.select_mode, wl.topk)[0, 0]
    assert (mask.sum(axis=1) == 2).all()
    g = orc.head_backward(Q, K, V, gate, mask, geo, scale, dO)
    f = lambda q, k, v, gt: (orc.head_forward(q, k, v, gt, mask, geo, scale)["O"] * dO).sum()
    rng = np.random.default_rng(13)
    eps = 1e-5
    for which, name in enumerate(("dQ", "dK", "dV", "dGate")):
        args = [Q, K, V, gate]
        direction = rng.standard_normal(args[which].shape)
        plus, minus = list(args), list(args)
        plus[which] = args[which] + eps * direction
        minus[which] = args[which] - eps * direction
        fd = (f(*plus) - f(*minus)) / (2 * eps)
        an = (g[name] * direction).sum()
        assert abs(fd - an) < 1e-6 * max(1.0, abs(an)), (name, fd, an)


def test_gqa_backward_sums_group_and_heads_permute():
    grid, D = (4, 8, 8), 16
    rng = np.random.default_rng(14)
    geo = orc.Geometry(grid)
    Q = rng.standard_normal((1, 4, 256, D)); K = rng.standard_normal((1, 2, 256, D)); V = rng.standard_normal((1, 2, 256, D))
    dO = rng.standard_normal((1, 4, 256, D)); gate = np.tanh(rng.standard_normal((1, 4, 256)))
    masks = orc.route(Q, K, geo, 0.25, orc.PER_QUERY, topk=2)
    O, lse = orc.forward(Q, K, V, gate, masks, geo, 0.25)
    dQ, dK, dV, dG = orc.backward(Q, K, V, gate, masks, geo, 0.25, dO)
    # the same problem written as MHA with the KV heads repeated
    Kx, Vx = np.repeat(K, 2, axis=1), np.repeat(V, 2, axis=1)
    mx = orc.route(Q, Kx, geo, 0.25, orc.PER_QUERY, topk=2)
    assert np.array_equal(masks, mx)
    Ox, _ = orc.forward(Q, Kx, Vx, gate, mx, geo, 0.25)
    dQx, dKx, dVx, dGx = orc.backward(Q, Kx, Vx, gate, mx, geo, 0.25, dO)
    assert np.array_equal(O, Ox) and np.array_equal(dQ, dQx)
    assert np.abs(dK - dKx.reshape(1, 2, 2, 256, D).sum(2)).max() < 1e-12
    assert np.abs(dV - dVx.reshape(1, 2, 2, 256, D).sum(2)).max() < 1e-12
    # permuting heads permutes masks, outputs and gradients
    p = np.array([2, 0, 3, 1])
    mp = orc.route(Q[:, p], Kx[:, p], geo, 0.25, orc.PER_QUERY, topk=2)
    assert np.array_equal(mp, mx[:, p])
    Op, _ = orc.forward(Q[:, p], Kx[:, p], Vx[:, p], gate[:, p], mp, geo, 0.25)
    assert np.array_equal(Op, Ox[:, p])


def test_all_blocks_kept_removes_any_dependence_on_the_router():
    grid, D = (4, 8, 8), 16
    Q, K, V, dO, gate, geo, _ = rand_problem(grid, D, 15)
    m = orc.route(Q[None, None], K[None, None], geo, 0.25, orc.PER_SEQUENCE, topk=geo.N + 5)
    assert m.all()                                           # K > N is clamped to N
    m = orc.route(Q[None, None], K[None, None], geo, 0.25, orc.PER_QUERY, topk=geo.N)
    assert m.all()


# ---------------------------------------------------------------------------
# Appendix "Sparsity Computation" against the values printed in Table 1
# ---------------------------------------------------------------------------
def test_sparsity_formula_reproduces_table1():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_sparsity.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for k, tokens, printed in rows:
        s = orc.sparsity(int(k), 128, 8, int(tokens))
        assert round(s, 2) == float(printed), (k, tokens, s)
    # the fine-branch cost fraction N K B^2 / L^2 equals K B / L on an unpadded grid (Eq. 15)
    geo = orc.Geometry((8, 16, 16))
    mask = orc.select_blocks(np.random.default_rng(0).random((geo.N, geo.N)), orc.PER_SEQUENCE, topk=8)
    pairs = sum(len(geo.cube_tokens[i]) * len(geo.cube_tokens[j]) for i, j in zip(*np.nonzero(mask)))
    assert pairs / geo.L ** 2 == orc.fine_cost_fraction(8, geo.B, geo.L)


# ---------------------------------------------------------------------------
# input generators: deterministic, right shapes, locality really is there
# ---------------------------------------------------------------------------
def test_input_generators_are_seeded_and_structured():
    wl = syn.CONFIGS[1]
    a = syn.head_tensor(wl, "q", 0, 3)
    b = syn.head_tensor(wl, "q", 0, 3)
    assert a.dtype == np.uint16 and a.shape == (2048, 128) and np.array_equal(a, b)
    assert not np.array_equal(a, syn.head_tensor(wl, "k", 0, 3))
    x = syn.bf16_bits_to_f32(a).reshape(8, 16, 16, 128)
    # neighbouring tokens correlate (smooth field of unit variance plus 0.3 noise)
    c = np.corrcoef(x[:, :, :-1].reshape(-1), x[:, :, 1:].reshape(-1))[0, 1]
    assert 0.7 < c < 0.95
    assert abs(x.std() - np.sqrt(1 + 0.09)) < 0.05
    g = syn.head_gate(wl, 0, 0)
    assert g.shape == (2048,) and np.abs(g).max() < 1
    assert np.all(syn.head_gate(syn.CONFIGS[0], 0, 0) == 0.5)
    bud = syn.head_budgets(syn.CONFIGS[4], 0, 0)
    assert bud.shape == (1440,) and bud.min() >= 16 and bud.max() <= 256


def test_gate_projection_matches_autograd_and_its_special_cases():
    """Eq. 13: gate = tanh(X W_g).  Pinned against torch's tanh / matmul / autograd (library routines), the
    zero-initialised projection of the paper's recipe (W_g = 0 => gate = 0 => O = O_f), saturation and oddness."""
    rng = np.random.default_rng(17)
    L, C, H = 37, 24, 5
    X = rng.standard_normal((L, C))
    Wg = rng.standard_normal((C, H)) * 0.3
    dgate = rng.standard_normal((H, L))
    gate = orc.gate_forward(X, Wg)
    assert gate.shape == (H, L)
    xt = torch.tensor(X, requires_grad=True)
    wt = torch.tensor(Wg, requires_grad=True)
    gt = torch.tanh(xt @ wt).T
    np.testing.assert_allclose(gate, gt.detach().numpy(), rtol=1e-13, atol=1e-15)
    gt.backward(torch.tensor(dgate))
    dX, dW = orc.gate_backward(X, Wg, dgate)
    np.testing.assert_allclose(dX, xt.grad.numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(dW, wt.grad.numpy(), rtol=1e-12, atol=1e-14)
    # W_g = 0: gate = 0 everywhere, dX = 0, dW_g = X^T dgate^T
    z = np.zeros_like(Wg)
    assert not orc.gate_forward(X, z).any()
    dX0, dW0 = orc.gate_backward(X, z, dgate)
    assert not dX0.any()
    np.testing.assert_allclose(dW0, X.T @ dgate.T, rtol=1e-13)
    # odd in X, bounded by 1, saturating
    np.testing.assert_allclose(orc.gate_forward(-X, Wg), -gate, rtol=1e-13)
    assert np.abs(orc.gate_forward(50.0 * X, Wg)).max() <= 1.0
    # central finite difference of sum(gate * dgate) w.r.t. one weight and one hidden state
    f = lambda Xv, Wv: float((orc.gate_forward(Xv, Wv) * dgate).sum())
    h = 1e-6
    Wp, Wm = Wg.copy(), Wg.copy(); Wp[3, 2] += h; Wm[3, 2] -= h
    assert abs((f(X, Wp) - f(X, Wm)) / (2 * h) - dW[3, 2]) < 1e-6
    Xp, Xm = X.copy(), X.copy(); Xp[11, 7] += h; Xm[11, 7] -= h
    assert abs((f(Xp, Wg) - f(Xm, Wg)) / (2 * h) - dX[11, 7]) < 1e-6


def test_group_shared_routing_is_the_topk_of_the_summed_head_scores():
    """Sec. 4 "Group Head": the query heads of a KV group share one map.  Pins: identical masks inside a group, equal to the
    brute-force TopK of the summed per-head scores; one head per group changes nothing; other groups are untouched."""
    rng = np.random.default_rng(23)
    geo = orc.Geometry((4, 8, 8), (4, 4, 4), (2, 2, 2))
    L, D, Hq, Hkv = geo.L, 16, 4, 2
    Q = rng.standard_normal((1, Hq, L, D)).astype(np.float32).astype(np.float64)
    K = rng.standard_normal((1, Hkv, L, D)).astype(np.float32).astype(np.float64)
    own, P = orc.route(Q, K, geo, 0.25, orc.PER_SEQUENCE, 2, return_scores=True)
    shared, Pg = orc.route(Q, K, geo, 0.25, orc.PER_SEQUENCE, 2, return_scores=True, share_group=True)
    for hk in range(Hkv):
        a, b = 2 * hk, 2 * hk + 1
        assert np.array_equal(shared[0, a], shared[0, b])
        summed = (P[0, a] + P[0, b]).astype(np.float32)
        np.testing.assert_allclose(Pg[0, a], P[0, a] + P[0, b], rtol=1e-14)
        keep = _brute_topk(summed.reshape(-1), geo.N * 2)
        assert set(np.nonzero(shared[0, a].reshape(-1))[0].tolist()) == keep
        assert shared[0, a].sum() == geo.N * 2
    assert not np.array_equal(own[0, 0], own[0, 1])                      # the heads would have chosen differently
    # a group of one head is the ordinary routing
    same = orc.route(Q[:, :2], K, geo, 0.25, orc.PER_QUERY, 3, share_group=True)
    assert np.array_equal(same, orc.route(Q[:, :2], K, geo, 0.25, orc.PER_QUERY, 3))


@pytest.mark.parametrize("grid,cube", [((4, 8, 8), (4, 4, 4)), ((5, 6, 9), (4, 4, 4)), ((3, 5, 13), (2, 4, 8))])
def test_cube_major_permutation_matches_a_reshape_of_the_padded_volume(grid, cube):
    """Sec. 2.2 "Permutation": (T, H, W) -> (N_t N_h N_w) x (B_t B_h B_w).  Pinned against a reshape / transpose of the
    zero-padded volume (numpy routines), the cube token lists, and its own inverse."""
    geo = orc.Geometry(grid, cube, (1, 1, 1))
    rng = np.random.default_rng(3)
    X = rng.standard_normal((geo.L, 6))
    Y = orc.to_cube_major(X, geo, fill=0.0)
    vol = pad_volume(X, grid, cube)
    np.testing.assert_array_equal(Y, to_cube_major(vol, cube).reshape(geo.N * geo.B, 6))
    for n in (0, geo.N - 1):
        rows = Y[n * geo.B:(n + 1) * geo.B]
        np.testing.assert_array_equal(rows[np.abs(rows).sum(axis=1) > 0], X[geo.cube_tokens[n]])
    np.testing.assert_array_equal(orc.from_cube_major(Y, geo), X)


# ---------------------------------------------------------------------------
# Sec. 2.2, the sentence after Eq. 12: text tokens share the attention space (MMDiT)
# ---------------------------------------------------------------------------
def rand_text(Lt, D, seed):
    rng = np.random.default_rng(seed)
    return tuple(orc.bf16_bits_to_f64(syn.f32_to_bf16_bits(rng.standard_normal((Lt, D), dtype=np.float32))) for _ in range(4))


@pytest.mark.parametrize("grid,Lt", [((4, 8, 8), 37), ((5, 6, 9), 70)])
def test_text_tokens_with_all_blocks_kept_are_dense_attention_over_the_concatenation(grid, Lt):
    D, scale = 16, 0.3
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, D, 41)
    Qt, Kt, Vt, dOt = rand_text(Lt, D, 42)
    mask[:] = True
    O_f, lse, O_t, lse_t = orc.joint_fine_attention(Q, K, V, Qt, Kt, Vt, mask, geo, scale)
    qc, kc, vc = (torch.from_numpy(np.concatenate(p)) for p in ((Q, Qt), (K, Kt), (V, Vt)))
    ref = F.scaled_dot_product_attention(qc[None], kc[None], vc[None], scale=scale)[0].numpy()
    ref_lse = torch.logsumexp(qc @ kc.T * scale, dim=1).numpy()
    assert np.abs(np.concatenate((O_f, O_t)) - ref).max() < 1e-12
    assert np.abs(np.concatenate((lse, lse_t)) - ref_lse).max() < 1e-12
    # without text tokens the joint functions are the plain ones
    e = np.zeros((0, D))
    O0, l0, Ot0, lt0 = orc.joint_fine_attention(Q, K, V, e, e, e, mask, geo, scale)
    O1, l1 = orc.fine_attention(Q, K, V, mask, geo, scale)
    assert np.array_equal(O0, O1) and np.array_equal(l0, l1) and Ot0.shape == (0, D)


def test_text_tokens_merge_with_the_video_part_by_log_sum_exp():
    """A video query's joint softmax over (kept video blocks, text) is the log-sum-exp merge of the block-sparse result
    (pinned above) with a library softmax attention over the text keys alone; an empty video row leaves the text part."""
    grid, D, Lt, scale = (5, 6, 9), 16, 45, 0.25
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, D, 43, density=0.3)
    mask[3, :] = False
    Qt, Kt, Vt, dOt = rand_text(Lt, D, 44)
    O_f, lse, O_t, lse_t = orc.joint_fine_attention(Q, K, V, Qt, Kt, Vt, mask, geo, scale)
    O_vv, lse_vv = orc.fine_attention(Q, K, V, mask, geo, scale)
    st = torch.from_numpy(Q @ Kt.T * scale)
    lse_vt = torch.logsumexp(st, dim=1).numpy()
    O_vt = (torch.softmax(st, dim=1) @ torch.from_numpy(Vt)).numpy()
    tot = np.logaddexp(lse_vv, lse_vt)
    merged = np.exp(lse_vv - tot)[:, None] * O_vv + np.exp(lse_vt - tot)[:, None] * O_vt
    assert np.abs(lse - tot).max() < 1e-12 and np.abs(O_f - merged).max() < 1e-12
    rows3 = geo.cube_tokens[3]
    assert np.abs(O_f[rows3] - O_vt[rows3]).max() < 1e-12
    # text queries: dense over everything (library)
    kc, vc = torch.from_numpy(np.concatenate((K, Kt))), torch.from_numpy(np.concatenate((V, Vt)))
    ref_t = F.scaled_dot_product_attention(torch.from_numpy(Qt)[None], kc[None], vc[None], scale=scale)[0].numpy()
    assert np.abs(O_t - ref_t).max() < 1e-12
    # restricting the rows computes the same values on those rows
    Of2, l2, Ot2, lt2 = orc.joint_fine_attention(Q, K, V, Qt, Kt, Vt, mask, geo, scale, rows=(1, 3), text_rows=(0, 44))
    sel = np.concatenate([geo.cube_tokens[1], geo.cube_tokens[3]])
    assert np.array_equal(Of2[sel], O_f[sel]) and np.array_equal(Ot2[[0, 44]], O_t[[0, 44]]) and (Ot2[1:44] == 0).all()


def test_text_tokens_backward_matches_autograd_of_a_dense_masked_restatement():
    grid, cube, D, Lt, scale = (5, 6, 9), (4, 4, 4), 16, 21, 0.2
    Q, K, V, dO, gate, geo, mask = rand_problem(grid, D, 45, cube=cube, density=0.4)
    mask[2, :] = False
    Qt, Kt, Vt, dOt = rand_text(Lt, D, 46)
    g = orc.joint_head_backward(Q, K, V, Qt, Kt, Vt, gate, mask, geo, scale, dO, dOt)
    # restatement: one [L + Lt] x [L + Lt] score matrix in raster order, boolean mask built from the cube index of every
    # token by reshape (never the oracle's index formula), library softmax; coarse branch from dense_restatement
    L = geo.L
    cube_of = to_cube_major(pad_volume(np.arange(L), grid, cube, fill=-1), cube)          # [N, B] raster ids
    tok_cube = np.zeros(L, dtype=np.int64)
    for n in range(cube_of.shape[0]):
        ids = cube_of[n][cube_of[n] >= 0]
        tok_cube[ids] = n
    allow = np.ones((L + Lt, L + Lt), dtype=bool)
    allow[:L, :L] = mask[tok_cube][:, tok_cube]
    t = {n: torch.from_numpy(a).requires_grad_(True) for n, a in
         (("q", Q), ("k", K), ("v", V), ("qt", Qt), ("kt", Kt), ("vt", Vt), ("gate", gate))}
    s = torch.cat((t["q"], t["qt"])) @ torch.cat((t["k"], t["kt"])).T * scale
    s = s.masked_fill(~torch.from_numpy(allow), float("-inf"))
    O_all = torch.softmax(s, dim=1) @ torch.cat((t["v"], t["vt"]))
    _, _, coarse = dense_restatement(t["q"], t["k"], t["v"], t["gate"], mask, grid, cube, scale)
    B = cube[0] * cube[1] * cube[2]
    flat = torch.from_numpy(cube_of.reshape(-1))
    O_c = torch.zeros(L, D, dtype=torch.float64).index_put((flat[flat >= 0],), coarse["Oc_hat"].repeat_interleave(B, dim=0)[flat >= 0])
    O = t["gate"][:, None] * O_c + O_all[:L]
    ((O * torch.from_numpy(dO)).sum() + (O_all[L:] * torch.from_numpy(dOt)).sum()).backward()
    for name, key in (("dQ", "q"), ("dK", "k"), ("dV", "v"), ("dQt", "qt"), ("dKt", "kt"), ("dVt", "vt"), ("dGate", "gate")):
        err = np.abs(g[name] - t[key].grad.numpy()).max()
        assert err < 1e-11, (name, err)
    fwd = orc.joint_head_forward(Q, K, V, Qt, Kt, Vt, gate, mask, geo, scale)
    assert np.abs(fwd["O"] - O.detach().numpy()).max() < 1e-12 and np.abs(fwd["O_t"] - O_all[L:].detach().numpy()).max() < 1e-12
