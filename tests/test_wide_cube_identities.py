"""The identities that let a 128-token cube (4 x 4 x 8) run as two 64-token half-cubes, checked on the oracle alone:
cube-level router scores, pooled means and block masks follow from the half-cube quantities (Eq. 1, Eq. 5-7, Eq. 12)."""
import numpy as np
import pytest

from oracle import vsa2_oracle as orc


@pytest.mark.parametrize("grid", [(8, 8, 16), (7, 10, 29), (5, 6, 13)])
def test_cube_scores_are_a_weighted_fold_of_half_cube_scores(grid):
    wide = orc.Geometry(grid, (4, 4, 8), (2, 2, 2))
    half = orc.Geometry(grid, (4, 4, 4), (2, 2, 2))
    assert half.N == 2 * wide.N and wide.G == 2 * half.G
    rng = np.random.default_rng(11)
    L, D = wide.L, 16
    Q = rng.standard_normal((L, D)).astype(np.float32).astype(np.float64)
    K = rng.standard_normal((L, D)).astype(np.float32).astype(np.float64)
    Qw, vqw = orc.mean_pool_router(Q, wide)
    Kw, vkw = orc.mean_pool_router(K, wide)
    Qh, vqh = orc.mean_pool_router(Q, half)
    Kh, vkh = orc.mean_pool_router(K, half)
    Pw = orc.router_block_scores(Qw, Kw, vqw, vkw, 0.25)
    Ph = orc.router_block_scores(Qh, Kh, vqh, vkh, 0.25)
    vq = vqh.sum(axis=1).astype(np.float64)                       # valid query sub-cubes per half-cube
    w = vq.reshape(-1, 2) / (2.0 * vq.reshape(-1, 2).sum(axis=1, keepdims=True))
    fold = (Ph.reshape(wide.N, 2, wide.N, 2).sum(axis=3) * w[:, :, None]).sum(axis=1)
    np.testing.assert_allclose(fold, Pw, rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("grid", [(8, 8, 16), (7, 10, 29)])
def test_cube_means_and_mask_expansion(grid):
    wide = orc.Geometry(grid, (4, 4, 8), (2, 2, 2))
    half = orc.Geometry(grid, (4, 4, 4), (2, 2, 2))
    rng = np.random.default_rng(12)
    L, D = wide.L, 8
    X = rng.standard_normal((L, D))
    Xw, Xh = orc.mean_pool_cube(X, wide), orc.mean_pool_cube(X, half)
    c = np.asarray(half.cube_count, dtype=np.float64).reshape(-1, 2)
    fold = (Xh.reshape(wide.N, 2, D) * c[:, :, None]).sum(axis=1) / c.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(fold, Xw, rtol=1e-12, atol=1e-15)
    # a cube is its two half-cubes, in order
    for n in range(wide.N):
        both = np.concatenate([half.cube_tokens[2 * n], half.cube_tokens[2 * n + 1]])
        assert sorted(both) == sorted(wide.cube_tokens[n])
    # fine attention under a cube mask equals fine attention under the expanded half-cube mask
    Q, K, V = (rng.standard_normal((L, D)) for _ in range(3))
    mask = rng.random((wide.N, wide.N)) < 0.4
    mask[np.arange(wide.N), np.arange(wide.N)] = True
    Ow, lw = orc.fine_attention(Q, K, V, mask, wide, 0.3)
    Oh, lh = orc.fine_attention(Q, K, V, np.kron(mask, np.ones((2, 2), dtype=bool)), half, 0.3)
    np.testing.assert_allclose(Oh, Ow, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lh, lw, rtol=1e-12, atol=1e-14)
