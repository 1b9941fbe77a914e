"""GPU check of the cube-major copy (Sec. 2.2 "Permutation") against the oracle: byte-exact both ways."""
import numpy as np
import pytest
import torch

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("grid,cube,D,heads", [((5, 6, 9), (4, 4, 4), 128, 3), ((7, 10, 28), (4, 4, 8), 64, 2),
                                               ((8, 16, 16), (4, 4, 4), 64, 1)])
def test_cube_major_copy_and_back(grid, cube, D, heads):
    geo = orc.Geometry(grid, cube, (2, 2, 2))
    rng = np.random.default_rng(sum(grid))
    bits = syn.f32_to_bf16_bits(rng.standard_normal((2, heads, geo.L, D)).astype(np.float32))
    p = vb.make_params(batch=2, heads_q=heads, heads_kv=heads, head_dim=D, grid=grid, cube=cube, topk=1)
    s = vb.vsa2_query_sizes(p)
    assert (s.n_cubes, s.block_tokens) == (geo.N, geo.B)
    x = torch.from_numpy(bits.view(np.int16)).cuda()
    y = torch.full((2, heads, geo.N * geo.B, D), -1, dtype=torch.int16, device="cuda")
    vb.vsa2_permute_cube_major(p, heads, x, y)
    want = np.stack([[orc.to_cube_major(bits[b, h], geo, fill=0) for h in range(heads)] for b in range(2)])
    assert np.array_equal(y.cpu().numpy().view(np.uint16), want)
    back = torch.full_like(x, -1)
    vb.vsa2_permute_cube_major(p, heads, y, back, inverse=True)
    assert torch.equal(back, x)
