"""GPU parity on seeded random small geometries: grids with ragged edges in every dimension, odd list lengths,
both head dimensions, the three selection modes, GQA groupings and both output dtypes, each run route -> forward ->
backward through the C ABI and compared with the oracle element by element."""
import numpy as np
import pytest

from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn
from test_gpu_parity import full_parity

pytestmark = pytest.mark.gpu


def random_workload(case: int, wide: bool = False) -> tuple:
    rng = np.random.default_rng((3000 if wide else 1000) + case)
    grid = (int(rng.integers(3, 10)), int(rng.integers(4, 15)), int(rng.integers(4, 19)))
    cube = (4, 4, 4)
    if wide:
        # cubes of 128 tokens; w up to 33 so that every remainder mod 8 occurs (1..4: the last cube's second half is empty)
        cube = (4, 4, 8)
        grid = (grid[0], grid[1], int(rng.integers(5, 34)))
    heads_kv = int(rng.integers(1, 4))
    rep = int(rng.choice([1, 1, 2, 4]))
    head_dim = int(rng.choice([64, 128]))
    mode = int(rng.choice([syn.PER_SEQUENCE, syn.PER_QUERY, syn.PER_QUERY_BUDGET]))
    n_cubes = int(np.prod([-(-g // c) for g, c in zip(grid, cube)]))
    topk = 0 if mode == syn.PER_QUERY_BUDGET else int(rng.integers(1, max(2, min(n_cubes, 12))))
    batch = int(rng.choice([1, 1, 2]))
    wl = syn.Workload(f"fuzz_{case}", batch, heads_kv * rep, heads_kv, head_dim, grid, cube=cube, select_mode=mode,
                      topk=topk, seed=500 + case)
    out_dtype = vb.F32 if rng.integers(0, 2) else vb.BF16
    return wl, out_dtype


def run_case(wl, out_dtype, flags=0):
    data = syn.make_inputs(wl)
    nnz_cap = 0
    if wl.select_mode == syn.PER_QUERY_BUDGET:
        nnz_cap = int(np.minimum(data["budgets"], wl.n_cubes).sum(axis=-1).max())
    full_parity(wl, data, out_dtype=out_dtype, nnz_cap=nnz_cap, flags=flags)


@pytest.mark.parametrize("case", range(24))
def test_random_geometry_full_parity(case):
    run_case(*random_workload(case))


@pytest.mark.parametrize("case", range(16))
def test_random_geometry_cubes_of_128_tokens(case):
    run_case(*random_workload(case, wide=True))


@pytest.mark.parametrize("case,wide", [(186, False), (102, True), (187, True), (189, True)])
def test_geometries_with_sharply_peaked_rows(case, wide):
    """Four geometries of a wider sweep (cases 100-219) whose rows keep one to seven blocks: the softmax is sharply peaked,
    gradients reach |g| = 5..30, and with every P and dS rounded once to bf16 (and the output normalised by the unrounded
    row sum) the worst element of dV or dQ missed 2e-2 (2.2e-2 .. 2.8e-2).  The three GQA cases pass with the defaults (the
    forward normalises by the sum of the rounded weights; the dQ pass and the GQA dK/dV pass carry P and dS as bf16 pairs);
    the single-head case needs the pairs in the dK/dV pass as well, which is what VSA2_FLAG_PRECISE_BWD is for."""
    wl, out_dtype = random_workload(case, wide)
    run_case(wl, out_dtype, flags=vb.FLAG_PRECISE_BWD if wl.heads_q == wl.heads_kv else 0)


def test_fast_backward_flag_stays_close():
    """VSA2_FLAG_FAST_BWD (P and dS rounded once to bf16): same results within the looser figure its documentation states."""
    from oracle import vsa2_oracle as orc
    from vsa2_testlib import CudaPath, oracle_arrays
    wl, _ = random_workload(3)
    data = syn.make_inputs(wl)
    nnz_cap = int(np.minimum(data["budgets"], wl.n_cubes).sum(axis=-1).max()) if wl.select_mode == syn.PER_QUERY_BUDGET else 0
    outs = []
    for flags in (0, vb.FLAG_FAST_BWD):
        run = CudaPath(wl, data, out_dtype=vb.F32, flags=flags, nnz_cap=nnz_cap)
        run.route()
        run.forward()
        outs.append(run.backward())
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    a = oracle_arrays(data)
    want = orc.backward(a["q"], a["k"], a["v"], a["gate"], run.mask, geo, 1.0 / np.sqrt(wl.head_dim), a["do"])
    for name, precise, fast, ref in zip(("dQ", "dK", "dV"), outs[0], outs[1], want):
        e_p, e_f = np.abs(precise - ref).max(), np.abs(fast - ref).max()
        assert e_p <= 2e-2 and e_f <= 4e-2, (name, e_p, e_f)
        assert e_p <= e_f + 1e-6, (name, e_p, e_f)           # the split never makes things worse
