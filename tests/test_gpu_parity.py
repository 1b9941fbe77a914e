"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn
from vsa2_testlib import (TOL_ABS, CudaPath, assert_close, assert_lse_close, check_routing, dev_bf16, oracle_arrays, to_f64)

pytestmark = pytest.mark.gpu

# small workloads that span several tiles, a ragged (padded) grid and GQA
MINI_PADDED = syn.Workload("mini_padded_gqa", 1, 4, 2, 128, (5, 6, 9), select_mode=syn.PER_QUERY, topk=3, seed=21)
MINI_SEQ = syn.Workload("mini_per_sequence", 2, 3, 3, 64, (6, 9, 10), select_mode=syn.PER_SEQUENCE, topk=4, seed=22)
MINI_COARSE = syn.Workload("mini_two_coarse_tiles", 1, 2, 1, 128, (8, 24, 28), select_mode=syn.PER_QUERY, topk=16, seed=24)
MINI_BUDGET = syn.Workload("mini_budget", 1, 2, 1, 128, (8, 8, 12), select_mode=syn.PER_QUERY_BUDGET, seed=23)


def full_parity(wl, data, out_dtype=vb.BF16, nnz_cap=0, check_route=True):
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    scale = 1.0 / np.sqrt(wl.head_dim)
    run = CudaPath(wl, data, out_dtype=out_dtype, nnz_cap=nnz_cap)
    a = oracle_arrays(data)
    gmask = run.route()
    if check_route:
        omask, P_r = orc.route(a["q"], a["k"], geo, scale, wl.select_mode, wl.topk, data.get("budgets"), return_scores=True)
        for b in range(wl.batch):
            for h in range(wl.heads_q):
                check_routing(gmask[b, h], omask[b, h], P_r[b, h], wl.select_mode)
        # the GPU's own block scores
        pr_gpu = to_f64(run.attn.scores())
        assert np.abs(pr_gpu - P_r).max() <= 1e-4 * P_r.max()
    # attention parity for the GPU's map
    O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], a["gate"], gmask, geo, scale)
    O, lse = run.forward()
    st = out_dtype == vb.BF16
    assert_close("O", O, O_ref, bf16_storage=st)
    assert_lse_close(lse, lse_ref)
    dQ_ref, dK_ref, dV_ref, dG_ref = orc.backward(a["q"], a["k"], a["v"], a["gate"], gmask, geo, scale, a["do"])
    dQ, dK, dV, dG = run.backward()
    assert_close("dQ", dQ, dQ_ref, bf16_storage=st)
    tol_kv = TOL_ABS * np.sqrt(wl.heads_q // wl.heads_kv)          # group-summed gradients (see vsa2_testlib)
    assert_close("dK", dK, dK_ref, tol_abs=tol_kv, bf16_storage=st)
    assert_close("dV", dV, dV_ref, tol_abs=tol_kv, bf16_storage=st)
    assert_close("dGate", dG, dG_ref)
    return run


def test_config0_tiny_full_parity():
    wl = syn.CONFIGS[0]
    full_parity(wl, syn.make_inputs(wl))


def test_config0_fp32_outputs():
    wl = syn.CONFIGS[0]
    full_parity(wl, syn.make_inputs(wl), out_dtype=vb.F32, check_route=False)


def test_config1_small_video_full_parity():
    wl = syn.CONFIGS[1]
    full_parity(wl, syn.make_inputs(wl))


def test_config1_small_video_fp32_outputs_plain_tolerance():
    wl = syn.CONFIGS[1]
    full_parity(wl, syn.make_inputs(wl), out_dtype=vb.F32, check_route=False)


def test_padded_grid_gqa_full_parity():
    full_parity(MINI_PADDED, syn.make_inputs(MINI_PADDED))


def test_per_sequence_batch2_d64_full_parity():
    run = full_parity(MINI_SEQ, syn.make_inputs(MINI_SEQ))
    rows = run.mask.sum(axis=-1)
    assert (run.mask.sum(axis=(-1, -2)) == run.N * 4).all()          # exactly N*K per (batch, head)
    assert rows.min() != rows.max()                                    # per-sequence TopK gives variable rows


def test_per_query_budget_full_parity():
    wl = MINI_BUDGET
    data = syn.make_inputs(wl)
    N = wl.n_cubes
    rng = np.random.default_rng(5)
    data["budgets"] = rng.integers(0, N + 3, size=(1, 2, N), dtype=np.int32)   # includes 0 (empty rows) and > N
    cap = int(np.minimum(data["budgets"], N).sum(axis=-1).max())
    run = full_parity(wl, data, nnz_cap=cap)
    assert np.array_equal(run.mask.sum(axis=-1), np.minimum(data["budgets"], N))


def test_all_blocks_kept_equals_dense_attention():
    wl = syn.CONFIGS[1].replace(heads_q=2, heads_kv=2, select_mode=syn.PER_SEQUENCE, topk=32)
    data = syn.make_inputs(wl)
    run = CudaPath(wl, data, flags=vb.FLAG_NO_COARSE)
    assert run.route().all()
    O, lse = run.forward()
    q, k, v = (t.float() for t in (run.q, run.k, run.v))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v)
    assert_close("O vs dense SDPA", O, to_f64(ref), bf16_storage=True)


def test_gate_none_and_no_coarse_flag_give_fine_only():
    wl = MINI_PADDED
    data = syn.make_inputs(wl)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    a = oracle_arrays(data)
    run = CudaPath(wl, data, flags=vb.FLAG_NO_COARSE)
    gmask = run.route()
    O, lse = run.forward()
    zero = np.zeros_like(a["gate"])
    O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], zero, gmask, geo, 1 / np.sqrt(wl.head_dim))
    assert_close("O_f", O, O_ref, bf16_storage=True)
    dQ, dK, dV, dG = run.backward()
    dQ_ref, dK_ref, dV_ref, _ = orc.backward(a["q"], a["k"], a["v"], zero, gmask, geo, 1 / np.sqrt(wl.head_dim), a["do"])
    assert_close("dQ", dQ, dQ_ref, bf16_storage=True)
    assert_close("dK", dK, dK_ref, bf16_storage=True)
    assert_close("dV", dV, dV_ref, bf16_storage=True)
    assert (dG == 0).all()


def test_results_are_bitwise_reproducible():
    wl = MINI_PADDED
    data = syn.make_inputs(wl)
    outs = []
    for _ in range(2):
        run = CudaPath(wl, data)
        run.route()
        run.forward()
        run.backward()
        outs.append([t.clone() for t in (run.o, run.lse, run.dq, run.dk, run.dv, run.dgate, run.attn.col_idx, run.attn.row_idx)])
    for x, y in zip(*outs):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))


def test_router_pool_is_bit_exact():
    """Q_r of the GPU equals the oracle's bf16 pooled operands bit for bit (same summation order)."""
    wl = MINI_PADDED
    data = syn.make_inputs(wl)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    run = CudaPath(wl, data)
    run.route()
    s = run.attn.sizes
    n = wl.batch * wl.heads_q * s.n_cubes * s.n_subcubes * wl.head_dim
    qr = run.attn.ws_route[256:256 + 2 * n].view(torch.bfloat16).view(wl.batch, wl.heads_q, s.n_cubes, s.n_subcubes, wl.head_dim)
    for h in range(wl.heads_q):
        ref, valid = orc.mean_pool_router(orc.bf16_bits_to_f64(data["q"][0, h]), geo)
        got = to_f64(qr[0, h])
        assert np.array_equal(got[valid], ref[valid])


def test_bad_arguments_are_rejected_on_the_gpu_box_too():
    wl = syn.CONFIGS[0]
    data = syn.make_inputs(wl)
    run = CudaPath(wl, data)
    with pytest.raises(vb.Vsa2Error) as e:
        vb.vsa2_route(run.p, run.q, run.k, None, run.attn.map, run.attn.ws_route, workspace_bytes=1024)
    assert e.value.code == vb.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(vb.Vsa2Error) as e:
        vb.vsa2_route(run.p, run.q.data_ptr() + 2, run.k, None, run.attn.map, run.attn.ws_route)
    assert e.value.code == vb.ERR_MISALIGNED


def test_tensor_core_forward_matches_exact_maximum_kernel():
    wl = MINI_PADDED
    data = syn.make_inputs(wl)
    outs = []
    for flags in (0, vb.FLAG_EXACT_MAX_FWD):
        run = CudaPath(wl, data, flags=flags, out_dtype=vb.F32)
        run.route()
        outs.append(run.forward())
    assert np.abs(outs[0][0] - outs[1][0]).max() < 2e-2
    assert_lse_close(outs[0][1], outs[1][1])


def test_forward_survives_a_late_dominant_key_block():
    """Scores of the first KV tile are tiny and a later block holds keys scoring hundreds of nats higher:
    the fixed softmax reference of the tensor-core kernel overflows there and the query block must come
    back correct through the exact-maximum fallback."""
    wl = syn.Workload("late_max", 1, 1, 1, 128, (4, 8, 16), select_mode=syn.PER_QUERY, topk=8, kind="iid", seed=41)
    data = syn.make_inputs(wl)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    q = syn.bf16_bits_to_f32(data["q"]).copy()
    k = syn.bf16_bits_to_f32(data["k"]).copy()
    k *= 0.01
    big = geo.cube_tokens[7]
    k[0, 0, big] = 8.0 * np.sign(q[0, 0, big[0]])            # late block: huge, aligned keys
    q[0, 0, geo.cube_tokens[2]] = 8.0 * np.sign(q[0, 0, big[0]])   # one query block points at them
    data["q"], data["k"] = syn.f32_to_bf16_bits(q), syn.f32_to_bf16_bits(k)
    a = oracle_arrays(data)
    run = CudaPath(wl, data, flags=vb.FLAG_NO_COARSE, out_dtype=vb.F32)
    gmask = run.route()
    assert gmask.all()
    O, lse = run.forward()
    O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], np.zeros_like(a["gate"]), gmask, geo, 1 / np.sqrt(128))
    assert lse_ref.max() > 300
    assert_close("O", O, O_ref)
    assert_lse_close(lse, lse_ref)
    rescued = int(run.attn.ws_fwd[8:12].view(torch.int32).item())
    assert rescued >= 1


def test_tensor_core_backward_matches_first_generation_kernels():
    wl = MINI_PADDED
    data = syn.make_inputs(wl)
    outs = []
    for flags in (0, vb.FLAG_SIMPLE_BWD):
        run = CudaPath(wl, data, flags=flags, out_dtype=vb.F32)
        run.route()
        run.forward()
        outs.append(run.backward())
    for name, x, y in zip(("dQ", "dK", "dV", "dGate"), *outs):
        assert np.abs(x - y).max() < 2e-2, name


def test_tensor_core_router_matches_first_generation_kernel():
    wl = MINI_PADDED
    data = syn.make_inputs(wl)
    scores = []
    for flags in (0, vb.FLAG_SIMPLE_ROUTER):
        run = CudaPath(wl, data, flags=flags)
        run.route()
        scores.append(to_f64(run.attn.scores()))
    assert np.abs(scores[0] - scores[1]).max() <= 1e-5 * scores[1].max()
    assert np.allclose(scores[0].sum(axis=-1), 1.0 / 8, atol=1e-5)      # rows of P_r sum to 1/G


def test_coarse_branch_spanning_two_tiles_with_a_ragged_tail():
    # 84 cubes: the coarse kernels' 64-row tiles see one full and one partial tile on both operands
    full_parity(MINI_COARSE, syn.make_inputs(MINI_COARSE), out_dtype=vb.F32, check_route=False)


def test_tensor_core_coarse_branch_matches_fp32_kernels():
    wl = MINI_COARSE
    data = syn.make_inputs(wl)
    outs = []
    for flags in (0, vb.FLAG_SIMPLE_COARSE):
        run = CudaPath(wl, data, flags=flags, out_dtype=vb.F32)
        run.route()
        O, lse = run.forward()
        outs.append((O,) + tuple(run.backward()))
    for name, x, y in zip(("O", "dQ", "dK", "dV", "dGate"), *outs):
        # TF32 operands carry 2^-11 relative rounding; dGate sums 128 such products of magnitude up to ~4
        assert np.abs(x - y).max() < 5e-3, name


def test_bf16_coarse_forward_flag_keeps_the_output_bound():
    # the optional forward of the coarse branch on the pooled grid (bf16 operands): O and LSE within the stated bounds
    for wl in (syn.CONFIGS[1], MINI_COARSE):
        data = syn.make_inputs(wl)
        geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
        scale = 1.0 / np.sqrt(wl.head_dim)
        run = CudaPath(wl, data, flags=vb.FLAG_BF16_COARSE_FWD, out_dtype=vb.F32)
        gmask = run.route()
        a = oracle_arrays(data)
        O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], a["gate"], gmask, geo, scale)
        O, lse = run.forward()
        assert_close("O", O, O_ref)
        assert_lse_close(lse, lse_ref)


@pytest.mark.parametrize("wl", [
    syn.Workload("shared_gqa", 1, 8, 2, 128, (5, 6, 9), select_mode=syn.PER_SEQUENCE, topk=3, seed=31),
    syn.Workload("shared_gqa_rows", 2, 4, 2, 64, (6, 9, 10), select_mode=syn.PER_QUERY, topk=4, seed=32),
    syn.Workload("shared_gqa_wide", 1, 4, 2, 128, (7, 10, 28), cube=(4, 4, 8), select_mode=syn.PER_SEQUENCE, topk=8, seed=33),
], ids=lambda w: w.name)
def test_group_shared_routing(wl):
    """VSA2_FLAG_GROUP_ROUTING: one map per KV group, selected on the summed scores of the group's heads; the attention
    forward and backward then run on those maps as on any other."""
    data = syn.make_inputs(wl)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    scale = 1.0 / np.sqrt(wl.head_dim)
    a = oracle_arrays(data)
    run = CudaPath(wl, data, flags=vb.FLAG_GROUP_ROUTING)
    gmask = run.route()
    omask, P = orc.route(a["q"], a["k"], geo, scale, wl.select_mode, wl.topk, return_scores=True, share_group=True)
    rep = wl.heads_q // wl.heads_kv
    for b in range(wl.batch):
        for h in range(wl.heads_q):
            assert np.array_equal(gmask[b, h], gmask[b, h - h % rep])            # identical inside a group
            check_routing(gmask[b, h], omask[b, h], P[b, h], wl.select_mode)
    pr_gpu = to_f64(run.attn.scores())
    assert np.abs(pr_gpu - P).max() <= 1e-4 * P.max()
    O, lse = run.forward()
    O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], a["gate"], gmask, geo, scale)
    assert_close("O", O, O_ref, bf16_storage=True)
    assert_lse_close(lse, lse_ref)
    got = run.backward()
    want = orc.backward(a["q"], a["k"], a["v"], a["gate"], gmask, geo, scale, a["do"])
    for name, x, y in zip(("dQ", "dK", "dV", "dGate"), got, want):
        tol = TOL_ABS * (np.sqrt(rep) if name in ("dK", "dV") else 1.0)
        assert_close(name, x, y, tol_abs=tol, bf16_storage=name != "dGate")


def test_group_shared_routing_is_refused_for_per_row_budgets():
    wl = MINI_BUDGET
    data = syn.make_inputs(wl)
    data["budgets"] = np.full((1, 2, wl.n_cubes), 2, dtype=np.int32)
    run = CudaPath(wl, data, flags=vb.FLAG_GROUP_ROUTING, nnz_cap=2 * wl.n_cubes)
    with pytest.raises(vb.Vsa2Error) as e:
        run.route()
    assert e.value.code == vb.ERR_UNSUPPORTED
