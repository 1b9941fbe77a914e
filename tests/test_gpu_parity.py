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


def full_parity(wl, data, out_dtype=vb.BF16, nnz_cap=0, check_route=True, flags=0):
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    scale = 1.0 / np.sqrt(wl.head_dim)
    run = CudaPath(wl, data, out_dtype=out_dtype, nnz_cap=nnz_cap, flags=flags)
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
    assert_close("dK", dK, dK_ref, bf16_storage=st)
    assert_close("dV", dV, dV_ref, bf16_storage=st)
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


def test_map_overflow_is_reported_and_the_truncated_map_stays_inside_its_capacity():
    """Per-row budgets that need more entries than nnz_cap: vsa2_route reports VSA2_ERR_MAP_OVERFLOW, the row and column
    pointers stop at the capacity (rows past it are empty, the row that crosses it is cut), and forward + backward on that
    map compute the attention of exactly the truncated map (CSR and CSC list the same pairs)."""
    from oracle import vsa2_oracle as orc
    from vsa2_testlib import CudaPath, assert_close, assert_lse_close, csr_to_mask, oracle_arrays, to_f64
    wl = MINI_BUDGET
    data = syn.make_inputs(wl)
    N = wl.n_cubes
    data["budgets"] = np.full((wl.batch, wl.heads_q, N), 3, dtype=np.int32)
    cap = 3 * N - 7                                  # seven entries short
    run = CudaPath(wl, data, out_dtype=vb.F32, nnz_cap=cap)
    run.attn.route(run.q, run.k, run.budgets)
    with pytest.raises(vb.Vsa2Error) as e:
        run.attn.check_status()
    assert e.value.code == vb.ERR_MAP_OVERFLOW
    rp, ci, cp, ri = (t.cpu().numpy() for t in run.attn.map_views())
    assert rp.max() == cap and cp.max() <= cap and (np.diff(rp, axis=-1) >= 0).all() and (np.diff(cp, axis=-1) >= 0).all()
    mask = csr_to_mask(rp, ci, N)
    counts = mask.sum(axis=-1)
    assert (counts[..., :-3] == 3).all() and counts.sum(axis=-1).max() == cap       # only the last rows are cut
    O, lse = run.attn.forward(run.q, run.k, run.v, run.gate)
    a = oracle_arrays(data)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], a["gate"], mask, geo, 1.0 / np.sqrt(wl.head_dim))
    assert_close("O", to_f64(O), O_ref)
    assert_lse_close(to_f64(lse), lse_ref)
    assert np.array_equal(np.swapaxes(csr_to_mask(cp, ri, N), -1, -2), mask), "the transposed map lists other pairs"
    got = run.attn.backward(run.q, run.k, run.v, run.gate, O, lse, run.do)
    want = orc.backward(a["q"], a["k"], a["v"], a["gate"], mask, geo, 1.0 / np.sqrt(wl.head_dim), a["do"])
    for name, x, y in zip(("dQ", "dK", "dV", "dGate"), got, want):
        assert_close(name, to_f64(x), y)


def test_rescue_list_overflow_is_reported_and_stays_inside_the_list():
    """More query blocks leave the safe range of the fixed-reference softmax than the rescue list may hold (capacity
    lowered to 1 through the test hook): the status word reports it, the list holds exactly one entry, the words behind
    it keep the canary, and the blocks that were not redone are the only wrong ones -- nothing is read or written out of
    bounds and no fault is involved."""
    wl = syn.Workload("late_max_many", 1, 1, 1, 128, (4, 8, 16), select_mode=syn.PER_QUERY, topk=8, kind="iid", seed=43)
    data = syn.make_inputs(wl)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    q = syn.bf16_bits_to_f32(data["q"]).copy()
    k = syn.bf16_bits_to_f32(data["k"]).copy()
    k *= 0.01
    big = geo.cube_tokens[7]
    sgn = np.sign(q[0, 0, big[0]])
    k[0, 0, big] = 8.0 * sgn
    for i in (1, 2, 4):                                         # three query blocks point at the late, huge keys
        q[0, 0, geo.cube_tokens[i]] = 8.0 * sgn
    data["q"], data["k"] = syn.f32_to_bf16_bits(q), syn.f32_to_bf16_bits(k)
    a = oracle_arrays(data)
    O_ref, lse_ref = None, None
    try:
        assert vb._lib().vsa2_debug_rescue_capacity(1) == 1
        run = CudaPath(wl, data, flags=vb.FLAG_NO_COARSE, out_dtype=vb.F32)
        gmask = run.route()
        assert gmask.all()
        run.attn.ws_fwd.view(torch.int32)[64:].fill_(0x5A5A5A5A)          # canary over the list region and beyond
        o, lse = run.attn.forward(run.q, run.k, run.v, run.gate)
        with pytest.raises(vb.Vsa2Error) as e:
            run.attn.check_status()
        assert e.value.code == vb.ERR_UNSUPPORTED
        words = run.attn.ws_fwd.view(torch.int32).cpu().numpy()
        n_over = int(words[2])
        assert n_over >= 3                                                 # at least the three aimed blocks were counted
        assert 0 <= words[64] < geo.N                                      # one was listed and redone
        redone = int(words[64])
        assert (words[65:65 + 4096] == 0x5A5A5A5A).all()                   # nothing written behind the capacity
        O_ref, lse_ref = orc.forward(a["q"], a["k"], a["v"], np.zeros_like(a["gate"]), gmask, geo, 1 / np.sqrt(128))
        O = to_f64(o)
        # blocks whose scores stay small never left the safe range; the listed one was redone: those must be right
        calm = [i for i in range(geo.N) if lse_ref[0, 0, geo.cube_tokens[i]].max() < 40]
        assert len(calm) >= geo.N - n_over
        fine = np.concatenate([geo.cube_tokens[i] for i in calm] + [geo.cube_tokens[redone]])
        assert np.abs(O[0, 0, fine] - O_ref[0, 0, fine]).max() <= TOL_ABS
    finally:
        assert vb._lib().vsa2_debug_rescue_capacity(16384) == 16384
    # with the full capacity the same problem comes back correct and clean
    run = CudaPath(wl, data, flags=vb.FLAG_NO_COARSE, out_dtype=vb.F32)
    run.route()
    O, lse = run.forward()
    assert_close("O", O, O_ref)
    assert_lse_close(lse, lse_ref)


@pytest.mark.parametrize("rpool,G", [((4, 4, 4), 1), ((2, 2, 4), 4), ((1, 2, 2), 16)])
def test_router_with_other_sub_cube_counts(rpool, G):
    """G = 1 is the VSA router of Sec. 2.1 (one pooled token per cube); G = 4 has no tensor-core layout and runs on the
    general router kernel; G = 16 on a 64-token cube (R = 1 x 2 x 2) runs on the tensor-core one."""
    wl = syn.Workload(f"router_g{G}", 1, 2, 1, 128, (5, 10, 12), rpool=rpool, select_mode=syn.PER_SEQUENCE, topk=3, seed=44)
    data = syn.make_inputs(wl, with_grad=False)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    assert geo.G == G
    a = oracle_arrays(data)
    run = CudaPath(wl, data)
    gmask = run.route()
    omask, P = orc.route(a["q"], a["k"], geo, 1.0 / np.sqrt(wl.head_dim), wl.select_mode, wl.topk, return_scores=True)
    pr = to_f64(run.attn.scores())
    assert np.abs(pr - P).max() <= 1e-4 * P.max()
    for h in range(wl.heads_q):
        check_routing(gmask[0, h], omask[0, h], P[0, h], wl.select_mode)


def test_coarse_branch_spanning_two_tiles_with_a_ragged_tail():
    # 84 cubes: the coarse kernels' 64-row tiles see one full and one partial tile on both operands
    full_parity(MINI_COARSE, syn.make_inputs(MINI_COARSE), out_dtype=vb.F32, check_route=False)


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
        assert_close(name, x, y, bf16_storage=name != "dGate")


def test_group_shared_routing_is_refused_for_per_row_budgets():
    wl = MINI_BUDGET
    data = syn.make_inputs(wl)
    data["budgets"] = np.full((1, 2, wl.n_cubes), 2, dtype=np.int32)
    run = CudaPath(wl, data, flags=vb.FLAG_GROUP_ROUTING, nnz_cap=2 * wl.n_cubes)
    with pytest.raises(vb.Vsa2Error) as e:
        run.route()
    assert e.value.code == vb.ERR_UNSUPPORTED


MINI_GQA_TOP8 = syn.Workload("mini_gqa_top8", 1, 4, 2, 128, (8, 12, 12), select_mode=syn.PER_QUERY, topk=8, seed=25)
MINI_SEQ_128 = MINI_SEQ.replace(name="mini_per_sequence_cubes_of_128", cube=(4, 4, 8), rpool=(2, 2, 2), topk=3)


def _grads_of(wl, data, flags):
    run = CudaPath(wl, data, out_dtype=vb.F32, flags=flags)
    run.route()
    run.forward()
    run.backward()
    return (run.dq.clone(), run.dk.clone(), run.dv.clone()), run


@pytest.mark.parametrize("what", ["in_range", "large_k", "large_do"])
@pytest.mark.parametrize("wl", [MINI_SEQ, MINI_GQA_TOP8, MINI_SEQ_128], ids=lambda w: w.name)
def test_backward_leaves_its_fp16_forms_when_a_value_leaves_the_fp16_range(wl, what):
    """The default dQ pass works on fp16 copies of Q and K and rounds dS to fp16; the dK/dV pass does the same for its dK
    product and, for GQA groups that keep 8 blocks or more per row, for all four products.  A finite |K| beyond the fp16
    range, or a dS beyond it (here: a large dO), must hand the passes back to the bf16-pair forms.  VSA2_FLAG_PRECISE_BWD runs
    those directly: dQ then agrees bit for bit, and so do dK and dV of the GQA case (with one query head per KV head the
    fallback of the dK/dV pass takes pairs only for lists longer than 256 -- and none with cubes of 128 tokens --, so here it
    must equal the once-rounded form).  In range the
    forms differ in the last bits, which shows that the fp16 forms are the ones that ran, and all sit inside the stated bound."""
    data = syn.make_inputs(wl)
    if what == "large_k":
        k = data["k"].copy()
        k[0, 0, 5, 3] = 0x4780           # bf16 bits of 65536: finite, beyond the largest fp16 value
        data["k"] = k
    if what == "large_do":
        data["do"] = syn.f32_to_bf16_bits(syn.bf16_bits_to_f32(data["do"]) * np.float32(3.0e6))
    gqa = wl.heads_q != wl.heads_kv
    got, run = _grads_of(wl, data, 0)
    pair, _ = _grads_of(wl, data, vb.FLAG_PRECISE_BWD)
    for t in got:
        assert torch.isfinite(t).all()
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    a = oracle_arrays(data)
    want = orc.backward(a["q"], a["k"], a["v"], a["gate"], run.mask, geo, 1.0 / np.sqrt(wl.head_dim), a["do"])
    if what == "in_range":
        assert not torch.equal(got[0], pair[0]) and not torch.equal(got[1], pair[1])
        for name, x, y, w in zip(("dQ", "dK", "dV"), got, pair, want):
            assert_close(name + " (fp16 form)", to_f64(x), w)
            assert_close(name + " (pair form)", to_f64(y), w)
    else:
        assert torch.equal(got[0], pair[0])
        if gqa:
            assert torch.equal(got[1], pair[1]) and torch.equal(got[2], pair[2])
        else:
            # no list of this problem is longer than 256: the fallback is the once-rounded kernel, which FAST_BWD runs directly
            fast, _ = _grads_of(wl, data, vb.FLAG_FAST_BWD)
            assert torch.equal(got[1], fast[1]) and torch.equal(got[2], fast[2])


def test_dq_pass_falls_back_when_a_row_without_a_token_overflows():
    """The fp16 dQ pass does not mask the dS of key rows that hold no token (positions of an edge cube outside the grid): their
    K rows are zero.  If every score of a query row lies below -88, exp(0 - lse) of such a row overflows, the product turns its
    query column into NaN, and the pass must notice and hand over to the pair form, which masks.  Here all scores are -128 on a
    grid with ragged edges: the results must be finite and equal, bit for bit, to the forms the fallback runs (the problem is
    too ill-conditioned -- all weights equal, gradients from cancellation -- to be compared with the oracle at the usual bound)."""
    # grid (6, 9, 10): ragged in all three directions; every query keeps all 18 cubes, the cut ones at the edges included
    wl = MINI_SEQ.replace(name="mini_dense_ragged", select_mode=syn.PER_QUERY, topk=18)
    data = syn.make_inputs(wl)
    rng = np.random.default_rng(7)
    data["q"] = syn.f32_to_bf16_bits(np.full(data["q"].shape, -16.0, dtype=np.float32))
    data["k"] = syn.f32_to_bf16_bits((1.0 + 0.01 * rng.standard_normal(data["k"].shape)).astype(np.float32))
    got, run = _grads_of(wl, data, 0)
    pair, _ = _grads_of(wl, data, vb.FLAG_PRECISE_BWD)
    fast, _ = _grads_of(wl, data, vb.FLAG_FAST_BWD)
    for t in got:
        assert torch.isfinite(t).all()
    assert run.mask.all()
    assert torch.equal(got[0], pair[0])
    assert torch.equal(got[1], fast[1]) and torch.equal(got[2], fast[2])
