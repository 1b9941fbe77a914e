"""GPU parity with text tokens (the sentence after Eq. 12: video and text tokens share the attention space): every token
tensor holds the video tokens followed by the text tokens; video queries attend their kept video cubes plus all text keys,
text queries attend everything.  Compared element by element with the oracle's joint functions."""
import numpy as np
import pytest
import torch

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn
from vsa2_testlib import CudaPath, assert_close, assert_lse_close, check_routing, to_f64

pytestmark = pytest.mark.gpu


def joint_oracle(wl, data, gmask, backward=True):
    """Oracle forward (and backward) of every head for the GPU's map; returns arrays shaped like the library's."""
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    L, Lt, D = wl.L, wl.text_len, wl.head_dim
    scale = 1.0 / np.sqrt(D)
    rep = wl.heads_q // wl.heads_kv
    f = {k: orc.bf16_bits_to_f64(data[k]) for k in ("q", "k", "v", "do") if k in data}
    gate = data["gate"].astype(np.float64)
    B, Hq, Hk = wl.batch, wl.heads_q, wl.heads_kv
    out = dict(O=np.zeros((B, Hq, L + Lt, D)), lse=np.zeros((B, Hq, L + Lt)), dQ=np.zeros((B, Hq, L + Lt, D)),
               dK=np.zeros((B, Hk, L + Lt, D)), dV=np.zeros((B, Hk, L + Lt, D)), dGate=np.zeros((B, Hq, L)))
    for b in range(B):
        for h in range(Hq):
            hk = h // rep
            Q, K, V = f["q"][b, h], f["k"][b, hk], f["v"][b, hk]
            args = (Q[:L], K[:L], V[:L], Q[L:], K[L:], V[L:], gate[b, h], gmask[b, h], geo, scale)
            fw = orc.joint_head_forward(*args)
            out["O"][b, h] = np.concatenate((fw["O"], fw["O_t"]))
            out["lse"][b, h] = np.concatenate((fw["lse"], fw["lse_t"]))
            if backward:
                dO = f["do"][b, h]
                gr = orc.joint_head_backward(*args, dO[:L], dO[L:], fwd=fw)
                out["dQ"][b, h] = np.concatenate((gr["dQ"], gr["dQt"]))
                out["dK"][b, hk] += np.concatenate((gr["dK"], gr["dKt"]))
                out["dV"][b, hk] += np.concatenate((gr["dV"], gr["dVt"]))
                out["dGate"][b, h] = gr["dGate"]
    return out


def run_case(wl, out_dtype=vb.BF16, nnz_cap=0):
    data = syn.make_inputs(wl)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    L = wl.L
    run = CudaPath(wl, data, out_dtype=out_dtype, nnz_cap=nnz_cap)
    assert run.attn.sizes.tokens_per_head == L + wl.text_len and run.attn.sizes.text_blocks == -(-wl.text_len // 64)
    gmask = run.route()
    # routing sees the video tokens only
    q = orc.bf16_bits_to_f64(data["q"])[:, :, :L]
    k = orc.bf16_bits_to_f64(data["k"])[:, :, :L]
    omask, P = orc.route(q, k, geo, 1.0 / np.sqrt(wl.head_dim), wl.select_mode, wl.topk, data.get("budgets"), return_scores=True)
    for b in range(wl.batch):
        for h in range(wl.heads_q):
            check_routing(gmask[b, h], omask[b, h], P[b, h], wl.select_mode)
    ref = joint_oracle(wl, data, gmask)
    st = out_dtype == vb.BF16
    O, lse = run.forward()
    assert_close("O (video)", O[:, :, :L], ref["O"][:, :, :L], bf16_storage=st)
    assert_close("O (text)", O[:, :, L:], ref["O"][:, :, L:], bf16_storage=st)
    assert_lse_close(lse, ref["lse"])
    dQ, dK, dV, dG = run.backward()
    for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
        assert_close(name + " (video)", got[:, :, :L], ref[name][:, :, :L], bf16_storage=st)
        assert_close(name + " (text)", got[:, :, L:], ref[name][:, :, L:], bf16_storage=st)
    assert dG.shape == ref["dGate"].shape
    assert_close("dGate", dG, ref["dGate"])
    return run


@pytest.mark.parametrize("wl,dt", [
    (syn.Workload("text_tiny", 1, 2, 2, 64, (4, 8, 8), select_mode=syn.PER_QUERY, topk=2, kind="iid", seed=51, text_len=37), vb.F32),
    (syn.Workload("text_padded_gqa", 1, 4, 2, 128, (5, 6, 9), select_mode=syn.PER_QUERY, topk=3, seed=52, text_len=100), vb.BF16),
    (syn.Workload("text_per_sequence", 2, 3, 3, 64, (6, 9, 10), select_mode=syn.PER_SEQUENCE, topk=4, seed=53, text_len=64), vb.F32),
    (syn.Workload("text_small_video", 1, 4, 4, 128, (8, 16, 16), select_mode=syn.PER_QUERY, topk=8, seed=54, text_len=130), vb.BF16),
], ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_text_tokens_full_parity(wl, dt):
    run_case(wl, out_dtype=dt)


def test_text_tokens_with_empty_video_rows():
    """Per-row budgets of zero: such a video query attends the text keys only."""
    wl = syn.Workload("text_budget", 1, 2, 1, 128, (8, 8, 12), select_mode=syn.PER_QUERY_BUDGET, seed=55, text_len=50)
    data = syn.make_inputs(wl)
    N = wl.n_cubes
    rng = np.random.default_rng(5)
    data["budgets"] = rng.integers(0, 4, size=(wl.batch, wl.heads_q, N), dtype=np.int32)
    data["budgets"][0, 0, 3] = 0

    def make(w, **kw):
        return data
    orig = syn.make_inputs
    syn.make_inputs = make
    try:
        run = run_case(wl, out_dtype=vb.F32, nnz_cap=int(data["budgets"].sum(axis=-1).max()))
    finally:
        syn.make_inputs = orig
    assert np.array_equal(run.mask.sum(axis=-1), data["budgets"])


@pytest.mark.parametrize("wl,dt", [
    (syn.Workload("text_wide_gqa", 1, 4, 2, 128, (7, 10, 29), select_mode=syn.PER_QUERY, topk=3, seed=56, text_len=100,
                  cube=(4, 4, 8), rpool=(2, 2, 2)), vb.BF16),
    (syn.Workload("text_wide_per_sequence", 1, 2, 2, 64, (8, 8, 32), select_mode=syn.PER_SEQUENCE, topk=4, seed=57, text_len=70,
                  cube=(4, 4, 8), rpool=(2, 2, 2)), vb.F32),
], ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_text_tokens_with_cubes_of_128_tokens(wl, dt):
    """The paper's own cube with text tokens: the map is expanded to the 64-token halves, the text blocks are appended to that
    block problem, and the 64-token kernels run it."""
    run = run_case(wl, out_dtype=dt)
    assert run.attn.sizes.block_tokens == 128


def test_zero_text_tokens_is_the_plain_problem():
    wl = syn.CONFIGS[1]
    data = syn.make_inputs(wl)
    a = CudaPath(wl, data)
    b = CudaPath(wl.replace(text_len=0), data)
    a.route(); b.route()
    Oa, la = a.forward()
    Ob, lb = b.forward()
    assert np.array_equal(Oa, Ob) and np.array_equal(la, lb)
