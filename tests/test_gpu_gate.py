"""GPU parity of the gate projection gate = tanh(X W_g) (Eq. 13) and its backward, through the C ABI, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn

pytestmark = pytest.mark.gpu


def run_gate(batch, heads, grid, hidden, seed, out_dtype=vb.BF16, w_scale=None):
    rng = np.random.default_rng(seed)
    L = int(np.prod(grid))
    xb = syn.f32_to_bf16_bits(rng.standard_normal((batch, L, hidden)).astype(np.float32))
    w_scale = w_scale if w_scale is not None else 1.0 / np.sqrt(hidden)
    wb = syn.f32_to_bf16_bits((rng.standard_normal((hidden, heads)) * w_scale).astype(np.float32))
    dgate = rng.standard_normal((batch, heads, L)).astype(np.float32)
    p = vb.make_params(batch=batch, heads_q=heads, heads_kv=heads, head_dim=64, grid=grid, topk=1, out_dtype=out_dtype)
    dev = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()
    x, w = dev(xb), dev(wb)
    gate = torch.empty(batch, heads, L, dtype=torch.float32, device="cuda")
    vb.vsa2_gate_fwd(p, hidden, x, w, gate)
    ws = torch.empty(max(256, vb.vsa2_gate_bwd_workspace_bytes(p, hidden)), dtype=torch.uint8, device="cuda")
    d_w = torch.empty(hidden, heads, dtype=torch.float32, device="cuda")
    dx = torch.empty(batch, L, hidden, dtype=torch.float32 if out_dtype == vb.F32 else torch.bfloat16, device="cuda")
    vb.vsa2_gate_bwd(p, hidden, x, w, gate, torch.from_numpy(dgate).cuda(), d_w, dx, ws)
    torch.cuda.synchronize()
    X = orc.bf16_bits_to_f64(xb)
    W = orc.bf16_bits_to_f64(wb)
    gate_ref = np.stack([orc.gate_forward(X[b], W) for b in range(batch)])
    dX_ref = np.zeros_like(X)
    dW_ref = np.zeros_like(W)
    for b in range(batch):
        dxb, dwb = orc.gate_backward(X[b], W, dgate[b].astype(np.float64))
        dX_ref[b] = dxb
        dW_ref += dwb
    got = dict(gate=gate.cpu().numpy().astype(np.float64), dx=dx.float().cpu().numpy().astype(np.float64),
               dw=d_w.cpu().numpy().astype(np.float64))
    return got, dict(gate=gate_ref, dx=dX_ref, dw=dW_ref), (p, hidden, x, w, gate, dgate, ws)


def check(got, ref, bf16_dx):
    assert np.abs(got["gate"] - ref["gate"]).max() <= 1e-3                       # bf16 operands are exact, fp32 accumulation
    ex = np.abs(got["dx"] - ref["dx"]) - (2.0 ** -8 * np.abs(ref["dx"]) if bf16_dx else 0.0)
    assert ex.max() <= 2e-2                                                       # dz enters its products rounded to bf16
    scale = np.abs(ref["dw"]).max()
    assert np.abs(got["dw"] - ref["dw"]).max() <= 5e-3 * scale
    assert np.abs(got["dw"] - ref["dw"]).mean() <= 2e-3 * np.abs(ref["dw"]).mean() + 1e-6


@pytest.mark.parametrize("batch,heads,grid,hidden,out_dtype", [
    (2, 5, (3, 5, 7), 72, vb.BF16),            # ragged everywhere: 105 tokens, 72 channels, 5 heads
    (1, 40, (4, 8, 16), 256, vb.BF16),         # the 40 heads of the 720p configuration
    (1, 12, (2, 9, 11), 136, vb.F32),          # channels not a multiple of the 128-channel chunk, fp32 dX
    (2, 64, (4, 4, 9), 64, vb.F32),            # the largest supported head count
])
def test_gate_projection_forward_and_backward(batch, heads, grid, hidden, out_dtype):
    got, ref, _ = run_gate(batch, heads, grid, hidden, seed=7 * heads + hidden, out_dtype=out_dtype)
    check(got, ref, out_dtype == vb.BF16)


def test_gate_projection_at_the_720p_token_count():
    got, ref, args = run_gate(1, 40, (21, 45, 80), 1024, seed=3)
    check(got, ref, True)
    # the reduction over the tokens runs in a fixed order: a second call gives the same bits
    p, hidden, x, w, gate, dgate, ws = args
    d_w2 = torch.empty(hidden, 40, dtype=torch.float32, device="cuda")
    dx2 = torch.empty(1, 75600, hidden, dtype=torch.bfloat16, device="cuda")
    vb.vsa2_gate_bwd(p, hidden, x, w, gate, torch.from_numpy(dgate).cuda(), d_w2, dx2, ws)
    torch.cuda.synchronize()
    assert np.array_equal(d_w2.cpu().numpy().astype(np.float64), got["dw"])


def test_zero_projection_gives_zero_gate_and_zero_dx():
    """The zero-initialised W_g of the paper's training recipe: gate = 0, so O = O_f; dW_g = X^T dgate^T, dX = 0."""
    got, ref, _ = run_gate(1, 8, (2, 4, 8), 64, seed=5, w_scale=0.0, out_dtype=vb.F32)
    assert not got["gate"].any() and not got["dx"].any()
    check(got, ref, False)


def test_gate_feeds_the_attention_forward():
    """The gate written by vsa2_gate_fwd has the layout vsa2_attn_fwd reads."""
    from vsa2_testlib import CudaPath, assert_close, oracle_arrays
    wl = syn.CONFIGS[0]
    data = syn.make_inputs(wl)
    rng = np.random.default_rng(9)
    hidden = 64
    xb = syn.f32_to_bf16_bits(rng.standard_normal((wl.batch, wl.L, hidden)).astype(np.float32))
    wb = syn.f32_to_bf16_bits((rng.standard_normal((hidden, wl.heads_q)) * 0.2).astype(np.float32))
    run = CudaPath(wl, data)
    dev = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()
    vb.vsa2_gate_fwd(run.p, hidden, dev(xb), dev(wb), run.gate)
    gmask = run.route()
    O, _ = run.forward()
    a = oracle_arrays(data)
    gate_ref = np.stack([orc.gate_forward(orc.bf16_bits_to_f64(xb[b]), orc.bf16_bits_to_f64(wb)) for b in range(wl.batch)])
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    O_ref, _ = orc.forward(a["q"], a["k"], a["v"], gate_ref, gmask, geo, 1.0 / np.sqrt(wl.head_dim))
    assert_close("O with the projected gate", O, O_ref, bf16_storage=True)
