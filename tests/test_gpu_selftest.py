"""GPU check of the tensor-core building blocks (TMA cube tiles, 128-byte swizzle, tcgen05 products)."""
import numpy as np
import pytest
import torch

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn
from vsa2_testlib import dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl,cubes", [
    (syn.Workload("t128", 1, 1, 1, 128, (8, 8, 12), seed=31, kind="iid"), (1, 4, 11)),
    (syn.Workload("t128pad", 1, 1, 1, 128, (5, 6, 9), seed=32, kind="iid"), (0, 5, 11)),   # cubes 5 and 11 are ragged
    (syn.Workload("t64", 1, 1, 1, 64, (4, 8, 8), seed=33, kind="iid"), (3, 0, 2)),
])
def test_tma_cube_tiles_and_tcgen05_products(wl, cubes):
    data = syn.make_inputs(wl, with_grad=False, threads=1)
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    D = wl.head_dim
    p = vb.params_from_workload(wl, topk=1)
    q, k, v = (dev_bf16(data[n]) for n in ("q", "k", "v"))
    rng = np.random.default_rng(7)
    pt_bits = syn.f32_to_bf16_bits(rng.random((128, 64), dtype=np.float32))
    pt = dev_bf16(pt_bits)
    st = torch.zeros(128, 64, device="cuda")
    ot = torch.zeros(128, 64, device="cuda")
    nbytes = 2 * (D // 64) * 8192
    dump = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cq, ca, cb = cubes
    vb.vsa2_selftest_umma(p, q, k, v, cq, ca, cb, pt, st, ot, dump, status)
    torch.cuda.synchronize()
    assert status.item() == 0

    def tile(bits, n):   # 64 x D tile of cube n in (bt, bh, bw) order, zeros at padding
        x = syn.bf16_bits_to_f32(bits[0, 0]).astype(np.float64)
        out = np.zeros((64, D))
        idx = np.full((4, 4, 4), -1)
        nt, nh, nw = n // (geo.Nh * geo.Nw), (n // geo.Nw) % geo.Nh, n % geo.Nw
        for bt in range(4):
            for bh in range(4):
                for bw in range(4):
                    t, h, w = nt * 4 + bt, nh * 4 + bh, nw * 4 + bw
                    if t < geo.T and h < geo.H and w < geo.W:
                        out[(bt * 4 + bh) * 4 + bw] = x[(t * geo.H + h) * geo.W + w]
        return out

    kp = np.concatenate([tile(data["k"], ca), tile(data["k"], cb)])          # [128, D]
    vp = np.concatenate([tile(data["v"], ca), tile(data["v"], cb)])
    qt = tile(data["q"], cq)
    # shared-memory image: slab (half h, block) = 64 rows of 128 bytes, 16-byte chunk c of row r at c ^ (r & 7)
    img = dump.cpu().numpy().view(np.uint16).reshape(-1, 64, 8, 8)            # [slab, row, chunk, 8 elems]
    for h in range(D // 64):
        for blk in range(2):
            slab = img[2 * h + blk]
            got = np.zeros((64, 64), dtype=np.uint16)
            for r in range(64):
                for c in range(8):
                    got[r, c * 8:(c + 1) * 8] = slab[r, c ^ (r & 7)]
            want = syn.f32_to_bf16_bits(kp[blk * 64:(blk + 1) * 64, h * 64:(h + 1) * 64].astype(np.float32))
            assert np.array_equal(got, want), f"tile image differs (half {h}, block {blk})"
    s_ref = kp @ qt.T
    assert np.abs(st.cpu().numpy() - s_ref).max() < 1e-3 * max(1.0, np.abs(s_ref).max())
    o_ref = vp.T @ syn.bf16_bits_to_f32(pt_bits).astype(np.float64)          # [D, 64]
    got_o = ot.cpu().numpy()
    assert np.abs(got_o[:D] - o_ref).max() < 1e-3 * max(1.0, np.abs(o_ref).max())
    if D == 64:
        assert np.abs(got_o[64:] - o_ref).max() < 1e-3 * max(1.0, np.abs(o_ref).max())


def test_a_wait_that_runs_out_reports_a_timeout_and_leaves_the_context_usable():
    """The give-up path of the attention kernels, driven without any fault: a wait on a barrier nothing arrives at runs out
    after 1 ms, the CTA's second waiting role is released by the shared abort flag, the status word reads
    VSA2_ERR_DEVICE_TIMEOUT, tensor memory is handed back -- and an ordinary route + forward right after it succeeds (it
    allocates all 512 tensor-memory columns, so a leaked allocation would make it wait and time out as well)."""
    import time
    from vsa2_testlib import CudaPath
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    lib = vb._lib()
    t0 = time.time()
    for _ in range(3):
        status.zero_()
        rc = lib.vsa2_selftest_timeout(1000, status.data_ptr(), waited.data_ptr(), None)
        assert rc == vb.OK
        torch.cuda.synchronize()
        assert status.item() == vb.ERR_DEVICE_TIMEOUT
        assert 1_000_000 <= waited.item() < 50_000_000          # about 1 ms, nowhere near the kernels' own 2 s limit
    assert time.time() - t0 < 1.5                               # the second role did not sit out its 2 s either
    assert lib.vsa2_selftest_timeout(0, status.data_ptr(), None, None) == vb.ERR_INVALID_ARG
    assert lib.vsa2_selftest_timeout(1000, None, None, None) == vb.ERR_INVALID_ARG
    wl = syn.CONFIGS[0]
    run = CudaPath(wl, syn.make_inputs(wl, threads=1))
    run.route()
    O, lse = run.forward()                                      # check_status inside: VSA2_OK
    assert np.isfinite(O).all()
