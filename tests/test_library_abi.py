"""CPU-only checks of the C ABI: the library builds and loads, exports every symbol the header
declares, and its host-side argument logic behaves as documented (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import build as vbuild
from paper_2609_32882_b200 import inputs as syn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    vbuild.build_library()
    return ctypes.CDLL(vb.LIB_PATH)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "vsa2.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vsa2_[a-z_0-9]+)\s*\(", text)))


def test_header_functions_are_exported(lib):
    names = declared_functions()
    assert {"vsa2_query_sizes", "vsa2_route", "vsa2_attn_fwd", "vsa2_attn_bwd", "vsa2_device_status",
            "vsa2_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/vsa2.h but not exported"
    for n in vb.EXPORTS:
        assert n in names


def test_query_sizes_matches_the_geometry_of_the_five_configs():
    expect = {0: (4, 256, 2), 1: (32, 2048, 8), 2: (624, 32760, 78), 3: (1440, 75600, 64)}
    for c, (N, L, K) in expect.items():
        wl = syn.CONFIGS[c]
        s = vb.vsa2_query_sizes(vb.params_from_workload(wl))
        assert (s.n_cubes, s.seq_len, s.topk_eff, s.n_subcubes, s.block_tokens) == (N, L, K, 8, 64)
        assert s.nnz_cap == N * K
        assert s.ptr_elems == wl.batch * wl.heads_q * (N + 1)
        assert s.idx_elems == wl.batch * wl.heads_q * N * K
        assert s.pooled_q_elems == wl.batch * wl.heads_q * N * wl.head_dim
        assert s.pooled_kv_elems == wl.batch * wl.heads_kv * N * wl.head_dim
        assert s.route_workspace_bytes > wl.batch * wl.heads_q * N * N * 4
        assert s.route_workspace_bytes % 256 == 0 and s.bwd_workspace_bytes % 256 == 0


def test_backward_workspace_holds_the_fp16_copies_of_the_default_forms():
    """Without a precision flag the backward keeps fp16 copies of Q and K in its workspace (2 bytes per element), for GQA
    groups that keep 8 blocks or more per row also of V and dO; the once-rounded and the pair forms need none."""
    def up(x):
        return (x + 255) // 256 * 256

    def bwd_bytes(wl, **kw):
        return vb.vsa2_query_sizes(vb.params_from_workload(wl, **kw)).bwd_workspace_bytes

    wl = syn.CONFIGS[3]                                    # one query head per KV head
    q16 = up(wl.batch * wl.heads_q * wl.L * wl.head_dim * 2)
    k16 = up(wl.batch * wl.heads_kv * wl.L * wl.head_dim * 2)
    plain = bwd_bytes(wl, flags=vb.FLAG_FAST_BWD)
    assert bwd_bytes(wl, flags=vb.FLAG_PRECISE_BWD) == plain
    assert bwd_bytes(wl) == up(plain) + q16 + k16
    wl = syn.CONFIGS[2]                                    # 12 query heads on 3 KV heads, top-78
    q16 = up(wl.batch * wl.heads_q * wl.L * wl.head_dim * 2)
    k16 = up(wl.batch * wl.heads_kv * wl.L * wl.head_dim * 2)
    plain = bwd_bytes(wl, flags=vb.FLAG_FAST_BWD)
    assert bwd_bytes(wl) == up(plain) + 2 * (q16 + k16)
    assert bwd_bytes(wl, topk=4) == up(plain) + q16 + k16  # rows that keep few blocks: the dK/dV pass stays with its pairs


def test_topk_is_clamped_and_keep_fraction_is_honoured():
    wl = syn.CONFIGS[1]
    assert vb.vsa2_query_sizes(vb.params_from_workload(wl, topk=1000)).topk_eff == 32
    s = vb.vsa2_query_sizes(vb.params_from_workload(wl, topk=0, keep_fraction=0.125))
    assert s.topk_eff == 4
    assert vb.vsa2_query_sizes(vb.params_from_workload(wl, topk=0, keep_fraction=0.001)).topk_eff == 1
    s = vb.vsa2_query_sizes(vb.params_from_workload(syn.CONFIGS[2], topk=0, keep_fraction=0.125))
    assert s.topk_eff == 78                                     # 87.5 % block sparsity of 624 cubes


def test_query_sizes_for_cubes_of_128_tokens():
    s = vb.vsa2_query_sizes(vb.make_params(batch=1, heads_q=4, heads_kv=2, head_dim=128, grid=(7, 10, 29),
                                           cube=(4, 4, 8), topk=5))
    assert (s.n_cubes, s.n_subcubes, s.block_tokens, s.topk_eff) == (2 * 3 * 4, 16, 128, 5)
    assert s.nnz_cap == 24 * 5 and s.ptr_elems == 4 * 25 and s.idx_elems == 4 * 24 * 5
    narrow = vb.vsa2_query_sizes(vb.make_params(batch=1, heads_q=4, heads_kv=2, head_dim=128, grid=(7, 10, 29), topk=10))
    assert narrow.n_cubes == 2 * s.n_cubes
    # the wide problem carries the half-cube problem's scratch plus the cube-level link tensors
    assert s.route_workspace_bytes > 4 * 48 * 48 * 4 and s.bwd_workspace_bytes > narrow.bwd_workspace_bytes // 2


@pytest.mark.parametrize("kw,code", [
    (dict(heads_kv=5), vb.ERR_INVALID_ARG),                       # heads_q % heads_kv
    (dict(head_dim=96), vb.ERR_UNSUPPORTED),
    (dict(cube=(4, 8, 8)), vb.ERR_UNSUPPORTED),                   # 256 tokens per cube
    (dict(cube=(4, 4, 8), rpool=(2, 2, 8)), vb.ERR_UNSUPPORTED),  # router pooling straddles the two half-cubes
    (dict(rpool=(3, 2, 2)), vb.ERR_INVALID_ARG),                  # must divide the cube
    (dict(select_mode=7), vb.ERR_INVALID_ARG),
    (dict(topk=0, keep_fraction=0.0), vb.ERR_INVALID_ARG),
    (dict(topk=-1), vb.ERR_INVALID_ARG),
    (dict(grid=(0, 4, 4)), vb.ERR_INVALID_ARG),
    (dict(out_dtype=3), vb.ERR_INVALID_ARG),
    (dict(select_mode=vb.PER_QUERY_BUDGET, nnz_cap=0), vb.ERR_INVALID_ARG),
])
def test_bad_params_are_rejected(kw, code):
    base = dict(batch=1, heads_q=12, heads_kv=12, head_dim=128, grid=(8, 16, 16), topk=8)
    base.update(kw)
    with pytest.raises(vb.Vsa2Error) as e:
        vb.vsa2_query_sizes(vb.make_params(**base))
    assert e.value.code == code


def test_null_pointers_are_rejected_before_any_cuda_call(lib):
    p = vb.params_from_workload(syn.CONFIGS[0])
    m = vb.Map(0, 0, 0, 0)
    rc = vb._lib().vsa2_route(ctypes.byref(p), None, None, None, ctypes.byref(m), None, 0, None)
    assert rc == vb.ERR_INVALID_ARG
    rc = vb._lib().vsa2_attn_fwd(ctypes.byref(p), None, None, None, None, ctypes.byref(m), None, None, None, None, 0, None)
    assert rc == vb.ERR_INVALID_ARG
    rc = vb._lib().vsa2_attn_bwd(ctypes.byref(p), None, None, None, None, ctypes.byref(m), None, None, None, None,
                                 None, None, None, None, None, 0, None)
    assert rc == vb.ERR_INVALID_ARG
    assert vb._lib().vsa2_device_status(None, None, None) == vb.ERR_INVALID_ARG
    assert vb._lib().vsa2_query_sizes(None, None) == vb.ERR_INVALID_ARG


def test_index_division_by_multiply_is_exact(lib):
    """Every kernel decodes cube and token indices with floor(n * ceil(2^32 / d) / 2^32); the library checks that form on the
    host against n / d: all n < 2^22 for the divisors a grid produces most (up to 64), multiples of d and their neighbours
    for the rest up to 1024."""
    assert lib.vsa2_selftest_divmod(1 << 22, 1, 64, 1024) == 0
    # and the check itself bites: far outside the range the form is exact for (n d < 2^32) it reports mismatches
    assert lib.vsa2_selftest_divmod(0x7fffffff, 1000003, 0, 1000003) > 0


def test_strerror_covers_every_code():
    seen = set()
    for code in range(0, -9, -1):
        msg = vb._lib().vsa2_strerror(code).decode()
        assert msg and "unknown" not in msg
        seen.add(msg)
    assert len(seen) == 9
    assert "unknown" in vb._lib().vsa2_strerror(-99).decode()


def test_binding_refuses_host_tensors():
    import torch
    with pytest.raises(ValueError):
        vb._ptr(torch.zeros(4))


def test_gate_entry_points_reject_unsupported_shapes_before_any_cuda_call():
    lib = vb._lib()                                  # the handle with argument types (size_t arguments)
    p = vb.make_params(batch=1, heads_q=8, heads_kv=8, head_dim=64, grid=(2, 4, 8), topk=1)
    one = ctypes.c_void_p(256)
    assert lib.vsa2_gate_fwd(ctypes.byref(p), 60, one, one, one, None) == vb.ERR_UNSUPPORTED          # hidden % 8
    assert lib.vsa2_gate_fwd(ctypes.byref(p), 64, None, one, one, None) == vb.ERR_INVALID_ARG
    assert lib.vsa2_gate_fwd(ctypes.byref(p), 64, ctypes.c_void_p(8), one, one, None) == vb.ERR_MISALIGNED
    many = vb.make_params(batch=1, heads_q=80, heads_kv=80, head_dim=64, grid=(2, 4, 8), topk=1)
    assert lib.vsa2_gate_fwd(ctypes.byref(many), 64, one, one, one, None) == vb.ERR_UNSUPPORTED       # more than 64 heads
    assert vb.vsa2_gate_bwd_workspace_bytes(many, 64) == 0
    assert vb.vsa2_gate_bwd_workspace_bytes(p, 64) == 16 * 64 * 8 * 4 + 2 * 64 * 16 * 2      # dW_g partials + dz in two layouts
    assert lib.vsa2_gate_bwd(ctypes.byref(p), 64, one, one, one, one, one, one, one, 100, None) == vb.ERR_WORKSPACE_TOO_SMALL
