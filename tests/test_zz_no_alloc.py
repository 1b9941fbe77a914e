"""vsa2_route_noalloc: the allocation-free router entry point, for callers that cannot allocate device memory
where they need a block map (allocation forbidden or stalling at that point, or a memory budget fixed at start-up).
Its scratch is an 8 MiB array inside the library shared by all calls, so the checks run two calls in a row on
different problems and compare each, bit for bit, with what vsa2_route writes for the same inputs."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import build as vbuild
from paper_2609_32882_b200 import inputs as syn


def test_problems_beyond_the_built_in_scratch_are_rejected_without_a_gpu():
    vbuild.build_library()
    p = vb.params_from_workload(syn.CONFIGS[2])                      # 480p shape: 37 MiB of scratch
    assert vb.vsa2_query_sizes(p).route_workspace_bytes > 8 << 20
    m = vb.Map(0, 0, 0, 0)
    rc = vb._lib().vsa2_route_noalloc(ctypes.byref(p), None, None, None, ctypes.byref(m), None, None)
    assert rc == vb.ERR_STATIC_SCRATCH
    assert "8 MiB" in vb._lib().vsa2_strerror(rc).decode()


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_workspace_entry_point():
    from vsa2_testlib import dev_bf16
    big = syn.CONFIGS[1]                                                              # per-query TopK, 1.8 MiB
    small = syn.Workload("mini_seq", 2, 3, 3, 64, (6, 9, 10), select_mode=syn.PER_SEQUENCE, topk=4, seed=22)
    wide = syn.Workload("mini_wide", 1, 4, 2, 128, (7, 10, 28), cube=(4, 4, 8), select_mode=syn.PER_SEQUENCE, topk=5, seed=65)
    for n_call, wl in enumerate((big, small, wide, big)):   # every call after the first runs over the previous call's leftovers
        data = syn.make_inputs(wl, with_grad=False)
        p = vb.params_from_workload(wl)
        q, k = dev_bf16(data["q"]), dev_bf16(data["k"])
        ref = vb.Vsa2Attention(p)
        ref.route(q, k)
        ref.check_status()
        s = ref.sizes
        bufs = [torch.full((n,), -7, dtype=torch.int32, device="cuda")
                for n in (s.ptr_elems, s.idx_elems, s.ptr_elems, s.idx_elems)]
        status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
        m = vb.Map(*(b.data_ptr() for b in bufs))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        vb.vsa2_route_noalloc(p, q, k, None, m, status)
        torch.cuda.synchronize()
        if n_call > 0:       # (the first call on a device may make the driver load the library's device code and back the array)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert status.item() == vb.OK
        for got, want in zip(bufs, (ref.row_ptr, ref.col_idx, ref.col_ptr, ref.row_idx)):
            assert torch.equal(got, want[:got.numel()])
        assert int(bufs[0].view(-1, s.n_cubes + 1)[:, -1].min().item()) == s.nnz_cap     # every head filled its budget
