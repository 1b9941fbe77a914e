"""ctypes binding of libvsa2.so: argument marshalling only, every step runs in the CUDA library.

The functions ``vsa2_query_sizes``, ``vsa2_route``, ``vsa2_attn_fwd``, ``vsa2_attn_bwd`` and
``vsa2_device_status`` mirror the C entry points of ``include/vsa2.h`` and take torch CUDA tensors
(used only for their device pointers) or raw integer addresses.  ``Vsa2Attention`` is a
convenience wrapper that allocates the outputs, maps and workspaces with torch and calls
them in order.  There is no fallback: if the library cannot be loaded, or a call returns an
error code, a ``Vsa2Error`` is raised.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libvsa2.so")

PER_SEQUENCE, PER_QUERY, PER_QUERY_BUDGET = 0, 1, 2
BF16, F32 = 0, 1
FLAG_NO_COARSE = 1
FLAG_EXACT_MAX_FWD = 2
FLAG_FAST_BWD = 4
FLAG_PRECISE_BWD = 8
FLAG_BF16_COARSE_FWD = 64
FLAG_GROUP_ROUTING = 256

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_MISALIGNED = -1, -2, -3, -4
ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_MAP_OVERFLOW = -5, -6, -7
ERR_STATIC_SCRATCH = -8

EXPORTS = ("vsa2_query_sizes", "vsa2_route", "vsa2_route_scores", "vsa2_attn_fwd", "vsa2_attn_bwd",
           "vsa2_device_status", "vsa2_strerror", "vsa2_profile_events", "vsa2_launch_count", "vsa2_selftest_umma", "vsa2_route_noalloc", "vsa2_last_cuda_error",
           "vsa2_gate_fwd", "vsa2_gate_bwd", "vsa2_gate_bwd_workspace_bytes", "vsa2_permute_cube_major",
           "vsa2_selftest_timeout", "vsa2_debug_rescue_capacity", "vsa2_selftest_divmod")

KERNELS = ("pool", "router_lse", "router_pool", "select", "coarse_fwd", "fine_fwd", "bwd_pre", "coarse_bwd",
           "fine_bwd_dq", "fine_bwd_dkv", "pool_router")


class Vsa2Error(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = _lib().vsa2_strerror(code).decode() if _LIB is not None else "library not loaded"
        if code == ERR_CUDA and _LIB is not None:
            msg += ": " + _lib().vsa2_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (code {code})")


class Params(C.Structure):
    _fields_ = [("batch", C.c_int32), ("heads_q", C.c_int32), ("heads_kv", C.c_int32), ("head_dim", C.c_int32),
                ("grid_t", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
                ("cube_t", C.c_int32), ("cube_h", C.c_int32), ("cube_w", C.c_int32),
                ("rpool_t", C.c_int32), ("rpool_h", C.c_int32), ("rpool_w", C.c_int32),
                ("select_mode", C.c_int32), ("topk", C.c_int32), ("keep_fraction", C.c_float),
                ("softmax_scale", C.c_float), ("out_dtype", C.c_int32), ("flags", C.c_int32), ("text_len", C.c_int32),
                ("nnz_cap", C.c_int64)]


class Sizes(C.Structure):
    _fields_ = [("n_cubes", C.c_int32), ("n_subcubes", C.c_int32), ("block_tokens", C.c_int32),
                ("topk_eff", C.c_int32), ("seq_len", C.c_int64), ("nnz_cap", C.c_int64),
                ("ptr_elems", C.c_int64), ("idx_elems", C.c_int64), ("pooled_q_elems", C.c_int64),
                ("pooled_kv_elems", C.c_int64), ("lse_c_elems", C.c_int64), ("o_res_elems", C.c_int64),
                ("route_workspace_bytes", C.c_size_t), ("fwd_workspace_bytes", C.c_size_t),
                ("bwd_workspace_bytes", C.c_size_t), ("tokens_per_head", C.c_int64), ("text_blocks", C.c_int32),
                ("reserved", C.c_int32)]


class Map(C.Structure):
    _fields_ = [("row_ptr", C.c_void_p), ("col_idx", C.c_void_p), ("col_ptr", C.c_void_p), ("row_idx", C.c_void_p)]


class Saved(C.Structure):
    _fields_ = [("qc", C.c_void_p), ("kc", C.c_void_p), ("vc", C.c_void_p), ("oc_hat", C.c_void_p),
                ("lse_c", C.c_void_p), ("o_res", C.c_void_p)]


_LIB = None


def _lib():
    """Loads libvsa2.so (built in-tree by ``build.build_library``); raises if it is missing."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2609_32882_b200.build` (nvcc, sm_100a)")
        lib = C.CDLL(LIB_PATH)
        vp, sz, i32p = C.c_void_p, C.c_size_t, C.POINTER(C.c_int32)
        lib.vsa2_query_sizes.argtypes = [C.POINTER(Params), C.POINTER(Sizes)]
        lib.vsa2_route.argtypes = [C.POINTER(Params), vp, vp, vp, C.POINTER(Map), vp, sz, vp]
        lib.vsa2_route_noalloc.argtypes = [C.POINTER(Params), vp, vp, vp, C.POINTER(Map), vp, vp]
        lib.vsa2_permute_cube_major.argtypes = [C.POINTER(Params), C.c_int32, C.c_int32, vp, vp, vp]
        lib.vsa2_gate_fwd.argtypes = [C.POINTER(Params), C.c_int32, vp, vp, vp, vp]
        lib.vsa2_gate_bwd_workspace_bytes.argtypes = [C.POINTER(Params), C.c_int32]
        lib.vsa2_gate_bwd_workspace_bytes.restype = C.c_size_t
        lib.vsa2_gate_bwd.argtypes = [C.POINTER(Params), C.c_int32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.vsa2_route_scores.argtypes = [C.POINTER(Params), vp]
        lib.vsa2_route_scores.restype = vp
        lib.vsa2_attn_fwd.argtypes = [C.POINTER(Params), vp, vp, vp, vp, C.POINTER(Map), vp, vp, C.POINTER(Saved), vp, sz, vp]
        lib.vsa2_attn_bwd.argtypes = [C.POINTER(Params), vp, vp, vp, vp, C.POINTER(Map), vp, vp, C.POINTER(Saved), vp,
                                      vp, vp, vp, vp, vp, sz, vp]
        lib.vsa2_device_status.argtypes = [vp, vp, i32p]
        lib.vsa2_last_cuda_error.argtypes = []
        lib.vsa2_last_cuda_error.restype = C.c_char_p
        lib.vsa2_strerror.argtypes = [C.c_int]
        lib.vsa2_strerror.restype = C.c_char_p
        lib.vsa2_profile_events.argtypes = [C.c_int32, vp, vp]
        lib.vsa2_selftest_umma.argtypes = [C.POINTER(Params), vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, vp, vp, vp, vp, vp, vp]
        lib.vsa2_selftest_timeout.argtypes = [C.c_uint32, vp, vp, vp]
        lib.vsa2_debug_rescue_capacity.argtypes = [C.c_int32]
        lib.vsa2_launch_count.argtypes = []
        lib.vsa2_launch_count.restype = C.c_int64
        lib.vsa2_selftest_divmod.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32]
        lib.vsa2_selftest_divmod.restype = C.c_int64
        for name in EXPORTS:
            if name not in ("vsa2_strerror", "vsa2_route_scores", "vsa2_launch_count", "vsa2_last_cuda_error", "vsa2_selftest_divmod"):
                getattr(lib, name).restype = C.c_int
        _LIB = lib
    return _LIB


def _ptr(t):
    """Device address of a torch tensor (or an int address, or None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(code, where):
    if code != OK:
        raise Vsa2Error(code, where)


def make_params(batch, heads_q, heads_kv, head_dim, grid, cube=(4, 4, 4), rpool=(2, 2, 2),
                select_mode=PER_SEQUENCE, topk=0, keep_fraction=0.0, softmax_scale=0.0, out_dtype=BF16,
                flags=0, nnz_cap=0, text_len=0) -> Params:
    return Params(batch, heads_q, heads_kv, head_dim, *grid, *cube, *rpool, select_mode, topk, keep_fraction,
                  softmax_scale, out_dtype, flags, text_len, nnz_cap)


def params_from_workload(wl, **overrides) -> Params:
    kw = dict(batch=wl.batch, heads_q=wl.heads_q, heads_kv=wl.heads_kv, head_dim=wl.head_dim, grid=wl.grid,
              cube=wl.cube, rpool=wl.rpool, select_mode=wl.select_mode, topk=wl.topk,
              text_len=getattr(wl, "text_len", 0))
    kw.update(overrides)
    return make_params(**kw)


# ---------------------------------------------------------------------------------------------
# one-to-one wrappers of the C entry points
# ---------------------------------------------------------------------------------------------
def vsa2_query_sizes(p: Params) -> Sizes:
    s = Sizes()
    _check(_lib().vsa2_query_sizes(C.byref(p), C.byref(s)), "vsa2_query_sizes")
    return s


def vsa2_route(p, q, k, budgets, vmap: Map, workspace, workspace_bytes=None, stream=None):
    nbytes = workspace_bytes if workspace_bytes is not None else workspace.numel() * workspace.element_size()
    _check(_lib().vsa2_route(C.byref(p), _ptr(q), _ptr(k), _ptr(budgets), C.byref(vmap), _ptr(workspace), nbytes,
                             _stream(stream)), "vsa2_route")


def vsa2_route_noalloc(p, q, k, budgets, vmap: Map, device_status=None, stream=None):
    """Router + selection without a caller workspace (scratch is a fixed 8 MiB array inside the library).

    For callers that cannot allocate device memory at this point; problems needing more scratch raise
    Vsa2Error(ERR_STATIC_SCRATCH).  `device_status`: optional int32 CUDA tensor receiving the status word."""
    _check(_lib().vsa2_route_noalloc(C.byref(p), _ptr(q), _ptr(k), _ptr(budgets), C.byref(vmap), _ptr(device_status),
                                     _stream(stream)), "vsa2_route_noalloc")


def vsa2_permute_cube_major(p, heads, src, dst, inverse=False, stream=None):
    """Raster [B, heads, L, D] -> cube-major [B, heads, N*B, D] (zero padding), or back with inverse=True; bf16."""
    _check(_lib().vsa2_permute_cube_major(C.byref(p), heads, 1 if inverse else 0, _ptr(src), _ptr(dst), _stream(stream)),
           "vsa2_permute_cube_major")


def vsa2_gate_fwd(p, hidden, x, w_g, gate, stream=None):
    """gate[b, h, l] = tanh(sum_c x[b, l, c] w_g[c, h]) (Eq. 13); x [B, L, hidden] bf16, w_g [hidden, Hq] bf16, gate [B, Hq, L] fp32."""
    _check(_lib().vsa2_gate_fwd(C.byref(p), hidden, _ptr(x), _ptr(w_g), _ptr(gate), _stream(stream)), "vsa2_gate_fwd")


def vsa2_gate_bwd_workspace_bytes(p, hidden) -> int:
    return int(_lib().vsa2_gate_bwd_workspace_bytes(C.byref(p), hidden))


def vsa2_gate_bwd(p, hidden, x, w_g, gate, dgate, d_w_g, dx, workspace, stream=None):
    """Backward of vsa2_gate_fwd: d_w_g [hidden, Hq] fp32 and dx [B, L, hidden] (the params' output dtype)."""
    nbytes = workspace.numel() * workspace.element_size()
    _check(_lib().vsa2_gate_bwd(C.byref(p), hidden, _ptr(x), _ptr(w_g), _ptr(gate), _ptr(dgate), _ptr(d_w_g), _ptr(dx),
                                _ptr(workspace), nbytes, _stream(stream)), "vsa2_gate_bwd")


def vsa2_route_scores(p, workspace) -> int:
    return _lib().vsa2_route_scores(C.byref(p), _ptr(workspace))


def vsa2_attn_fwd(p, q, k, v, gate, vmap: Map, o, lse, saved, workspace, workspace_bytes=None, stream=None):
    nbytes = workspace_bytes if workspace_bytes is not None else workspace.numel() * workspace.element_size()
    _check(_lib().vsa2_attn_fwd(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate), C.byref(vmap), _ptr(o), _ptr(lse),
                                C.byref(saved) if saved is not None else None, _ptr(workspace), nbytes,
                                _stream(stream)), "vsa2_attn_fwd")


def vsa2_attn_bwd(p, q, k, v, gate, vmap: Map, o, lse, saved, d_o, dq, dk, dv, dgate, workspace,
                  workspace_bytes=None, stream=None):
    nbytes = workspace_bytes if workspace_bytes is not None else workspace.numel() * workspace.element_size()
    _check(_lib().vsa2_attn_bwd(C.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate), C.byref(vmap), _ptr(o), _ptr(lse),
                                C.byref(saved) if saved is not None else None, _ptr(d_o), _ptr(dq), _ptr(dk),
                                _ptr(dv), _ptr(dgate), _ptr(workspace), nbytes, _stream(stream)), "vsa2_attn_bwd")


def vsa2_profile_events(kernel_id: int, start_event, stop_event):
    """start/stop: torch.cuda.Event objects (already recorded once, so that their handles exist) or None."""
    a = None if start_event is None else start_event.cuda_event
    b = None if stop_event is None else stop_event.cuda_event
    _check(_lib().vsa2_profile_events(kernel_id, a, b), "vsa2_profile_events")


def vsa2_selftest_umma(p, q, k, v, cube_q, cube_a, cube_b, p_t, s_t_out, o_t_out, k_tile_dump, status, stream=None):
    _check(_lib().vsa2_selftest_umma(C.byref(p), _ptr(q), _ptr(k), _ptr(v), cube_q, cube_a, cube_b, _ptr(p_t),
                                     _ptr(s_t_out), _ptr(o_t_out), _ptr(k_tile_dump), _ptr(status), _stream(stream)),
           "vsa2_selftest_umma")


def vsa2_launch_count() -> int:
    return int(_lib().vsa2_launch_count())


def vsa2_device_status(workspace, stream=None) -> int:
    out = C.c_int32(0)
    _check(_lib().vsa2_device_status(_ptr(workspace), _stream(stream), C.byref(out)), "vsa2_device_status")
    return out.value


# ---------------------------------------------------------------------------------------------
# convenience wrapper: owns maps, saved state and workspaces (torch is used for memory only)
# ---------------------------------------------------------------------------------------------
class Vsa2Attention:
    """Allocates what the C ABI wants with torch and calls route / forward / backward."""

    def __init__(self, params: Params, device="cuda"):
        import torch
        self.torch = torch
        self.p = params
        self.sizes = vsa2_query_sizes(params)
        s = self.sizes
        dev = torch.device(device)
        i32 = dict(dtype=torch.int32, device=dev)
        f32 = dict(dtype=torch.float32, device=dev)
        self.row_ptr = torch.empty(s.ptr_elems, **i32)
        self.col_idx = torch.empty(max(1, s.idx_elems), **i32)
        self.col_ptr = torch.empty(s.ptr_elems, **i32)
        self.row_idx = torch.empty(max(1, s.idx_elems), **i32)
        self.map = Map(self.row_ptr.data_ptr(), self.col_idx.data_ptr(), self.col_ptr.data_ptr(), self.row_idx.data_ptr())
        self.qc = torch.empty(s.pooled_q_elems, **f32)
        self.kc = torch.empty(s.pooled_kv_elems, **f32)
        self.vc = torch.empty(s.pooled_kv_elems, **f32)
        self.oc_hat = torch.empty(s.pooled_q_elems, **f32)
        self.lse_c = torch.empty(s.lse_c_elems, **f32)
        self.o_res = torch.empty(s.o_res_elems, dtype=torch.bfloat16, device=dev) if s.o_res_elems else None
        self.saved = Saved(self.qc.data_ptr(), self.kc.data_ptr(), self.vc.data_ptr(), self.oc_hat.data_ptr(),
                           self.lse_c.data_ptr(), self.o_res.data_ptr() if s.o_res_elems else None)
        u8 = dict(dtype=torch.uint8, device=dev)
        self.ws_route = torch.empty(s.route_workspace_bytes, **u8)
        self.ws_fwd = torch.empty(s.fwd_workspace_bytes, **u8)
        self.ws_bwd = torch.empty(s.bwd_workspace_bytes, **u8)
        for ws in (self.ws_route, self.ws_fwd, self.ws_bwd):
            ws[:256].zero_()          # status block
        self.out_torch_dtype = torch.float32 if params.out_dtype == F32 else torch.bfloat16

    # shapes ---------------------------------------------------------------------------------
    def map_views(self):
        """(row_ptr [B,Hq,N+1], col_idx [B,Hq,nnz_cap], col_ptr, row_idx) as torch views."""
        p, s = self.p, self.sizes
        shp = (p.batch, p.heads_q)
        return (self.row_ptr.view(*shp, s.n_cubes + 1), self.col_idx[:s.idx_elems].view(*shp, s.nnz_cap),
                self.col_ptr.view(*shp, s.n_cubes + 1), self.row_idx[:s.idx_elems].view(*shp, s.nnz_cap))

    def scores(self):
        """P_r [B,Hq,N,N] fp32 left in the route workspace by the last route() call (a copy)."""
        p, s = self.p, self.sizes
        addr = vsa2_route_scores(p, self.ws_route)
        off = addr - self.ws_route.data_ptr()
        n = p.batch * p.heads_q * s.n_cubes * s.n_cubes
        return self.ws_route[off:off + 4 * n].view(self.torch.float32).view(p.batch, p.heads_q, s.n_cubes, s.n_cubes).clone()

    # calls ----------------------------------------------------------------------------------
    def route(self, q, k, budgets=None, stream=None):
        vsa2_route(self.p, q, k, budgets, self.map, self.ws_route, stream=stream)

    def forward(self, q, k, v, gate, o=None, lse=None, stream=None):
        torch, p = self.torch, self.p
        if o is None:
            o = torch.empty(q.shape, dtype=self.out_torch_dtype, device=q.device)
        if lse is None:
            lse = torch.empty(q.shape[:-1], dtype=torch.float32, device=q.device)
        vsa2_attn_fwd(p, q, k, v, gate, self.map, o, lse, self.saved, self.ws_fwd, stream=stream)
        return o, lse

    def backward(self, q, k, v, gate, o, lse, d_o, dq=None, dk=None, dv=None, dgate=None, stream=None):
        torch, p = self.torch, self.p
        if dq is None:
            dq = torch.empty(q.shape, dtype=self.out_torch_dtype, device=q.device)
        if dk is None:
            dk = torch.empty(k.shape, dtype=self.out_torch_dtype, device=q.device)
        if dv is None:
            dv = torch.empty(v.shape, dtype=self.out_torch_dtype, device=q.device)
        if dgate is None:      # video tokens only (text tokens have no gate)
            dgate = torch.empty(q.shape[:-2] + (self.sizes.seq_len,), dtype=torch.float32, device=q.device)
        vsa2_attn_bwd(p, q, k, v, gate, self.map, o, lse, self.saved, d_o, dq, dk, dv, dgate, self.ws_bwd, stream=stream)
        return dq, dk, dv, dgate

    def check_status(self, stream=None):
        for name, ws in (("route", self.ws_route), ("fwd", self.ws_fwd), ("bwd", self.ws_bwd)):
            code = vsa2_device_status(ws, stream)
            if code != OK:
                raise Vsa2Error(code, f"device status after {name}")
