"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI, run the oracle
on the same seeded inputs, compare with the tolerances the build's target states.

Tolerances (fp32 comparison against the fp64 oracle):
  outputs and gradients: max abs err <= 2e-2 and mean rel err <= 5e-3, where
                         mean rel err = mean|a - b| / mean|b| over the tensor;
  lse:                   max abs err <= 1e-3 where finite, -inf must match -inf;
                         Runs with fp32 outputs (out_dtype F32) are held to exactly these bounds, MHA and GQA alike.
                         When the library stores a tensor in bf16 (out_dtype BF16) the storage rounding alone,
                         up to 2^-8 |x| per element (half an ulp at the bottom of a binade), can exceed 2e-2 for
                         |x| > 5: the elementwise bound of such runs is 2e-2 + 2^-8 |ref|.
  routing:               the map must equal the oracle's except at entries whose oracle score lies
                         within 1e-3 * tau (relative) of the threshold tau = smallest kept score of
                         that (batch, head) [per-sequence] or row [per-query]; counts must be exact.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import vsa2_oracle as orc
from paper_2609_32882_b200 import binding as vb
from paper_2609_32882_b200 import inputs as syn

TOL_ABS, TOL_REL, TOL_LSE, TOL_ROUTE = 2e-2, 5e-3, 1e-3, 1e-3


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def err(a: np.ndarray, b: np.ndarray):
    """(max abs err, mean rel err) of a against the reference b."""
    d = np.abs(a - b)
    return float(d.max()) if d.size else 0.0, float(d.mean() / max(np.abs(b).mean(), 1e-30)) if d.size else 0.0


def assert_close(name, a, b, tol_abs=TOL_ABS, tol_rel=TOL_REL, bf16_storage=False):
    mx, rel = err(a, b)
    if bf16_storage:
        excess = float((np.abs(a - b) - 2.0 ** -8 * np.abs(b)).max()) if a.size else 0.0
        ok_abs = excess <= tol_abs
    else:
        ok_abs = mx <= tol_abs
    assert ok_abs and rel <= tol_rel, (f"{name}: max abs err {mx:.3e} (tol {tol_abs}"
                                       f"{' + bf16 storage rounding' if bf16_storage else ''}), mean rel err {rel:.3e} (tol {tol_rel})")
    return mx, rel


def assert_lse_close(a, b):
    fin = np.isfinite(b)
    assert np.array_equal(np.isneginf(a), np.isneginf(b)), "lse: -inf pattern differs"
    if fin.any():
        mx = float(np.abs(a[fin] - b[fin]).max())
        assert mx <= TOL_LSE, f"lse: max abs err {mx:.3e}"


def csr_to_mask(row_ptr, col_idx, N):
    """row_ptr [..., N+1], col_idx [..., cap] (numpy) -> bool [..., N, N]; also checks ordering."""
    lead = row_ptr.shape[:-1]
    rp = row_ptr.reshape(-1, N + 1)
    ci = col_idx.reshape(rp.shape[0], -1)
    mask = np.zeros((rp.shape[0], N, N), dtype=bool)
    for h in range(rp.shape[0]):
        assert rp[h, 0] == 0 and np.all(np.diff(rp[h]) >= 0)
        for i in range(N):
            cols = ci[h, rp[h, i]:rp[h, i + 1]]
            if cols.size:
                assert np.all(np.diff(cols) > 0), "indices not strictly ascending"
                assert cols[0] >= 0 and cols[-1] < N
            mask[h, i, cols] = True
    return mask.reshape(lead + (N, N))


def check_routing(gpu_mask, oracle_mask, P_r, mode):
    """T1 rule on one (batch, head): gpu_mask, oracle_mask bool [N, N], P_r oracle scores."""
    N = P_r.shape[0]
    p32 = P_r.astype(np.float32).astype(np.float64)
    diff = gpu_mask != oracle_mask
    if mode == orc.PER_SEQUENCE:
        assert gpu_mask.sum() == oracle_mask.sum()
        if diff.any():
            tau = p32[oracle_mask].min()
            assert np.all(np.abs(p32[diff] - tau) <= TOL_ROUTE * tau), "routing differs away from the threshold"
    else:
        assert np.array_equal(gpu_mask.sum(axis=1), oracle_mask.sum(axis=1))
        for i in np.nonzero(diff.any(axis=1))[0]:
            tau = p32[i][oracle_mask[i]].min()
            assert np.all(np.abs(p32[i][diff[i]] - tau) <= TOL_ROUTE * tau), "routing differs away from the row threshold"
    return int(diff.sum())


class CudaPath:
    """Uploads a workload's tensors and drives the library through the binding."""

    def __init__(self, wl, data, out_dtype=vb.BF16, flags=0, nnz_cap=0, **param_overrides):
        self.wl = wl
        self.p = vb.params_from_workload(wl, out_dtype=out_dtype, flags=flags, nnz_cap=nnz_cap, **param_overrides)
        self.attn = vb.Vsa2Attention(self.p)
        self.q, self.k, self.v = dev_bf16(data["q"]), dev_bf16(data["k"]), dev_bf16(data["v"])
        self.gate = torch.from_numpy(data["gate"]).cuda()
        self.do = dev_bf16(data["do"]) if "do" in data else None
        self.budgets = torch.from_numpy(data["budgets"]).cuda() if "budgets" in data else None
        self.N = self.attn.sizes.n_cubes

    def route(self):
        self.attn.route(self.q, self.k, self.budgets)
        self.attn.check_status()
        rp, ci, cp, ri = (t.cpu().numpy() for t in self.attn.map_views())
        self.mask = csr_to_mask(rp, ci, self.N)
        mask_t = csr_to_mask(cp, ri, self.N)
        assert np.array_equal(self.mask, np.swapaxes(mask_t, -1, -2)), "CSR and CSC disagree"
        assert np.array_equal(rp[..., -1], cp[..., -1])
        return self.mask

    def forward(self):
        self.o, self.lse = self.attn.forward(self.q, self.k, self.v, self.gate)
        self.attn.check_status()
        return to_f64(self.o), to_f64(self.lse)

    def backward(self):
        self.dq, self.dk, self.dv, self.dgate = self.attn.backward(self.q, self.k, self.v, self.gate, self.o, self.lse, self.do)
        self.attn.check_status()
        return tuple(to_f64(t) for t in (self.dq, self.dk, self.dv, self.dgate))


def oracle_arrays(data):
    out = {k: orc.bf16_bits_to_f64(data[k]) for k in ("q", "k", "v", "do") if k in data}
    out["gate"] = data["gate"].astype(np.float64)
    return out


def sampled_attention_parity(wl, data, run, gmask, q_heads, rows, kv_groups=(), kv_cubes=(), backward=True):
    """Oracle vs GPU on sampled outputs of a full-size run (the full oracle would take hours):
    O, lse, dQ, dGate on the tokens of the query cubes `rows` of the query heads `q_heads`; dK, dV on the tokens
    of `kv_cubes` for the KV heads `kv_groups` (all query heads of the group, all query blocks that keep the cube).
    `run` is a CudaPath that has executed forward (and backward), or a list of them over the same inputs and map (e.g.
    one with bf16 and one with fp32 outputs): the oracle's sample is computed once and every run is held to the bound
    of its own output dtype.  Returns {tensor name: (max abs err, mean rel err)} of the last run."""
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    scale = 1.0 / np.sqrt(wl.head_dim)
    rep = wl.heads_q // wl.heads_kv
    runs = list(run) if isinstance(run, (list, tuple)) else [run]
    stats = {}

    def check(name, field, idx, ref, plain=False):
        for r in runs:
            st = (not plain) and r.p.out_dtype == vb.BF16
            stats[name] = assert_close(f"{name} ({'bf16' if r.p.out_dtype == vb.BF16 else 'fp32'} outputs)",
                                       to_f64(getattr(r, field)[idx[0], idx[1]][idx[2]]), ref, bf16_storage=st)

    def head_arrays(b, hq):
        hk = hq // rep
        return (orc.bf16_bits_to_f64(data["q"][b, hq]), orc.bf16_bits_to_f64(data["k"][b, hk]),
                orc.bf16_bits_to_f64(data["v"][b, hk]), data["gate"][b, hq].astype(np.float64),
                orc.bf16_bits_to_f64(data["do"][b, hq]) if backward else None)

    def coarse_fwd(Q, K, V):
        Qc, Kc, Vc = orc.mean_pool_cube(Q, geo), orc.mean_pool_cube(K, geo), orc.mean_pool_cube(V, geo)
        Oc_hat, lse_c = orc.coarse_attention(Qc, Kc, Vc, scale)
        return dict(Oc_hat=Oc_hat, lse_c=lse_c, Qc=Qc, Kc=Kc, Vc=Vc)

    b = 0
    for hq in q_heads:
        Q, K, V, gate, dO = head_arrays(b, hq)
        fwd = coarse_fwd(Q, K, V)
        toks = np.concatenate([geo.cube_tokens[i] for i in rows])
        O_f, lse = orc.fine_attention(Q, K, V, gmask[b, hq], geo, scale, rows=rows)
        O_ref = gate[toks, None] * fwd["Oc_hat"][geo.cube_of[toks]] + O_f[toks]
        check(f"O_h{hq}", "o", (b, hq, toks), O_ref)
        for r in runs:
            assert_lse_close(to_f64(r.lse[b, hq][toks]), lse[toks])
        if backward:
            c = orc.coarse_path_backward(Q, K, V, gate, geo, scale, dO, fwd)
            fq, _, _ = orc.fine_backward(Q, K, V, gmask[b, hq], geo, scale, dO, lse, O_f, rows=rows)
            check(f"dQ_h{hq}", "dq", (b, hq, toks), (c["dQ"] + fq)[toks])
            check(f"dGate_h{hq}", "dgate", (b, hq, toks), c["dGate"][toks], plain=True)
    if backward:
        for hk in kv_groups:
            toks = np.concatenate([geo.cube_tokens[j] for j in kv_cubes])
            dK_ref = np.zeros((toks.size, wl.head_dim))
            dV_ref = np.zeros((toks.size, wl.head_dim))
            for hq in range(hk * rep, (hk + 1) * rep):
                Q, K, V, gate, dO = head_arrays(b, hq)
                fwd = coarse_fwd(Q, K, V)
                c = orc.coarse_path_backward(Q, K, V, gate, geo, scale, dO, fwd)
                fk, fv = orc.fine_backward_kv_cubes(Q, K, V, gmask[b, hq], geo, scale, dO, kv_cubes)
                dK_ref += (c["dK"] + fk)[toks]
                dV_ref += (c["dV"] + fv)[toks]
            check(f"dK_g{hk}", "dk", (b, hk, toks), dK_ref)
            check(f"dV_g{hk}", "dv", (b, hk, toks), dV_ref)
    return stats
