#!/usr/bin/env python
"""Benchmark of the VSA2 routed block-sparse attention path on B200.

One step = one pass of the whole hot path over one synthetic 720p-shaped batch:
vsa2_route (pool, router scores, TopK, CSR/CSC) + vsa2_attn_fwd (coarse branch, fine branch, merge)
+ vsa2_attn_bwd (preprocess, coarse backward, dQ, dK/dV), all through the C ABI.

  python bench.py --gpus 1 --steps 5 --warmup 3            # this library
  python bench.py --impl reference --steps 2 --warmup 1    # the CPU oracle on a bounded sample

Prints ONE JSON line (rank 0).  `value` is the dense-equivalent TFLOP/s of forward + backward
(4 L^2 D Hq x 3.5 FLOP of dense attention over the valid tokens divided by the measured step time), the
figure the paper's speed-up over dense attention translates to; `ms_per_step`, the executed (actual)
TFLOP/s and the per-kernel times are reported next to it.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_32882_b200 import inputs as syn  # noqa: E402

METRIC = "720p routed sparse attn fwd+bwd ms and TFLOPS (actual & dense-equiv) vs B200 BF16 peak"
UNIT = "TFLOP/s dense-equivalent"
ORACLE_HOW = "the oracle as it stands: fp64 numpy whose matrix products run on the multithreaded BLAS numpy links"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the 720p top-64 launch with 40 heads: an
# 8-head ncu capture of the same kernels times 5 (every head streams its own tensors, so the traffic grows in
# proportion to the heads; the 40-head launch is too large for a full-set capture).
NCU_TRAFFIC_BYTES_720P_TOP64 = {"fine_fwd": 5 * (0.504200e9 + 0.295100e9),
                                "fine_bwd_dq": 5 * (0.663200e9 + 0.147600e9 + 0.309700e9 + 0.262100e9),   # with the fp16 copy of Q, K
                                "fine_bwd_dkv": 5 * (0.791600e9 + 0.304900e9)}


# What ncu shows as the busiest unit of each tensor kernel at 64-token cubes (8-head capture, profiles/): the roofline
# below is quoted against the tensor peak as the contract asks, these say what actually holds the kernel there.
NCU_LIMITER = {
    "fine_fwd": "L2 -> SM read rate: 12.9 TB/s against 11.8 TB/s sustained peak (tensor pipe 82 % active at the half rate of M = 64)",
    "fine_bwd_dq": "shared-memory data pipe: tensor-core operand fetches 64 % + thread loads/stores 37 % (tensor pipe 43 %)",
    "fine_bwd_dkv": "shared-memory data pipe: tensor-core operand fetches 67 % + thread loads/stores 32 % (tensor pipe 47 %)",
    "router_lse": "exponential unit 81 %, instruction issue 65 %",
    "router_pool": "exponential unit 77 %, instruction issue 69 %",
}
# L2 -> SM read rate that ncu reports as the sustained peak of this part (derived__lts__lts2xbar_bytes.sum.peak_sustained
# in the 8-head capture of profiles/kernels_720p_8heads_ncu_full.md, where the fine forward itself reads 12.0 TB/s).
NCU_L2_TO_SM_PEAK_TBS = 11.776


def workload(config: int, heads: int = 0, topk: int = 0, grid=None, cube=None, text_len: int = 0) -> syn.Workload:
    wl = syn.CONFIGS[config]
    if text_len:
        wl = wl.replace(text_len=text_len, name=f"{wl.name}_text{text_len}")
    if grid:
        wl = wl.replace(grid=tuple(grid), name=f"{wl.name}_grid{'x'.join(map(str, grid))}")
    if cube:
        wl = wl.replace(cube=tuple(cube), name=f"{wl.name}_cube{'x'.join(map(str, cube))}")
    if heads:
        wl = wl.replace(heads_q=heads, heads_kv=max(1, heads * wl.heads_kv // wl.heads_q), name=f"{wl.name}_{heads}heads")
    if topk:
        wl = wl.replace(topk=topk, name=f"{wl.name}_top{topk}")
    return wl


def config_dict(wl: syn.Workload, forward_only: bool) -> dict:
    """The `config` object of the JSON line: what the workload is (both arms print the same)."""
    gb = (2 * wl.heads_q + 2 * wl.heads_kv) * wl.batch * (wl.L + wl.text_len) * wl.head_dim * 2 / 1e9
    return {"workload": wl.name, "grid": list(wl.grid), "tokens": wl.L, "text_tokens": wl.text_len, "heads_q": wl.heads_q, "heads_kv": wl.heads_kv,
            "head_dim": wl.head_dim, "cube": list(wl.cube), "rpool": list(wl.rpool), "select_mode": wl.select_mode,
            "topk": wl.topk, "forward_only": bool(forward_only),
            "l2": f"inputs (Q,K,V,dO: {gb:.1f} GB) far larger than the 126 MB L2; no explicit flush"}


def flop_counts(wl: syn.Workload, nnz_total: int) -> dict:
    """Algorithmic work of one step.  nnz_total = selected (query block, KV block) pairs over all heads."""
    B, D = int(np.prod(wl.cube)), wl.head_dim
    L, Hq, N, G = wl.L + wl.text_len, wl.heads_q * wl.batch, wl.n_cubes, int(np.prod(wl.cube)) // int(np.prod(wl.rpool))
    pair = B * B * D
    return {
        "dense_equiv_fwd": 4.0 * L * L * D * Hq,
        "dense_equiv_fwd_bwd": 3.5 * 4.0 * L * L * D * Hq,
        "fine_fwd": 4.0 * pair * nnz_total,
        "fine_bwd_algorithmic": 10.0 * pair * nnz_total,
        "fine_bwd_dq_executed": 6.0 * pair * nnz_total,
        "fine_bwd_dkv_executed": 8.0 * pair * nnz_total,
        "router_per_pass": 2.0 * (N * G) ** 2 * D * Hq,
        "coarse_fwd": 4.0 * N * N * D * Hq,
    }


def peaks() -> tuple[dict, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample (the reference arm and the cpu_baseline leg)
# ------------------------------------------------------------------------------------------------
def oracle_sample_step(wl: syn.Workload, head_data: dict, n_rows: int) -> dict:
    """Times the oracle, as it stands, on ONE head of the workload: full routing, the coarse branch, and
    the fine branch forward + backward over `n_rows` query blocks; extrapolates to the whole workload."""
    from oracle import vsa2_oracle as orc
    geo = orc.Geometry(wl.grid, wl.cube, wl.rpool)
    scale = 1.0 / np.sqrt(wl.head_dim)
    Q, K, V, dO = (orc.bf16_bits_to_f64(head_data[k]) for k in ("q", "k", "v", "do"))
    gate = head_data["gate"].astype(np.float64)
    t0 = time.perf_counter()
    mask = orc.route(Q[None, None], K[None, None], geo, scale, wl.select_mode, wl.topk,
                     None if "budgets" not in head_data else head_data["budgets"][None, None])[0, 0]
    t1 = time.perf_counter()
    Qc, Kc, Vc = orc.mean_pool_cube(Q, geo), orc.mean_pool_cube(K, geo), orc.mean_pool_cube(V, geo)
    Oc_hat, lse_c = orc.coarse_attention(Qc, Kc, Vc, scale)
    fwd = dict(Oc_hat=Oc_hat, lse_c=lse_c, Qc=Qc, Kc=Kc, Vc=Vc)
    orc.coarse_path_backward(Q, K, V, gate, geo, scale, dO, fwd)
    t2 = time.perf_counter()
    rows = np.linspace(0, geo.N - 1, num=min(n_rows, geo.N)).astype(int)
    O_f, lse = orc.fine_attention(Q, K, V, mask, geo, scale, rows=rows)
    orc.fine_backward(Q, K, V, mask, geo, scale, dO, lse, O_f, rows=rows)
    t3 = time.perf_counter()
    pairs_sample = int(mask[rows].sum())
    pairs_head = int(mask.sum())
    t_fine_head = (t3 - t2) * pairs_head / max(1, pairs_sample)
    t_head = (t1 - t0) + (t2 - t1) + t_fine_head
    heads = wl.heads_q * wl.batch
    return {"t_route_s": t1 - t0, "t_coarse_s": t2 - t1, "t_fine_sample_s": t3 - t2, "rows": len(rows),
            "pairs_sample": pairs_sample, "pairs_head": pairs_head, "t_step_extrapolated_s": t_head * heads,
            "measured_s": t3 - t0}


def head_inputs(wl: syn.Workload, b: int, h: int) -> dict:
    hk = h // (wl.heads_q // wl.heads_kv)
    d = {"q": syn.head_tensor(wl, "q", b, h), "k": syn.head_tensor(wl, "k", b, hk), "v": syn.head_tensor(wl, "v", b, hk),
         "do": syn.head_tensor(wl, "do", b, h), "gate": syn.head_gate(wl, b, h)}
    if wl.select_mode == syn.PER_QUERY_BUDGET:
        d["budgets"] = syn.head_budgets(wl, b, h)
    return d


def cpu_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload(args.config, args.heads, args.topk, args.grid, args.cube, args.text_len)
    hd = head_inputs(wl, 0, 0)
    flops = flop_counts(wl, 0)
    for _ in range(args.warmup):
        oracle_sample_step(wl, hd, args.ref_rows)
    times, last = [], None
    for _ in range(args.steps):
        last = oracle_sample_step(wl, hd, args.ref_rows)
        times.append(last["t_step_extrapolated_s"])
    t = float(np.mean(times))
    value = flops["dense_equiv_fwd_bwd"] / t / 1e12
    sample = (f"head 0 of {wl.heads_q}: full routing + coarse branch + fine fwd/bwd over {last['rows']} of "
              f"{wl.n_cubes} query blocks ({last['pairs_sample']} of {last['pairs_head']} block pairs), "
              f"{last['measured_s']:.1f} s measured per step, extrapolated to all heads and blocks")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(wl, args.forward_only),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": sample,
                             "how": ORACLE_HOW},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2609_32882_b200 import binding as vb
    from paper_2609_32882_b200 import build as vbuild
    from paper_2609_32882_b200 import replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "VERSION")       # one line per job on stderr: the NCCL build in use
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        print(f"[bench] rank {rank} of {dist.get_world_size()} on cuda:{local_rank} ({torch.cuda.get_device_name(local_rank)})",
              file=sys.stderr, flush=True)
    if rank == 0:
        vbuild.build_library()
    if world > 1:
        dist.barrier()
    vb._lib()

    # every rank runs its own replica of the workload (heads are independent: no data-path collective)
    wl = workload(args.config, args.heads, args.topk, args.grid, args.cube, args.text_len)
    wl = wl.replace(seed=replicas.replica_seed(wl.seed, rank))
    t_gen = time.time()
    data = syn.make_inputs(wl, threads=max(1, min(32, cpu_cores() // max(1, world))))
    t_gen = time.time() - t_gen

    def pinned(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).pin_memory()

    host = {k: pinned(data[k]) for k in ("q", "k", "v", "do")}
    host["gate"] = torch.from_numpy(data["gate"]).pin_memory()
    dev = {k: v.cuda(non_blocking=True) for k, v in host.items()}
    budgets = torch.from_numpy(data["budgets"]).cuda() if "budgets" in data else None
    nnz_cap = 0
    if budgets is not None:
        nnz_cap = int(np.minimum(data["budgets"], wl.n_cubes).sum(axis=-1).max())
    p = vb.params_from_workload(wl, nnz_cap=nnz_cap, flags=args.flags)
    attn = vb.Vsa2Attention(p)
    odt = attn.out_torch_dtype
    o = torch.empty_like(dev["q"], dtype=odt)
    lse = torch.empty(dev["q"].shape[:-1], dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(dev["q"], dtype=odt), torch.empty_like(dev["k"], dtype=odt), torch.empty_like(dev["v"], dtype=odt)
    dgate = torch.empty_like(lse)
    host_out = {k: torch.empty(t.shape, dtype=t.dtype).pin_memory() for k, t in (("o", o), ("dq", dq), ("dk", dk), ("dv", dv))}
    stream = torch.cuda.current_stream()

    def step():
        attn.route(dev["q"], dev["k"], budgets)
        attn.forward(dev["q"], dev["k"], dev["v"], dev["gate"], o=o, lse=lse)
        if args.forward_only:
            return
        attn.backward(dev["q"], dev["k"], dev["v"], dev["gate"], o, lse, dev["do"], dq=dq, dk=dk, dv=dv, dgate=dgate)

    # End to end: every step copies its inputs from pinned host memory and its results back, inside the timed region.
    # As a training loop would, the copies run on side streams and overlap the kernels.  Heads are independent, so a
    # step is cut into head chunks (units) that flow through a two-deep pipeline: the inputs of unit i + 1 load and the
    # results of unit i - 1 drain while unit i computes; inside a unit the router starts as soon as Q and K have
    # arrived, the forward when V has, the backward when dO has, and O leaves while the backward runs.
    chunks = next(c for c in range(args.e2e_chunks, 0, -1) if wl.heads_kv % c == 0) if wl.batch == 1 else 1
    hq_c, hk_c = wl.heads_q // chunks, wl.heads_kv // chunks
    attn_e = attn if chunks == 1 else vb.Vsa2Attention(
        vb.params_from_workload(wl.replace(heads_q=hq_c, heads_kv=hk_c), nnz_cap=nnz_cap, flags=args.flags))
    heads_of = {"q": hq_c, "do": hq_c, "gate": hq_c, "k": hk_c, "v": hk_c, "o": hq_c, "dq": hq_c, "dk": hk_c, "dv": hk_c}

    def part(t, name, c):
        return t if chunks == 1 else t[:, c * heads_of[name]:(c + 1) * heads_of[name]]

    def like(t, name, dtype=None):
        return torch.empty_like(part(t, name, 0), dtype=dtype or t.dtype)

    in_sets = [{k: like(dev[k], k) for k in dev} for _ in range(2)]
    out_sets = [dict(o=like(o, "o"), lse=like(lse, "gate"), dq=like(dq, "dq"), dk=like(dk, "dk"), dv=like(dv, "dv"),
                     dgate=like(dgate, "gate")) for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def run_e2e(n_steps):
        units = n_steps * chunks
        ev = {k: [torch.cuda.Event() for _ in range(units)] for k in ("qk", "v", "do", "fwd", "comp", "out")}

        def h2d(i):
            c, d = i % chunks, in_sets[i % 2]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev["comp"][i - 2])       # the buffer set is free once unit i - 2 has computed
                for names, mark in ((("q", "k"), "qk"), (("gate", "v"), "v"), (("do",), "do")):
                    for k in names:
                        d[k].copy_(part(host[k], k, c), non_blocking=True)
                    ev[mark][i].record(s_in)

        h2d(0)
        for i in range(units):
            if i + 1 < units:
                h2d(i + 1)
            c, d, r = i % chunks, in_sets[i % 2], out_sets[i % 2]
            stream.wait_event(ev["qk"][i])
            if i >= 2:
                stream.wait_event(ev["out"][i - 2])          # the result set has been read back
            attn_e.route(d["q"], d["k"], None if budgets is None else part(budgets, "q", c))
            stream.wait_event(ev["v"][i])
            attn_e.forward(d["q"], d["k"], d["v"], d["gate"], o=r["o"], lse=r["lse"])
            ev["fwd"][i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev["fwd"][i])
                part(host_out["o"], "o", c).copy_(r["o"], non_blocking=True)
            if not args.forward_only:
                stream.wait_event(ev["do"][i])
                attn_e.backward(d["q"], d["k"], d["v"], d["gate"], r["o"], r["lse"], d["do"], dq=r["dq"], dk=r["dk"],
                                dv=r["dv"], dgate=r["dgate"])
            ev["comp"][i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev["comp"][i])
                for k in (() if args.forward_only else ("dq", "dk", "dv")):
                    part(host_out[k], k, c).copy_(r[k], non_blocking=True)
                ev["out"][i].record(s_out)
        stream.wait_event(ev["out"][units - 1])              # the timed region ends when the last result is on the host

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    attn.check_status()
    nnz_total = int(attn.map_views()[0][..., -1].sum().item())
    if wl.text_len:
        # block pairs the fine kernels compute with text tokens: every video row also keeps the text blocks, text rows keep all
        tb = -(-wl.text_len // 64)
        nnz_total += wl.batch * wl.heads_q * (wl.n_cubes * tb + tb * (wl.n_cubes + tb))

    # per-kernel events: one (start, stop) pair per kernel group and step
    nk = len(vb.KERNELS)
    evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nk)]
           for _ in range(args.steps)]
    for per_step in evs:
        for a, b in per_step:
            a.record(); b.record()
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    launches0 = vb.vsa2_launch_count()
    barrier()
    if rank == 0:
        sampler.start()
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for s in range(args.steps):
        for kid in range(nk):
            vb.vsa2_profile_events(kid, *evs[s][kid])
        step()
    t_stop.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    for kid in range(nk):
        vb.vsa2_profile_events(kid, None, None)
    launches = vb.vsa2_launch_count() - launches0
    ms_total = t_start.elapsed_time(t_stop)
    kernel_ms = {name: float(np.mean([evs[s][kid][0].elapsed_time(evs[s][kid][1]) for s in range(args.steps)]))
                 for kid, name in enumerate(vb.KERNELS)}
    attn.check_status()

    # end to end: host buffers in, results back to the host, copies inside the timed region
    ms_e2e = float("nan")
    if not args.no_e2e:
        run_e2e(2)
        barrier()
        e_start, e_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e_start.record()
        run_e2e(args.steps)
        e_stop.record()
        barrier()
        ms_e2e = e_start.elapsed_time(e_stop)

    ms_total, ms_e2e = replicas.max_over_ranks([ms_total, ms_e2e], device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    flops = flop_counts(wl, nnz_total)
    if args.forward_only:
        flops["dense_equiv_fwd_bwd"] = flops["dense_equiv_fwd"]
        flops["fine_bwd_dq_executed"] = flops["fine_bwd_dkv_executed"] = 0.0
    ms_step = ms_total / args.steps
    ms_step_e2e = ms_e2e / args.steps
    value = replicas.whole_job_throughput(flops["dense_equiv_fwd_bwd"], world, ms_step * 1e-3) / 1e12
    value_e2e = replicas.whole_job_throughput(flops["dense_equiv_fwd_bwd"], world, ms_step_e2e * 1e-3) / 1e12
    pk, pk_kind = peaks()
    executed = flops["fine_fwd"] + flops["fine_bwd_dq_executed"] + flops["fine_bwd_dkv_executed"] + 2 * flops["router_per_pass"]
    kernel_flops = {"fine_fwd": flops["fine_fwd"], "fine_bwd_dq": flops["fine_bwd_dq_executed"],
                    "fine_bwd_dkv": flops["fine_bwd_dkv_executed"], "router_lse": flops["router_per_pass"],
                    "router_pool": flops["router_per_pass"]}
    tensor_kernels = {k: kernel_ms[k] for k in kernel_flops}
    dominant = max(tensor_kernels, key=tensor_kernels.get)
    peak_tf = pk["bf16_tflops_sustained"]
    achieved = kernel_flops[dominant] / (kernel_ms[dominant] * 1e-3) / 1e12
    roofline = {"kernel": dominant, "bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": achieved / peak_tf,
                "traffic": NCU_TRAFFIC_BYTES_720P_TOP64.get(dominant) if (args.config == 3 and not (args.heads or args.topk or args.grid or args.cube)) else None,
                "peak_kind": pk_kind + " sustained bf16",
                "flops_per_launch": kernel_flops[dominant], "ms_per_launch": kernel_ms[dominant],
                "limiter_ncu": NCU_LIMITER.get(dominant) if wl.cube[0] * wl.cube[1] * wl.cube[2] == 64 else None}
    fine_fwd_tf = flops["fine_fwd"] / (kernel_ms["fine_fwd"] * 1e-3) / 1e12
    # operand bytes the fine forward has to bring into shared memory: a K and a V tile per selected (query block, KV block)
    # pair and a Q tile per query block, in bf16 -- none of it can be reused between the query blocks of a head, whose
    # lists differ, so this is the kernel's compulsory L2 -> SM traffic
    blk = 64
    q_rows = 128 if (wl.cube[0] * wl.cube[1] * wl.cube[2] == 128 or (args.flags & 256)) else 64   # query rows that share a K / V tile
    fwd_tile_bytes = nnz_total * 2 * blk * wl.head_dim * 2 * blk // q_rows
    fwd_l2_tbs = fwd_tile_bytes / (kernel_ms["fine_fwd"] * 1e-3) / 1e12
    bytes_in = sum(host[k].numel() * host[k].element_size() for k in host)
    bytes_out = sum(t.numel() * t.element_size() for k, t in host_out.items() if k == "o" or not args.forward_only)

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        hd = {k: data[k][0, 0] for k in ("q", "k", "v", "do", "gate")}
        if "budgets" in data:
            hd["budgets"] = data["budgets"][0, 0]
        r = oracle_sample_step(wl, hd, args.ref_rows)
        cpu_baseline = {"value": flops["dense_equiv_fwd_bwd"] / r["t_step_extrapolated_s"] / 1e12, "unit": UNIT,
                        "cores": cpu_cores(), "kind": "oracle", "how": ORACLE_HOW,
                        "sample": (f"head 0 of {wl.heads_q}: full routing + coarse branch + fine fwd/bwd over {r['rows']} of "
                                   f"{wl.n_cubes} query blocks ({r['pairs_sample']} of {r['pairs_head']} pairs), "
                                   f"{r['measured_s']:.1f} s measured, extrapolated to the whole step "
                                   f"({r['t_step_extrapolated_s']:.0f} s)")}

    gate_info = None
    if args.gate_hidden:
        # context only: the projection that produces the gate (Eq. 13) and its backward, device-resident operands
        hid = args.gate_hidden
        gx = torch.randn(wl.batch, wl.L, hid, device="cuda").to(torch.bfloat16)
        gw = (torch.randn(hid, wl.heads_q, device="cuda") / hid ** 0.5).to(torch.bfloat16)
        gg = torch.empty(wl.batch, wl.heads_q, wl.L, dtype=torch.float32, device="cuda")
        gdw = torch.empty(hid, wl.heads_q, dtype=torch.float32, device="cuda")
        gdx = torch.empty_like(gx)
        gws = torch.empty(max(256, vb.vsa2_gate_bwd_workspace_bytes(p, hid)), dtype=torch.uint8, device="cuda")
        times = []
        for fn in (lambda: vb.vsa2_gate_fwd(p, hid, gx, gw, gg),
                   lambda: vb.vsa2_gate_bwd(p, hid, gx, gw, gg, dgate, gdw, gdx, gws)):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(5):
                fn()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) / 5)
        xbytes = gx.numel() * 2
        gate_info = {"hidden": hid, "fwd_ms": times[0], "bwd_ms": times[1], "x_bytes": xbytes,
                     "fwd_gbs": xbytes / times[0] / 1e6, "bwd_gbs": 2 * xbytes / times[1] / 1e6}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": config_dict(wl, args.forward_only),
        "run": {"selected_pairs": nnz_total, "replicas": world, "input_gen_s": round(t_gen, 1)},
        "clocks": clocks,
        "e2e": {"value": value_e2e, "unit": UNIT, "ms_per_step": ms_step_e2e, "h2d_bytes_per_step": bytes_in,
                "d2h_bytes_per_step": bytes_out,
                "how": "pinned host -> device copies of Q,K,V,dO,gate and device -> host copies of O,dQ,dK,dV of every step inside "
                       f"the timed region, on side streams, each step cut into {chunks} head chunk(s): the next chunk's inputs load "
                       "and the previous chunk's results drain while a chunk computes"},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "actual_tflops": executed / (ms_step * 1e-3) / 1e12 * world,
        "fine_fwd": {"ms": kernel_ms["fine_fwd"], "tflops": fine_fwd_tf, "frac_of_sustained_peak": fine_fwd_tf / peak_tf,
                     "frac_of_burst_peak": fine_fwd_tf / pk["bf16_tflops"], "frac_of_nominal_2250": fine_fwd_tf / 2250.0,
                     "l2_to_sm": {"bytes_per_launch": fwd_tile_bytes, "achieved_tbs": fwd_l2_tbs, "peak_tbs": NCU_L2_TO_SM_PEAK_TBS,
                                  "frac": fwd_l2_tbs / NCU_L2_TO_SM_PEAK_TBS,
                                  "what": "K and V tiles of every selected block pair (64 FLOP per byte at D = 128 with 64 query rows per tile); "
                                          "peak = the sustained L2 -> SM rate ncu reports (at the profiled clock, so a run at a higher "
                                          "clock can read above 1); with 64-token cubes this rate, not the tensor pipe, bounds the kernel"}},
        "kernel_ms": kernel_ms,
        "gate": gate_info,
        "paper_context": "paper reports 8.9x attention speed-up over FlashAttention-3 on one H800 at 220K tokens (not comparable)",
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="index into the five baseline configurations (3 = 720p top-64)")
    ap.add_argument("--ref-rows", type=int, default=1440, help="query blocks the CPU oracle computes in its sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gate-hidden", type=int, default=0,
                    help="also time the gate projection tanh(X W_g) and its backward for this hidden width (context: 'gate' key)")
    ap.add_argument("--flags", type=int, default=0, help="VSA2_FLAG_* bits passed to the library (kernel variants)")
    ap.add_argument("--e2e-chunks", type=int, default=8, help="upper limit of head chunks per step in the end-to-end pipeline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end loop (profiling runs)")
    ap.add_argument("--topk", type=int, default=0, help="override the TopK of the configuration (context rows: top-128)")
    ap.add_argument("--forward-only", action="store_true", help="route + forward only (context rows: inference)")
    triple = lambda t: tuple(int(x) for x in t.split(","))
    ap.add_argument("--grid", type=triple, default=None, help="override the latent grid T,H,W (context rows: the paper's 61,45,80)")
    ap.add_argument("--cube", type=triple, default=None, help="override the cube, e.g. 4,4,8 (128 tokens; context rows)")
    ap.add_argument("--heads", type=int, default=0, help="override the number of heads (small cases for ncu captures)")
    ap.add_argument("--text-len", type=int, default=0,
                    help="text tokens appended to every head (context rows: joint video + text attention)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    # `python bench.py --gpus N` without a launcher starts its own N ranks (one per GPU); under torchrun it is one of them
    from paper_2609_32882_b200 import replicas
    cmd = replicas.launcher_command(args.gpus, os.path.abspath(__file__), sys.argv[1:], os.environ)
    if cmd is not None:
        raise SystemExit(subprocess.call(cmd))
    run_ours(args)


if __name__ == "__main__":
    main()
