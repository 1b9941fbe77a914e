"""Host-side logic of the multi-GPU mode: independent replicas, no data-path collective.

Every (batch, query head) of the operator is independent, so N GPUs run N replicas of the single-GPU
library on disjoint work; the only communication is a barrier and a MAX reduction of the measured times.
Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
import socket
import sys

import torch
import torch.distributed as dist


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own synthetic batch."""
    return int(base_seed) + 1000 * int(rank)


def head_shard(n_heads_kv: int, rep: int, rank: int, world: int):
    """KV-head groups owned by `rank` when ONE problem is sharded by head (a GQA group stays on one GPU).
    Returns (first_kv_head, n_kv_heads, first_q_head, n_q_heads)."""
    base, extra = divmod(n_heads_kv, world)
    n = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, n, first * rep, n * rep


def max_over_ranks(values, device="cpu"):
    """Elementwise maximum over ranks of a list of floats (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_throughput(units_per_rank: float, world: int, seconds: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / seconds


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launcher_command(gpus: int, script: str, argv: list, env: dict, port: int | None = None):
    """How `python <script> --gpus N ...` becomes N ranks.

    Under a launcher (WORLD_SIZE is set) the process is one of the ranks: returns None, after checking that the
    launcher's world size is the one asked for.  Started plainly with --gpus N > 1, the script must start its own
    ranks: returns the torch.distributed.run command line (one process per GPU of this node, rendezvous on 127.0.0.1)
    that re-runs the same script with the same arguments.
    """
    world = env.get("WORLD_SIZE")
    if world is not None:
        if int(world) != int(gpus):
            raise SystemExit(f"--gpus {gpus} disagrees with the launcher's WORLD_SIZE={world}")
        return None
    if gpus <= 1:
        return None
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(gpus)}",
            "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script] + list(argv)
