"""World-size-2 gloo test of the replica logic used by `bench.py --gpus N` (runs on CPU)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_32882_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        times = [10.0 + rank, 5.0 - rank]                    # rank 1 is slower on the first, faster on the second
        mx = replicas.max_over_ranks(times)
        seed = replicas.replica_seed(3, rank)
        shard = replicas.head_shard(10, 4, rank, world)
        dist.barrier()
        out.put((rank, mx, seed, shard))
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_take_disjoint_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, mx0, s0, sh0), (r1, mx1, s1, sh1) = res
    assert mx0 == mx1 == [11.0, 5.0]
    assert s0 != s1
    # head shards: disjoint, cover all 10 KV heads, GQA groups intact
    assert sh0[0] == 0 and sh0[1] + sh1[1] == 10 and sh1[0] == sh0[1]
    assert sh0[3] == 4 * sh0[1] and sh1[2] == 4 * sh1[0]
    assert replicas.whole_job_throughput(100.0, 2, 11.0) == 200.0 / 11.0


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.head_shard(3, 4, 0, 1) == (0, 3, 0, 12)
