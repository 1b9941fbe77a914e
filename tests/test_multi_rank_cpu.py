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


def test_launcher_arguments():
    """`bench.py --gpus N` started without a launcher re-runs itself under torch.distributed.run with N ranks; under a
    launcher it is a rank and only checks the world size."""
    import sys
    import pytest
    argv = ["--gpus", "4", "--steps", "2", "--warmup", "3"]
    cmd = replicas.launcher_command(4, "bench.py", argv, env={}, port=29999)
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29999"
    assert cmd[-7:] == ["bench.py"] + argv
    assert replicas.launcher_command(1, "bench.py", ["--gpus", "1"], env={}) is None
    assert replicas.launcher_command(4, "bench.py", argv, env={"WORLD_SIZE": "4", "RANK": "2"}) is None
    with pytest.raises(SystemExit):
        replicas.launcher_command(4, "bench.py", argv, env={"WORLD_SIZE": "2"})
    assert 1024 < replicas.free_port() < 65536


def _launched_rank_main():
    """Body of the script the launcher test runs under torch.distributed.run (gloo, CPU)."""
    import torch.distributed as d
    d.init_process_group("gloo")
    mx = replicas.max_over_ranks([float(d.get_rank())])
    if d.get_rank() == 0:
        print(f"LAUNCHED world={d.get_world_size()} max={mx[0]}", flush=True)
    d.destroy_process_group()


def test_launcher_command_starts_the_ranks(tmp_path):
    """The command line the launcher builds really starts two ranks that find each other (gloo on CPU)."""
    import subprocess
    import sys
    script = tmp_path / "ranks.py"
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script.write_text(f"import sys\nsys.path.insert(0, {root!r})\nsys.path.insert(0, {os.path.join(root, 'tests')!r})\n"
                      "import test_multi_rank_cpu as t\nt._launched_rank_main()\n")
    cmd = replicas.launcher_command(2, str(script), [], env={})
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "LAUNCHED world=2 max=1.0" in out.stdout
