"""bench.py --gpus N runs N independent replicas (the path has no exchange step); the only thing
the ranks share is the reduction of their timings and counts.  That reduction is covered here
with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    times, counts = bench.reduce_over_ranks([10.0 + rank, 5.0 - rank, 1.0], [256.0 * (rank + 1), 100.0], "cpu", world)
    out.put((rank, times, counts))
    dist.barrier()
    dist.destroy_process_group()


def test_reduce_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, counts in got:
        assert times == [11.0, 5.0, 1.0]          # MAX over ranks: the job is as slow as its slowest replica
        assert counts == [768.0, 200.0]           # SUM over ranks: whole-job tokens and launches


def test_reduce_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([1.5, 2.5], [3.0], "cpu", 1) == ([1.5, 2.5], [3.0])
