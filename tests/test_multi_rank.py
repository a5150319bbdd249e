"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas of the same workload.

The linears shard across GPUs as independent replicas (no data-path collective); the only exchange is the
reduction of the timing: the slowest rank's time and the sum of the bytes all ranks streamed.
"""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        # rank r took (r + 1) ms for 10 (r + 1) units
        t, u = bench.reduce_max_time_sum_units(1.0 + rank, 10.0 * (rank + 1), world, torch.device("cpu"))
        out.put((rank, t, u))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_max_time_and_sum_units():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, t, u in got:
        assert t == 2.0       # max over ranks
        assert u == 30.0      # 10 + 20
    assert [g[0] for g in got] == [0, 1]


def test_single_rank_is_identity():
    import bench
    assert bench.reduce_max_time_sum_units(3.5, 7.0, 1, None) == (3.5, 7.0)


def test_reference_arm_other_ranks_do_no_work(monkeypatch, capsys):
    """Under a multi-rank launch only rank 0 runs the CPU reference arm; the others return without printing."""
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setenv("LOCAL_RANK", "1")
    assert bench.dist_env() == (1, 1, 2)
    assert bench.run_reference(None) is None
    assert capsys.readouterr().out == ""
