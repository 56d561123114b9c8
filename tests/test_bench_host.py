"""Host logic of the benchmark on more than one rank: world_size-2 gloo processes on the CPU."""
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        # device-measured durations are reduced with MAX, counters with SUM
        t = bench.reduce_max_time(10.0 + 5.0 * rank, world)
        sums = bench.reduce_sum([1.0 + rank, 100.0 * (rank + 1)], world)
        seeds = [bench.rank_seed(7, rank, s) for s in range(3)]
        info = bench.shard_info(world, 256)
        q.put((rank, t, sums, seeds, info))
    finally:
        dist.barrier()
        dist.destroy_process_group()


def test_two_ranks_reduce_and_shard():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in ps:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, s0, seeds0, i0), (r1, t1, s1, seeds1, i1) = got
    assert t0 == t1 == 15.0                              # max over ranks
    assert s0 == s1 == [3.0, 300.0]                      # sum over ranks
    assert not set(seeds0) & set(seeds1)                 # every rank samples different chunks
    assert i0 == i1 == dict(envs_per_rank=256, envs_total=512, scaling="weak")


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_time(3.5, 1) == 3.5
    assert bench.reduce_sum([1, 2], 1) == [1, 2]


def test_reference_arm_other_ranks_do_no_work(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    args = type("A", (), dict(workload="toy_mlp", batch=0, warmup=0, steps=1))()
    bench.run_reference(args)
    assert capsys.readouterr().out == ""
