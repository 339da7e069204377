"""Multi-GPU host logic on CPU: (batch, head) units are split over ranks with no data-path
collective; the only communication is the max / sum of scalars.  Two gloo ranks."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2302_00787_b200 import sharding


def test_unit_partition_is_a_disjoint_cover():
    for n in (0, 1, 7, 48, 64):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(sharding.unit_partition(n, r, world))
            assert seen == list(range(n))
            sizes = [len(sharding.unit_partition(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.unit_partition(4, 2, 2)
    assert sharding.rank_seed(2000, 0) == 2000 and sharding.rank_seed(2000, 1) != 2000


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, lr, w = sharding.env_rank_world()
    import bench                                  # the benchmark's own rank set-up, as torchrun would start it
    assert bench.rank_setup(2) == (r, lr, w) == (rank, rank, world)

    class A:
        gpus, impl = 2, "native"
    assert bench.relaunch_if_needed(A) is False   # already under a launcher: no second one is started
    units = sharding.unit_partition(48, r, w)
    # each rank "times" its own share; the job's time is the slowest rank, its work the sum
    t = sharding.max_over_ranks(1.0 + 0.5 * r)
    n = sharding.sum_over_ranks(float(len(units)))
    dist.barrier()
    out.put((r, list(units), t, n))
    dist.destroy_process_group()


def test_two_gloo_ranks_share_units_and_reduce_time():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] + res[1][1] == list(range(48))
    assert all(abs(t - 1.5) < 1e-12 and n == 48.0 for _, _, t, n in res)


def test_bench_starts_its_own_ranks_only_when_asked(monkeypatch):
    """`python bench.py --gpus N` outside a launcher re-executes itself under torch.distributed.run with N
    ranks on 127.0.0.1; with one GPU, under a launcher, or for the CPU reference arm it does not."""
    import bench

    class A:
        gpus, impl = 1, "native"
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    assert bench.relaunch_if_needed(A) is False
    A.gpus, A.impl = 4, "reference"
    assert bench.relaunch_if_needed(A) is False
    A.impl = "native"
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    with pytest.raises(SystemExit):
        bench.relaunch_if_needed(A)
    cmd = seen["cmd"]
    assert "torch.distributed.run" in cmd and "--nproc-per-node=4" in cmd and "127.0.0.1" in cmd
    assert bench.rank_setup(1) == (0, 0, 1)
