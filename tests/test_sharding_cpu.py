"""Multi-rank host logic on CPU (gloo, world size 2): unit partition, max-over-ranks timing and the
whole-job rate bench.py reports for N > 1.  No GPU and no collective on the data path."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2411_17178_b200 import sharding


def test_split_units_partitions_exactly():
    for n in (0, 1, 7, 128, 288, 1920):
        for world in (1, 2, 3, 4, 8):
            ranges = [sharding.split_units(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a0, a1), (b0, b1) in zip(ranges[:-1], ranges[1:]):
                assert a1 == b0
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.split_units(4, 2, 2)


def test_single_process_is_identity():
    assert sharding.max_over_ranks([1.5, 2.0]) == [1.5, 2.0]
    assert sharding.whole_job_rate(10.0, 1, 1000.0) == 10.0


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, faster on the second
        got = sharding.max_over_ranks(ms)
        begin, end = sharding.split_units(129, world, rank)
        owned = torch.zeros(129, dtype=torch.int64)
        owned[begin:end] = 1
        dist.all_reduce(owned)                           # test-only check that the ranges tile the units once
        rate = sharding.whole_job_rate(2.0e12, world, got[0])
        q.put((rank, got, int(owned.min()), int(owned.max()), rate, sharding.rank_seed(100, rank)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, lo, hi, rate, seed in res:
        assert got == [15.0, 3.0]                        # the job is as slow as its slowest rank
        assert lo == 1 and hi == 1
        assert rate == pytest.approx(2 * 2.0e12 / 15e-3)
    assert res[0][5] != res[1][5]
