"""The N > 1 path on CPU: two gloo ranks shard a batch, 'measure' different times and aggregate.

The data path has no collective (sequences are independent), so what runs across ranks is only
this host logic: the shard of each rank, the maximum of the times, the sum of the units.
"""
import os
import socket

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_13797_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shard = sharding.shard_range(129, world, rank)          # ragged: 129 sequences over 2 ranks
        ms_local = [10.0 + 3.0 * rank, 7.0 - rank]              # two timed passes, rank-dependent
        ms = sharding.max_over_ranks(ms_local)
        units = sharding.sum_over_ranks([len(shard) * 5])       # 5 steps of the shard
        dist.barrier()
        q.put((rank, list(shard), ms, units, sharding.rank_seed_offset(11, rank)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_aggregate():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    shards = [g[1] for g in got]
    assert sorted(shards[0] + shards[1]) == list(range(129))               # disjoint and complete
    assert abs(len(shards[0]) - len(shards[1])) <= 1
    for _, _, ms, units, _ in got:
        assert ms == [13.0, 7.0]                                           # slowest rank per pass
        assert units == [129 * 5.0]
        assert sharding.job_throughput(units[0], ms[0]) == pytest.approx(129 * 5 / 13e-3)
    assert [g[4] for g in got] == [11, 12]                                  # every rank its own inputs


def test_single_process_is_identity():
    assert sharding.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert sharding.sum_over_ranks([3]) == [3.0]
    assert list(sharding.shard_range(10, 1, 0)) == list(range(10))
    assert [len(sharding.shard_range(10, 4, r)) for r in range(4)] == [3, 3, 2, 2]
    with pytest.raises(ValueError):
        sharding.shard_range(10, 2, 2)
