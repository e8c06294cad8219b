"""The multi-GPU mode is N independent replicas; its only host logic (sharding,
barrier, max-over-ranks timing, aggregation) is checked here with two gloo
ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_11816_b200 import replicas as R


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        R.barrier(dist)
        my_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        worst = R.max_over_ranks(my_ms, dist)
        mine = list(R.shard_sequences(7, world, rank))
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        R.barrier(dist)
        out.put((rank, worst, gathered, R.aggregate_tokens_per_s(32, 4, worst, world)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_cover_all_sequences():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, gathered, tps in res:
        assert worst == 15.0
        assert sorted(sum(gathered, [])) == list(range(7))
        assert abs(tps - 2 * 32 * 4 / 15e-3) < 1e-6


def test_single_process_needs_no_process_group():
    assert R.max_over_ranks(3.5) == 3.5
    assert list(R.shard_sequences(5, 1, 0)) == [0, 1, 2, 3, 4]
    assert [len(R.shard_sequences(10, 4, r)) for r in range(4)] == [2, 3, 2, 3]
    assert R.aggregate_tokens_per_s(32, 64, 3000.0, 1) == 32 * 64 / 3.0
