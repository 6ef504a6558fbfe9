"""Host-side logic of the multi-GPU path on CPU: two gloo ranks shard the queries, gather their
per-query results in query order and agree on the slowest rank's time."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_09135_b200.shard import gather_query_results, max_over_ranks, shard_queries, sum_over_ranks


def test_shards_tile_the_queries():
    for B in (0, 1, 7, 128, 129):
        for world in (1, 2, 3, 8):
            cur = 0
            for r in range(world):
                s, n = shard_queries(B, world, r)
                assert s == cur and n >= 0
                cur += n
            assert cur == B
            sizes = [shard_queries(B, world, r)[1] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_queries(4, 2, 2)


def _worker(rank, world, port, B, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        start, n = shard_queries(B, world, rank)
        local = torch.arange(start, start + n, dtype=torch.int32).unsqueeze(1).repeat(1, 3) * 10 + rank
        full = gather_query_results(local, B)
        slow = max_over_ranks(1.0 + rank)
        total = sum_over_ranks(10.0 + rank)
        q.put((rank, full.tolist(), slow, total))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gather_in_query_order():
    world, B = 2, 7
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, B, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = []
    for r in range(world):
        s0, n = shard_queries(B, world, r)
        want += [[i * 10 + r] * 3 for i in range(s0, s0 + n)]
    for rank, full, slow, total in got:
        assert full == want
        assert slow == 2.0
        assert total == 21.0
