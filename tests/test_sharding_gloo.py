"""The multi-rank host logic on CPU: two gloo ranks shard a batch, time a step, reduce the max."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2503_10501_b200 import sharding


def test_split_batch_covers_everything_once():
    for total, world in [(64, 1), (64, 2), (64, 8), (10, 4), (3, 8), (0, 2)]:
        parts = sharding.split_batch(total, world)
        assert len(parts) == world
        flat = [i for b, e in parts for i in range(b, e)]
        assert flat == list(range(total))
        sizes = [e - b for b, e in parts]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.image_range(2, 2, 4)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = list(sharding.image_range(rank, world, 5))
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    dist.barrier()
    slowest = sharding.max_over_ranks(10.0 + rank)       # rank 1 is "slower"
    total = torch.tensor([len(mine)], dtype=torch.int64)
    dist.all_reduce(total)
    q.put((rank, gathered, slowest, int(total.item())))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, gathered, slowest, total in results:
        assert gathered == [[0, 1, 2, 3, 4], [5, 6, 7, 8, 9]]     # disjoint, complete, ordered
        assert slowest == 11.0                                     # max over ranks, on every rank
        assert total == 10                                         # whole-job unit count
