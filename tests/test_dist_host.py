"""Multi-process host logic of the multi-GPU path, on CPU with the gloo backend (world size 2)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_16515_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 1.0 + rank                       # rank 1 is the slow one
        ups, ms = dist_util.aggregate_throughput(100.0, local_ms)
        mine = dist_util.shard_heads(2, 3, world, rank)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        out.put((rank, ups, ms, gathered))
    finally:
        dist.destroy_process_group()


def test_weak_scaling_aggregation_and_head_sharding_two_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ups, ms, gathered in results:
        assert ms == 2.0                                       # the slowest rank sets the time
        assert abs(ups - 100.0 * 2 / 2e-3) < 1e-6              # both ranks' units over that time
        owned = [x for part in gathered for x in part]
        assert sorted(owned) == [(b, h) for b in range(2) for h in range(3)]   # a partition
        assert abs(len(gathered[0]) - len(gathered[1])) <= 1


def test_single_process_is_identity():
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.shard_heads(1, 4, 1, 0) == [(0, 0), (0, 1), (0, 2), (0, 3)]
    ups, ms = dist_util.aggregate_throughput(10.0, 5.0)
    assert ms == 5.0 and abs(ups - 2000.0) < 1e-9
