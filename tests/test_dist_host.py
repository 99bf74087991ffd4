"""Multi-process host logic of the multi-GPU path, on CPU with the gloo backend (world size 2)."""
import os
import socket

import numpy as np
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
        # strong scaling by contiguous head ranges: every rank contributes its share of one layer
        h0, h1 = dist_util.head_range(5, world, rank)
        ranges = [None] * world
        dist.all_gather_object(ranges, (h0, h1))
        total = dist_util.sum_over_ranks(float(h1 - h0))
        out.put((rank, ups, ms, gathered, ranges, total))
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
    for rank, ups, ms, gathered, ranges, total in results:
        assert ranges == [(0, 2), (2, 5)] and total == 5.0       # disjoint, in rank order, covering every head
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


def test_head_ranges_partition_and_list_slicing():
    for H in (1, 5, 12, 40):
        for world in (1, 2, 3, 8):
            r = [dist_util.head_range(H, world, k) for k in range(world)]
            assert r[0][0] == 0 and r[-1][1] == H
            assert all(r[k][1] == r[k + 1][0] for k in range(world - 1))
            assert max(b - a for a, b in r) - min(b - a for a, b in r) <= 1
    # per-head lists: the slice of heads [1, 3) of three heads with two query blocks each
    rp = np.array([0, 2, 3, 3, 6, 7, 9], dtype=np.int32)
    ci = np.array([0, 1, 4, 1, 2, 3, 0, 5, 6], dtype=np.int32)
    rp2, ci2 = dist_util.slice_head_lists(rp, ci, 2, 1, 3)
    assert rp2.tolist() == [0, 0, 3, 4, 6] and ci2.tolist() == [1, 2, 3, 0, 5, 6]
    rp_all, ci_all = dist_util.slice_head_lists(rp, ci, 2, 0, 3)
    assert rp_all.tolist() == rp.tolist() and ci_all.tolist() == ci.tolist()


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    # `python bench.py --gpus N` without a launcher re-runs itself under torch's launcher with one rank per
    # GPU; here only the command it would run is checked (no GPU needed)
    import importlib.util
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("salad_bench", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    seen = {}
    real_call, real_argv = bench.subprocess.call, sys.argv
    bench.subprocess.call = lambda cmd: seen.setdefault("cmd", cmd) and 0
    sys.argv = ["bench.py", "--gpus", "4", "--steps", "7", "--shard", "heads"]
    try:
        class A:
            gpus = 4
        assert bench.self_launch(A) == 0
    finally:
        bench.subprocess.call, sys.argv = real_call, real_argv
    cmd = seen["cmd"]
    assert "torch.distributed.run" in cmd and "--nproc-per-node=4" in cmd and "127.0.0.1" in cmd
    assert cmd[-6:] == ["--gpus", "4", "--steps", "7", "--shard", "heads"]
