"""The N > 1 path on CPU: two gloo ranks exercise the token sharding, the per-rank seeding of
the synthetic tokens and the max-over-ranks timing reduction that bench.py uses."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_18663_b200 import dist as D
from paper_2505_18663_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, M, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = D.shard_tokens(M, rank, world)
        ranges = [None] * world
        dist.all_gather_object(ranges, (lo, hi))
        elapsed = D.max_over_ranks(10.0 + 5.0 * rank, dist)
        x = W.make_activations(W.WORKLOADS["tiny"], 256, M=8, salt=rank)
        sums = [None] * world
        dist.all_gather_object(sums, float(x.float().sum()))
        dist.barrier()
        if rank == 0:
            out.put({"ranges": ranges, "elapsed": elapsed, "sums": sums,
                     "rate": D.aggregate_rate(100.0, elapsed, world)})
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_tokens_and_reduce_timings():
    world, M = 2, 32760
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, M, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (a0, a1), (b0, b1) = res["ranges"]
    assert a0 == 0 and a1 == b0 and b1 == M and a1 % 128 == 0     # disjoint cover, tile-aligned cut
    assert abs((a1 - a0) - (b1 - b0)) <= 128
    assert res["elapsed"] == 15.0                                  # the slowest rank's time
    assert res["rate"] == 2 * 100.0 / 15.0e-3
    assert res["sums"][0] != res["sums"][1]                        # every rank draws its own tokens


def test_shard_tokens_edge_cases():
    assert D.shard_tokens(0, 0, 4) == (0, 0)
    assert D.shard_tokens(100, 0, 4) == (0, 100) and D.shard_tokens(100, 3, 4) == (100, 100)
    cover = [D.shard_tokens(118800, r, 8) for r in range(8)]
    assert cover[0][0] == 0 and cover[-1][1] == 118800
    assert all(cover[i][1] == cover[i + 1][0] for i in range(7))
    assert D.max_over_ranks(3.5) == 3.5
