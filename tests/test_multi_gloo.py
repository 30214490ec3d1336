"""The N > 1 path on CPU: two gloo ranks shard independent units with no overlap and agree on the
max-over-ranks time (the only exchanges the data-parallel use of the path needs)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1805_11046_b200.dist import max_over_ranks, shard_units, sum_over_ranks


def test_shards_partition_the_units():
    for total in (0, 1, 7, 256, 257):
        for world in (1, 2, 3, 8):
            spans = [shard_units(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b, e = shard_units(257, rank, world)
        slowest = max_over_ranks(10.0 + rank, world)
        total = sum_over_ranks(float(e - b), world)
        out.put((rank, b, e, slowest, total))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree():
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
    assert [r[1:3] for r in res] == [(0, 129), (129, 257)]
    assert all(r[3] == 11.0 and r[4] == 257.0 for r in res)
