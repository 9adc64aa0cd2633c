"""Host logic of the multi-GPU path (replicas over query ranges), run as two
gloo ranks on the CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2204_08400_b200 import replicas


def test_shard_ranges_partition_the_queries():
    for n in (0, 1, 7, 64, 65536, 65537):
        for world in (1, 2, 3, 8):
            spans = [replicas.shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            for a, b in zip(spans, spans[1:]):
                assert a[1] == b[0]
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = replicas.shard_range(1001, rank, world)
        ms = replicas.slowest_rank_ms(10.0 + 5.0 * rank)
        total = replicas.total_units(hi - lo)
        out.put((rank, ms, total))
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_slowest_time_and_total_queries():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]       # max over ranks
    assert [r[2] for r in res] == [1001, 1001]       # all ranks' queries


def test_single_process_is_identity():
    assert replicas.slowest_rank_ms(3.5) == 3.5
    assert replicas.total_units(12) == 12
