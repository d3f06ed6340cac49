"""The N > 1 path: replicas on token slices, timing by the slowest rank (gloo, 2 processes, CPU)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_02753_b200 import replicas


def test_token_slices_are_disjoint_and_cover_the_batch():
    for n in (0, 1, 7, 8, 64, 8191, 8192):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                start, count = replicas.shard_tokens(n, r, world)
                seen.extend(range(start, start + count))
            assert seen == list(range(n))
            counts = [replicas.shard_tokens(n, r, world)[1] for r in range(world)]
            assert max(counts) - min(counts) <= 1


def test_single_process_aggregate_is_identity():
    assert replicas.aggregate(2.5, 100) == (2.5, 100.0)
    assert replicas.job_throughput(2.0, 100) == pytest.approx(50000.0)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r was slower by r milliseconds and processed its slice of 1001 tokens
        start, count = replicas.shard_tokens(1001, rank, world)
        ms, units = replicas.aggregate(10.0 + rank, count, dist)
        tput = replicas.job_throughput(10.0 + rank, count, dist)
        out.put((rank, ms, units, tput, start, count))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_the_total_tokens():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, units, tput, start, count in results:
        assert ms == 11.0 and units == 1001.0
        assert tput == pytest.approx(1001.0 / 11e-3)
    assert results[0][4:] == (0, 501) and results[1][4:] == (501, 500)
