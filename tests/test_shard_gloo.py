"""The multi-GPU host logic (sharding of independent problems, barrier + max-over-ranks timing)
exercised with world_size 2 on CPU over gloo."""
import os
import socket

import pytest
import torch.multiprocessing as mp

from paper_2010_15884_b200 import shard


def test_split_range_covers_disjointly():
    for total in (0, 1, 7, 16, 17):
        for world in (1, 2, 3, 8):
            parts = [shard.split_range(total, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == total
            for a, b in zip(parts, parts[1:]):
                assert a[1] == b[0]
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1
    assert shard.split_range(16, 3, 8) == (6, 8)          # configuration 5: 16 images on 8 GPUs
    with pytest.raises(ValueError):
        shard.split_range(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = shard.split_range(16, rank, world)
        shard.barrier(world)
        slow = shard.max_over_ranks(1.0 + rank, world)            # rank 1 is the slow one
        total = shard.sum_over_ranks(hi - lo, world)
        thr = shard.aggregate_throughput(100.0 * (hi - lo), 1.0 + rank, world)
        out.put((rank, lo, hi, slow, total, thr))
    finally:
        dist.destroy_process_group()


def test_world_size_two_over_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1:3] for g in got] == [(0, 8), (8, 16)]
    for g in got:
        assert g[3] == 2.0                 # slowest rank's time on every rank
        assert g[4] == 16.0                # all items accounted for
        assert g[5] == pytest.approx(1600.0 / 2.0)


def test_single_rank_needs_no_process_group():
    shard.barrier(1)
    assert shard.max_over_ranks(3.5, 1) == 3.5
    assert shard.aggregate_throughput(10.0, 2.0, 1) == 5.0
