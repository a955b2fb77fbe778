"""The multi-GPU host logic on two CPU ranks (gloo): unit partition, max-over-ranks step time, gradient sums."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_20586_b200 import shard


def test_shard_units_cover_every_unit_exactly_once():
    for total in (0, 1, 7, 128, 1024):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                s, c = shard.shard_units(total, world, r)
                seen += list(range(s, s + c))
            assert seen == list(range(total))
            counts = [shard.shard_units(total, world, r)[1] for r in range(world)]
            assert max(counts) - min(counts) <= 1
    with pytest.raises(ValueError):
        shard.shard_units(4, 2, 2)


def test_shard_batch_heads_slices():
    B, H = 3, 5
    for world in (1, 2, 4):
        units = []
        for r in range(world):
            for b, h, n in shard.shard_batch_heads(B, H, world, r):
                assert 0 <= b < B and 0 <= h and h + n <= H and n > 0
                units += [b * H + h + i for i in range(n)]
        assert units == list(range(B * H))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        step_ms = shard.max_over_ranks(10.0 + 5.0 * rank, dist)           # rank 1 is the slow one
        g = torch.full((2, 4, 3), float(rank + 1))
        shard.sum_over_ranks(g, dist)
        start, count = shard.shard_units(9, world, rank)
        t = torch.zeros(9)
        t[start:start + count] = 1.0
        shard.sum_over_ranks(t, dist)                                       # every unit claimed exactly once
        out[rank] = (step_ms, float(g[0, 0, 0]), t.tolist(), shard.job_throughput(100.0, world, step_ms))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_job_numbers():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for r in (0, 1):
        step_ms, g, claimed, rate = res[r]
        assert step_ms == 15.0                       # max over ranks, same on both
        assert g == 3.0                              # 1 + 2
        assert claimed == [1.0] * 9
        assert abs(rate - 2 * 100.0 / 15e-3) < 1e-6


def test_no_process_group_is_the_identity():
    assert shard.max_over_ranks(3.5) == 3.5
    t = torch.ones(3)
    assert shard.sum_over_ranks(t) is t
