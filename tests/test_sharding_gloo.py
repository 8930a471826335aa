"""The N > 1 path on CPU: two gloo ranks shard requests and reduce their measurements."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_19830_b200 import sharding as S


def test_shard_requests_is_a_balanced_partition():
    for n in (0, 1, 5, 16, 17):
        for world in (1, 2, 3, 8):
            parts = S.shard_requests(n, world)
            assert parts[0][0] == 0 and parts[-1][1] == n
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in parts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        S.shard_requests(4, 0)


def test_rank_seeds_differ():
    assert len({S.rank_seed(20250621, r) for r in range(8)}) == 8


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        begin, end = S.shard_requests(5, world)[rank]
        tokens = 16.0 * (end - begin)          # every request verifies 16 draft tokens
        ms = 0.25 if rank == 0 else 0.40       # rank 1 is the slow one
        ms_max, total = S.reduce_measurement(ms, tokens)
        out.put((rank, begin, end, ms_max, total, S.job_throughput(ms_max, total)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_to_the_slowest_time_and_the_total_work():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [(r[1], r[2]) for r in res] == [(0, 3), (3, 5)]
    for r in res:
        assert r[3] == pytest.approx(0.40)
        assert r[4] == pytest.approx(80.0)
        assert r[5] == pytest.approx(80.0 / 0.40e-3)


def test_reduce_without_a_process_group_is_the_identity():
    assert S.reduce_measurement(1.5, 7.0) == (1.5, 7.0)
