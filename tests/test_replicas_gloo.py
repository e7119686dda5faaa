"""The multi-GPU form of the path is independent replicas; its host logic under a 2-process gloo group."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_18362_b200 import replicas


def test_sharding_covers_every_sequence_once():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                part = list(replicas.shard_sequences(n, world, r))
                assert part == sorted(part)
                seen += part
            assert seen == list(range(n))
            sizes = [len(replicas.shard_sequences(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.shard_sequences(4, 2, 2)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = replicas.shard_sequences(9, world, rank)
        ms = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
        dist.barrier()
        slowest = replicas.max_over_ranks(ms, dist)
        counts = torch.tensor([len(mine)], dtype=torch.int64)
        dist.all_reduce(counts)
        out.put((rank, slowest, int(counts.item()), replicas.job_throughput(3, world, 4, slowest)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_replicas_agree_on_the_slowest_time():
    world, port = 2, 29511 + os.getpid() % 1000
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, total, thr in res:
        assert slowest == 15.0 and total == 9
        assert abs(thr - 2 * 3 * 4 / 15e-3) < 1e-6
    assert replicas.max_over_ranks(3.5) == 3.5     # single process: identity
