"""Multi-rank host logic on CPU: two gloo ranks, sequence sharding and max-over-ranks timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_16994_b200 import shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shard.barrier(world)
        slow = shard.max_over_ranks(10.0 + 5.0 * rank, world)
        seqs = shard.shard_sequences(7, rank, world)
        local = torch.tensor(list(seqs), dtype=torch.int32)
        pad = torch.full((4,), -1, dtype=torch.int32)
        pad[:local.numel()] = local
        allr = shard.gather_results(pad, world)
        q.put((rank, slow, list(seqs), allr.tolist(), shard.rank_seeds(rank, world, 3)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_and_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]                 # the slowest rank sets the time
    assert got[0][2] == [0, 1, 2, 3] and got[1][2] == [4, 5, 6]  # disjoint cover of the batch
    assert got[0][3] == got[1][3] == [0, 1, 2, 3, 4, 5, 6, -1]
    assert not set(got[0][4]) & set(got[1][4])


def test_shard_sequences_covers_everything():
    for total in (0, 1, 5, 8, 13):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(shard.shard_sequences(total, r, world))
            assert seen == list(range(total))
