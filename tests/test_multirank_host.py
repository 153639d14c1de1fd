"""Two CPU ranks over gloo: the host logic of the multi-GPU run (prompt sharding, timing reduction)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_26209_b200 import synth
from paper_2604_26209_b200.dist import aggregate_throughput


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shard = synth.shard_prompts(13, world, rank)
    s = synth.config_main(n_prompts=len(shard), seed=rank)
    # rank r pretends its 10 steps took (r + 1) * 100 ms
    value, tmax, total = aggregate_throughput([100.0 * (rank + 1), 5.0 + rank], s.n_active, steps=10)
    out.put((rank, list(shard), s.n_active, value, tmax, total))
    dist.destroy_process_group()


def test_two_ranks_shard_prompts_and_reduce_timing():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    shards = [set(r[1]) for r in res]
    assert shards[0].isdisjoint(shards[1]) and shards[0] | shards[1] == set(range(13))
    assert abs(len(shards[0]) - len(shards[1])) <= 1
    tokens = sum(r[2] for r in res)
    assert tokens == 13 * 96
    for r in res:                                   # every rank sees the same aggregate
        assert r[5] == tokens and r[4] == [200.0, 6.0]
        assert np.isclose(r[3], tokens * 10 / 0.2)


def test_single_process_is_identity():
    value, tmax, total = aggregate_throughput([50.0], 6144, steps=5)
    assert tmax == [50.0] and total == 6144 and np.isclose(value, 6144 * 5 / 0.05)
