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


def _bench_worker(rank, world, port, out):
    """The rank set-up and the timing reduction of bench.py itself under gloo; only the kernels are stubbed out."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2604_26209_b200.dist import reduce_timing
    dist.init_process_group("gloo", rank=rank, world_size=world)
    s, mine = bench.rank_structure("main_p3", world, rank)
    n_blocks = bench.agree_block_count(10.0 * (rank + 1), 100.0, lambda x: reduce_timing([x], 0)[0][0])
    blocks = [1.0 + rank + 0.1 * i for i in range(n_blocks)]          # pretend block times, rank 1 slower
    head, tokens = reduce_timing(blocks, s.n_active)
    out.put((rank, list(mine), s.n_prompts, s.n_active, n_blocks, head, tokens, int(s.slot_depth[:8].sum())))
    dist.destroy_process_group()


def test_bench_rank_setup_and_block_reduction_two_ranks():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_bench_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the global list has world x 3 prompts; contiguous disjoint shards of 3 prompts each
    assert res[0][1] == [0, 1, 2] and res[1][1] == [3, 4, 5]
    assert all(r[2] == 3 and r[3] == 3 * 96 for r in res)
    assert res[0][7] != res[1][7]                              # different prompts: different drawn depths
    # every rank times the same number of blocks (the slower rank's first block decides: 100 ms / 20 ms)
    assert res[0][4] == res[1][4] == 5
    for r in res:
        assert r[6] == 2 * 3 * 96                              # rows of all ranks
        assert np.allclose(r[5], [2.0 + 0.1 * i for i in range(5)])   # block-wise max over ranks


def test_rank_zero_of_one_is_the_single_gpu_workload():
    import bench
    s, mine = bench.rank_structure("main", 1, 0)
    ref = synth.config_main(n_prompts=64, seed=0)
    assert list(mine) == list(range(64)) and np.array_equal(s.slot_depth, ref.slot_depth)


def test_single_process_is_identity():
    value, tmax, total = aggregate_throughput([50.0], 6144, steps=5)
    assert tmax == [50.0] and total == 6144 and np.isclose(value, 6144 * 5 / 0.05)
