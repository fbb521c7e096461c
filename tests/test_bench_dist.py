"""The bench's cross-rank reduction (sum of tokens, max of time) on two gloo ranks. CPU only."""
from __future__ import annotations

import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    tok, ms = bench.reduce_over_ranks(100 + rank, 5.0 + 2.0 * rank, world)
    q.put((rank, tok, ms, bench.dist_env()[0]))
    dist.barrier()
    dist.destroy_process_group()


def test_reduce_over_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1] and [g[3] for g in got] == [0, 1]
    for _, tok, ms, _ in got:
        assert tok == 201 and ms == 7.0


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(17, 3.5, 1) == (17, 3.5)


def _keys_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import torch
    from paper_2512_18337_b200.parallel import reduce_argmax_keys, shard_bounds
    rows = 5
    # rank r holds the largest word of rows r, r+2, ...; the last element plays the status word
    keys = torch.tensor([(10 + i) * (1 << 32) + 7 if i % world == rank else (1 + rank) * (1 << 32) + i
                         for i in range(rows)] + [rank + 1], dtype=torch.int64)
    reduce_argmax_keys(keys, rows)
    q.put((rank, keys.tolist(), shard_bounds(151936, rank, world), shard_bounds(10, rank, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_vocab_shard_words_are_max_reduced_over_two_ranks():
    """Host-side plumbing of the vocabulary-parallel verification: one MAX all-reduce over the packed
    per-row words (status word untouched), and shard bounds that tile the vocabulary."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_keys_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = [(10 + i) * (1 << 32) + 7 for i in range(5)]
    for rank, keys, big, small in got:
        assert keys[:5] == want and keys[5] == rank + 1
    assert [g[2] for g in got] == [(0, 75968), (75968, 151936)]
    assert [g[3] for g in got] == [(0, 8), (8, 10)]
