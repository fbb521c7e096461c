"""Rank body for the launcher test (not a test itself).

Does everything bench.py does around the step - rank discovery, the world-size check, the per-rank plan
(shared corpus, rank-specific stream scripts), the cross-rank reduction and the one JSON line of rank 0 -
over gloo, with the step itself replaced by a host stub that reports a rank-dependent token count and
time.  No automaton, no GPU and no library call is involved."""
from __future__ import annotations

import hashlib
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
import workload as W  # noqa: E402


def main():
    args = bench.parse_args(sys.argv[1:])
    rank, local_rank, world = bench.init_ranks("gloo", args)
    cfg, stream_cfg = bench.plan_rank(args, rank)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(stream_cfg, corpus)
    tokens = cfg.B * args.steps * (rank + 1)          # stub: rank r "commits" r + 1 tokens per stream and step
    ms = 10.0 * (rank + 1)
    all_tokens, max_ms = bench.reduce_over_ranks(tokens, ms, world)
    seeds = bench.gather_over_ranks(stream_cfg.seed, world)
    digests = bench.gather_over_ranks(hashlib.sha1(scripts.tobytes()).hexdigest(), world)
    corpora = bench.gather_over_ranks(hashlib.sha1(corpus.tobytes()).hexdigest(), world)
    locals_ = bench.gather_over_ranks(local_rank, world)
    if rank == 0:
        print(json.dumps(bench.headline(cfg, world, args, all_tokens, max_ms, stub=True, rank_seeds=seeds,
                                        script_digests=digests, corpus_digests=corpora, local_ranks=locals_)))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
