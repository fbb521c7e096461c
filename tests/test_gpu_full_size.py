"""Closed-loop parity at the full sizes of the three large workloads and of the paper's own evaluation shape, tolerance 0.

Same launch configuration as the benchmark (every stream, full vocabulary, the full corpus, the
fused step).  The noise logits are drawn once on the device and copied to the host, so the CPU
oracle and the CUDA path read the same bytes; every output of every stream is compared after
every step.  The number of steps is kept small because the oracle scans up to 10 GB per step."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import paper_2512_18337_b200 as S
import workload as W
from harness.cuda_backend import CudaBackend
from oracle.backend import OracleBackend

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft")


def _full_size_closed_loop(i, steps, variant=0):
    cfg = W.CONFIGS[i].scaled(steps=steps)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    logits, rowmax = W.make_noise_logits_device(cfg, DEV)
    assert logits.shape == (cfg.B * (cfg.K + 1), cfg.vocab)
    host_bits = W.device_bits_to_host(logits)
    gpu = CudaBackend(cfg, corpus, logits)
    S.sam_set_argmax_variant(variant)
    try:
        tr_g = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), gpu, steps)
    finally:
        S.sam_set_argmax_variant(0)
    assert gpu.status() == 0
    del gpu, logits
    torch.cuda.empty_cache()
    cpu = OracleBackend(cfg, corpus, host_bits, oracle.host_threads())
    tr_o = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), cpu, steps)
    for t, (o, g) in enumerate(zip(tr_o, tr_g)):
        for k in KEYS:
            assert (o[k] == g[k]).all(), (cfg.name, t, k)
    st = W.trace_stats(cfg, tr_g)
    # the loop must exercise drafting and both outcomes of verification, not idle at the root
    assert st["nonempty_frac"] > 0.2 and 0.05 < st["shr"] < 0.98, st
    return cfg, tr_g


def test_full_size_cfg2_metric_workload():
    """B=256, K=16, min_match=3, 16M-token corpus, 1.32 GB of logits per step."""
    _full_size_closed_loop(2, steps=6)


def test_full_size_cfg2_accept_inside_the_argmax_kernel():
    """The same workload with the accept step of every stream inside the argmax kernel (used rows first, one launch per
    step), drafts and n_draft rewritten in place while other CTAs still classify rows."""
    _full_size_closed_loop(2, steps=6, variant=2)


def test_full_size_cfg3_verify_heavy_with_ties():
    """B=512, K=16, 4M-token corpus, 2.64 GB of logits per step, 1 % planted exact ties at the row maximum."""
    cfg, tr = _full_size_closed_loop(3, steps=8)
    # a tie is planted on a share of the used rows; where the extra column is the lower one it must have won
    lower_tie_won = sum(int(((o["argmax"] != o["target"]) & (o["target"] >= 0)).sum()) for o in tr)
    assert lower_tie_won > 0


def test_full_size_cfg4_long_trace():
    """B=1024, K=32 (the largest draft length), min_match=4, 64M-token corpus, 10.3 GB of logits per step."""
    _full_size_closed_loop(4, steps=3)


def test_full_size_cfg5_paper_evaluation_shape():
    """B=4, K=3 (one autoregressive + three speculative tokens per step), 1M-token corpus, all 64 steps."""
    _full_size_closed_loop(5, steps=64)
