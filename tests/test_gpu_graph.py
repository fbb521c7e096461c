"""The fused step recorded once in a CUDA graph and replayed: same trace as the oracle.

A serving loop that calls sam_step thousands of times with the same buffers can record the call's launches in a
graph (after one ordinary call, which does the library's first-use set-up) and replay it; the replay does no host
work per kernel and keeps the dependent launch of the accept kernel.  Here the replayed step drives whole closed
loops and every output of every step is compared with the oracle.
"""
from __future__ import annotations

import pytest
import torch

import oracle
import paper_2512_18337_b200 as S
import workload as W
from harness.cuda_backend import CudaBackend, bits_to_device
from oracle.backend import OracleBackend

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("which,variant,flags", [
    ("tiny", 0, 0),
    ("cfg2_small", 0, 0),
    ("cfg2_small", 2, 0),
    ("cfg2_small", 3, 0),
    ("cfg2_small", 3, S.SAM_STEP_SKIP_UNUSED_ROWS),
    ("cfg2_small", 0, S.SAM_STEP_SKIP_UNUSED_ROWS),
    ("paper_shape", 0, 0),
])
def test_replayed_step_matches_the_oracle(which, variant, flags):
    cfg = {"tiny": W.CONFIGS[0],
           "cfg2_small": W.CONFIGS[2].scaled(sessions=64, B=48, steps=8),
           "paper_shape": W.CONFIGS[5].scaled(sessions=32, steps=12)}[which]
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    ob = OracleBackend(cfg, corpus, noise.copy(), oracle.host_threads())
    tr_o = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), ob, None)

    be = CudaBackend(cfg, corpus, bits_to_device(noise))
    be.flags = flags
    be.counters = torch.zeros(S.SAM_N_COUNTERS, dtype=torch.int64, device=be.device)
    S.sam_set_argmax_variant(variant)
    try:
        # one ordinary call first (first-use set-up), then everything it touched is put back
        keep = [t.clone() for t in (be.state, be.mlen, be.drafts, be.n_draft)]
        be.launch_step()
        torch.cuda.synchronize()
        for t, k in zip((be.state, be.mlen, be.drafts, be.n_draft), keep):
            t.copy_(k)
        be.counters.zero_()
        S.sam_workspace_init(be.ws, be.ws_bytes)
        graph = torch.cuda.CUDAGraph()
        before = S.sam_launch_count()
        with torch.cuda.graph(graph):
            be.launch_step()                     # recorded, not run
        assert S.sam_launch_count() - before >= 1
        be.launch_step = graph.replay
        tr_g = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), be, None)
    finally:
        S.sam_set_argmax_variant(0)
    assert be.status() == 0
    assert len(tr_o) == len(tr_g)
    skip = bool(flags & S.SAM_STEP_SKIP_UNUSED_ROWS)
    for t, (o, g) in enumerate(zip(tr_o, tr_g)):
        for k in ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft"):
            if k == "argmax" and skip:
                continue                         # rows beyond the proposal are not computed in this mode (the rest agrees)
            assert (o[k] == g[k]).all(), (t, k)
    committed = sum(int(o["n_accepted"].sum()) for o in tr_o)
    assert int(be.counters[1]) == committed
