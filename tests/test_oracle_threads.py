"""The oracle's batch drivers split rows / streams over OpenMP threads for the timed CPU baseline.  Threads only
partition independent work, so any thread count must give byte-identical outputs.  CPU only."""
from __future__ import annotations

import numpy as np

import oracle
import workload as W
from oracle.backend import OracleBackend


def test_argmax_batch_is_thread_count_independent():
    rng = np.random.default_rng(3)
    bits = W.f32_to_bf16_bits(rng.standard_normal((257, 4099), dtype=np.float32))
    bits[5, [7, 4000]] = 0x4170          # a tie at the maximum
    bits[9, :] = 0xFF80                  # nothing above -inf
    bits[11, 0] = 0x7FC0                 # NaN in front
    one = oracle.argmax_batch(bits, V=4096, threads=1)
    for th in (2, 3, max(2, oracle.host_threads())):
        assert (oracle.argmax_batch(bits, V=4096, threads=th) == one).all(), th


def test_closed_loop_is_thread_count_independent():
    cfg = W.CONFIGS[0].scaled(B=13, steps=6)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    traces = []
    for th in (1, 4, max(2, oracle.host_threads())):
        be = OracleBackend(cfg, corpus, noise.copy(), threads=th)
        traces.append(W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), be))
    for tr in traces[1:]:
        for t, (a, b) in enumerate(zip(traces[0], tr)):
            for k in ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft"):
                assert (a[k] == b[k]).all(), (t, k)


def test_draft_batch_is_thread_count_independent():
    cfg = W.CONFIGS[0]
    corpus = W.make_corpus(cfg)
    sam = oracle.OracleSAM(corpus, [cfg.separator])
    rng = np.random.default_rng(8)
    B, ld = 37, 11
    toks = np.empty((B, ld), np.int32)
    for b in range(B):
        s0 = int(rng.integers(0, corpus.shape[0] - ld))
        toks[b] = corpus[s0:s0 + ld]
    toks[rng.random((B, ld)) < 0.1] = 5
    n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
    outs = []
    for th in (1, 5):
        st, ml = np.zeros(B, np.int32), np.zeros(B, np.int32)
        d, nd = sam.draft_batch(st, ml, toks, n_new, cfg.K, cfg.min_match, th)
        outs.append((st, ml, d, nd))
    for x, y in zip(outs[0], outs[1]):
        assert (x == y).all()
