"""Generator shape/recipe checks and an oracle closed loop on the tiny config. CPU only."""
from __future__ import annotations

import numpy as np

import workload as W
from tests import naive
from oracle.backend import OracleBackend


def test_bf16_rounding():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.14159], np.float32)
    b = W.f32_to_bf16_bits(x)
    back = W.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[3] == -2.5 and back[4] == 0.0
    assert back[1] == 1.0            # 1 + 2^-8 is a tie -> rounds to even (1.0)
    assert back[2] == 1.015625       # 1 + 3*2^-8 is a tie -> rounds to even (1 + 2^-6)
    assert abs(back[5] - 3.14159) <= 2 ** -7 * 2


def test_corpus_shape_and_repeats():
    cfg = W.CONFIGS[0]
    c = W.make_corpus(cfg)
    assert c.shape == (8003,) and c.dtype == np.int32
    sep = np.nonzero(c == cfg.separator)[0]
    assert sep.tolist() == [2000, 4001, 6002]
    body = c[c != cfg.separator]
    assert body.min() >= 0 and body.max() < cfg.vocab
    # Zipf: the most frequent id is 0 and the head dominates
    cnt = np.bincount(body, minlength=cfg.vocab)
    assert cnt.argmax() == 0 and cnt[:10].sum() > 0.25 * body.shape[0]
    assert (W.make_corpus(cfg) == c).all()                # seeded


def test_closed_loop_oracle_tiny():
    cfg = W.CONFIGS[0]
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    pristine = noise.copy()
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    feeder = W.ClosedLoopFeeder(cfg, scripts, rowmax)
    be = OracleBackend(cfg, corpus, noise)
    hist = [list(scripts[b, :cfg.prime]) for b in range(cfg.B)]
    trace = W.run_closed_loop(cfg, feeder, be)
    assert (noise == pristine).all()                      # planting undone after every step
    used_tie = 0
    for out in trace:
        for b in range(cfg.B):
            nd = int(out["in_n_draft"][b])
            tgt = out["target"][b]
            # the planted token is the row argmax on used rows unless a planted tie sits lower
            am = out["argmax"][b]
            for j in range(nd + 1):
                assert am[j] <= tgt[j]
                used_tie += int(am[j] < tgt[j])
            acc, n = naive.naive_accept(out["in_drafts"][b], nd, am, cfg.K)
            assert n == out["n_accepted"][b] and (acc == out["accepted"][b]).all()
            hist[b].extend(acc[:n].tolist())
            L, end = naive.longest_suffix_match(corpus, hist[b])
            assert L == out["matched_len"][b]
            d, ndn = naive.naive_draft(corpus, [cfg.separator], L, end, cfg.K, cfg.min_match)
            assert ndn == out["n_draft"][b] and (d == out["drafts"][b]).all()
    st = W.trace_stats(cfg, trace)
    assert st["ote"] >= 1.0 and 0.0 <= st["shr"] <= 1.0
    assert st["nonempty_frac"] > 0.2 and st["ote"] > 1.3   # the loop keeps re-entering corpus spans
