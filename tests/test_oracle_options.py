"""Pins for the oracle's step options and statistics (CPU only): the adaptive switch of Section 5.4.3,
verification restricted to the rows a proposal uses, and the OTE / SHR counters of Section 6.5."""
from __future__ import annotations

import numpy as np

import oracle
import workload as W
from tests import naive


def _setup(seed, B=6, K=4, V=50):
    rng = np.random.default_rng(seed)
    corpus = rng.integers(0, 8, size=300).astype(np.int32)
    sam = oracle.OracleSAM(corpus, [99])
    bits = W.f32_to_bf16_bits(rng.standard_normal((B * (K + 1), V), dtype=np.float32))
    st = np.zeros(B, np.int32); ml = np.zeros(B, np.int32)
    toks = np.stack([corpus[s:s + 6] for s in rng.integers(0, 290, size=B)]).astype(np.int32)
    drafts, n_draft = sam.draft_batch(st, ml, toks, np.full(B, 6, np.int32), K, 2)
    return rng, corpus, sam, bits, st, ml, drafts, n_draft, B, K, V


def test_plain_step_equals_step_without_options_and_counts_by_hand():
    rng, corpus, sam, bits, st, ml, drafts, n_draft, B, K, V = _setup(0)
    # make some drafts right: plant the drafted token as the row maximum on a few rows
    am = oracle.argmax_batch(bits).reshape(B, K + 1)
    for b in range(B):
        for j in range(n_draft[b]):
            if rng.random() < 0.6:
                bits[b * (K + 1) + j, drafts[b, j]] = 0x4200
    st2, ml2 = st.copy(), ml.copy()
    ref = sam.step(bits, B, K, V, drafts, n_draft, st, ml, 2)
    cnt = np.zeros(6, np.int64)
    out = sam.step_ex(bits, B, K, V, drafts, n_draft, st2, ml2, 2, 0, cnt)
    for k in ref:
        assert (ref[k] == out[k]).all(), k
    assert (st == st2).all() and (ml == ml2).all()
    # counters against the definitions, written out from the step's own inputs and outputs
    a = np.array([naive.naive_accept(drafts[b], int(n_draft[b]), out["argmax"][b], K)[1] - 1 for b in range(B)])
    assert cnt.tolist() == [B, int((a + 1).sum()), int(n_draft.sum()), int(a.sum()), int((n_draft > 0).sum()), B * (K + 1)]
    assert a.sum() > 0 and n_draft.sum() > 0


def test_skip_unused_rows_only_changes_the_rows_beyond_the_proposal():
    rng, corpus, sam, bits, st, ml, drafts, n_draft, B, K, V = _setup(1)
    n_draft[0] = 0
    st2, ml2 = st.copy(), ml.copy()
    ref = sam.step(bits, B, K, V, drafts, n_draft, st, ml, 2)
    cnt = np.zeros(6, np.int64)
    out = sam.step_ex(bits, B, K, V, drafts, n_draft, st2, ml2, 2, oracle.SKIP_UNUSED_ROWS, cnt)
    j = np.arange(K + 1)[None, :]
    used = j <= n_draft[:, None]
    assert (out["argmax"][used] == ref["argmax"][used]).all() and (out["argmax"][~used] == -1).all()
    for k in ("accepted", "n_accepted", "drafts", "n_draft"):
        assert (ref[k] == out[k]).all(), k
    assert (st == st2).all() and (ml == ml2).all()
    assert cnt[5] == int((n_draft + 1).sum())


def test_no_speculation_is_plain_decoding():
    rng, corpus, sam, bits, st, ml, drafts, n_draft, B, K, V = _setup(2)
    st0, ml0 = st.copy(), ml.copy()
    cnt = np.zeros(6, np.int64)
    out = sam.step_ex(bits, B, K, V, drafts, n_draft, st, ml, 2, oracle.NO_SPECULATION | oracle.SKIP_UNUSED_ROWS, cnt)
    am0 = oracle.argmax_batch(bits).reshape(B, K + 1)[:, 0]
    assert (out["n_accepted"] == 1).all() and (out["accepted"][:, 0] == am0).all() and (out["accepted"][:, 1:] == -1).all()
    assert (out["n_draft"] == 0).all() and (out["drafts"] == -1).all()
    assert (out["argmax"][:, 0] == am0).all() and (out["argmax"][:, 1:] == -1).all()
    for b in range(B):                       # the walk still follows the committed token
        assert sam.walk(int(st0[b]), int(ml0[b]), [int(am0[b])]) == (int(st[b]), int(ml[b]))
    assert cnt.tolist() == [B, B, 0, 0, 0, B]


def test_adaptive_switch_thresholds():
    # on unless the context length or the batch size exceeds its threshold (Algorithm 3, step 4)
    assert oracle.speculation_enabled(1000, 4, 32768, 16)
    assert oracle.speculation_enabled(32768, 16, 32768, 16)
    assert not oracle.speculation_enabled(32769, 4, 32768, 16)
    assert not oracle.speculation_enabled(1000, 17, 32768, 16)
    assert not oracle.speculation_enabled(10 ** 6, 10 ** 4, 32768, 16)


# ---- the switch driven by the counters ----------------------------------------------------------------
def _window(rng, K, passes, skip, hit):
    """Per-pass (rows read, accepted drafts) of a window: proposals of random length, a share `hit` of them accepted."""
    nd = rng.integers(0, K + 1, size=passes)
    acc = np.minimum(nd, rng.binomial(nd, hit))
    rows = (nd + 1) if skip else np.full(passes, K + 1)
    return rows, acc


def _counters(rows, acc, nd=None):
    c = np.zeros(6, np.int64)
    c[0], c[1], c[3], c[5] = len(rows), int((acc + 1).sum()), int(acc.sum()), int(rows.sum())
    return c


def test_counter_switch_equals_the_cost_model_summed_pass_by_pass():
    """Exact rational arithmetic, one pass at a time: a pass over r rows costs 1 + (c - 1)(r - 1)/K, it commits
    accepted + 1 tokens, plain decoding commits one token per unit of cost.  Speculation pays when the window's
    tokens exceed its cost.  Cost ratios are dyadic so that the oracle's doubles are exact as well."""
    from fractions import Fraction
    rng = np.random.default_rng(17)
    seen = set()
    for _ in range(400):
        K = int(rng.integers(1, 33))
        c = Fraction(int(rng.integers(2, 65)), 16)            # 0.125 .. 4, sixteenths
        rows, acc = _window(rng, K, int(rng.integers(1, 60)), bool(rng.integers(0, 2)), float(rng.random()))
        cost = sum(1 + (c - 1) * Fraction(int(r) - 1, K) for r in rows)
        tokens = sum(int(a) + 1 for a in acc)
        want = tokens > cost
        assert oracle.speculation_pays(_counters(rows, acc), K, float(c)) == want
        seen.add(want)
    assert seen == {True, False}


def test_counter_switch_on_full_passes_is_ote_against_the_cost_ratio():
    """When every pass reads all K+1 rows the rule is OTE > cost ratio, OTE as Section 6.5 defines it (computed here
    by the workload's own statistics routine from a closed-loop trace of the oracle)."""
    cfg = W.CONFIGS[0].scaled(steps=10)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    from oracle.backend import OracleBackend
    trace = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), OracleBackend(cfg, corpus, noise))
    st = W.trace_stats(cfg, trace)
    cnt = np.zeros(6, np.int64)
    for o in trace:
        cnt += [cfg.B, int(o["n_accepted"].sum()), int(o["in_n_draft"].sum()), int((o["n_accepted"] - 1).sum()),
                int((o["in_n_draft"] > 0).sum()), cfg.B * (cfg.K + 1)]
    assert 1.5 < st["ote"] < cfg.K
    for ratio in (1.0, 1.25, st["ote"] - 0.01, st["ote"] + 0.01, float(cfg.K + 1)):
        assert oracle.speculation_pays(cnt, cfg.K, ratio) == (st["ote"] > ratio), ratio


def test_counter_switch_special_cases():
    K = 4
    # no passes in the window: no evidence, speculation stays on
    assert oracle.speculation_pays(np.zeros(6, np.int64), K, 3.0)
    # an exact tie between tokens and cost does not pay: 10 full passes at cost 2 each, 20 tokens
    rows, acc = np.full(10, K + 1), np.ones(10, np.int64)
    assert not oracle.speculation_pays(_counters(rows, acc), K, 2.0)
    acc[0] = 2
    assert oracle.speculation_pays(_counters(rows, acc), K, 2.0)
    # nothing accepted: pays only if a long pass costs less than a short one
    none = np.zeros(10, np.int64)
    assert not oracle.speculation_pays(_counters(rows, none), K, 1.0)
    assert not oracle.speculation_pays(_counters(rows, none), K, 1.5)
    # rows skipped and proposals empty: every pass is a one-row pass, which neither gains nor loses
    assert not oracle.speculation_pays(_counters(np.ones(10, np.int64), none), K, 5.0)
    # the same accepted tokens pay with skipped rows and not without
    rows_skip, acc2 = np.array([2, 1, 1, 1]), np.array([1, 0, 0, 0])
    assert oracle.speculation_pays(_counters(rows_skip, acc2), K, 4.0)          # 5 tokens against 4.75
    assert not oracle.speculation_pays(_counters(np.full(4, K + 1), acc2), K, 4.0)
