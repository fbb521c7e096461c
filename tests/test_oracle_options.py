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
