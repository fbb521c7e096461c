"""Pins for the oracle's growing automaton (appending verified tokens, Section 5.4.2) against brute
force on tiny inputs.  CPU only.

Appending is more steps of the same incremental construction, so every brute-force property of a
one-shot build must hold for a text that arrived in pieces; a stream's (state, matched_len) taken
before the text grew must, after renormalising, name the state that the extended automaton reaches
on that very string."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from tests import naive


def _pieces(rng, n, sigma, k):
    text = rng.integers(0, sigma, size=n).astype(np.int32)
    cuts = np.sort(rng.choice(np.arange(1, n), size=min(k, n - 1), replace=False))
    return text, np.split(text, cuts)


@pytest.mark.parametrize("seed,sigma,n", [(0, 1, 30), (1, 2, 90), (2, 3, 120), (3, 5, 150), (4, 40, 150)])
def test_text_that_arrives_in_pieces(seed, sigma, n):
    rng = np.random.default_rng(seed)
    text, parts = _pieces(rng, n, sigma, 6)
    sam = oracle.OracleSAM(parts[0], [10 ** 6])
    for p in parts[1:]:
        sam.extend(p)
    assert sam.n == n and (sam.corpus == text).all()
    ex = sam.export()
    subs = naive.all_substrings(text)
    assert int((ex["len"][1:] - ex["len"][ex["link"][1:]]).sum()) == len(subs)
    for s in range(1, ex["len"].shape[0]):
        e, ln = int(ex["firstpos"][s]), int(ex["len"][s])
        w = text[e - ln + 1:e + 1]
        assert sam.walk(0, 0, w) == (s, ln)
        assert naive.first_end_position(text, w) == e
    for row in range(ex["len"].shape[0]):
        toks = ex["edge_tok"][ex["row_ptr"][row]:ex["row_ptr"][row + 1]]
        assert (np.diff(toks) > 0).all()
    # membership of non-substrings
    for _ in range(100):
        m = int(rng.integers(1, 6))
        cand = tuple(int(x) for x in rng.integers(0, sigma + 1, size=m))
        if cand not in subs:
            assert sam.walk(0, 0, np.array(cand, np.int32))[1] < m


@pytest.mark.parametrize("seed,sigma", [(0, 2), (1, 3), (2, 4), (3, 12)])
def test_stream_states_survive_growth(seed, sigma):
    """Streams are walked, the text grows (splits move strings into new states), the pairs are
    renormalised, and walking goes on: after every event the pair names the right state."""
    rng = np.random.default_rng(100 + seed)
    text = rng.integers(0, sigma, size=60).astype(np.int32)
    sam = oracle.OracleSAM(text, [10 ** 6])
    n_streams = 8
    hist = [[] for _ in range(n_streams)]
    st = np.zeros(n_streams, np.int32)
    ml = np.zeros(n_streams, np.int32)
    moved = 0

    def check():
        ex = sam.export()
        for b in range(n_streams):
            L = int(ml[b])
            assert L <= len(hist[b])
            suffix = np.array(hist[b][len(hist[b]) - L:], np.int32)
            # the state reached on that string from the root of the current automaton
            s_ref, L_ref = sam.walk(0, 0, suffix)
            assert L_ref == L and s_ref == int(st[b])
            if L > 0:
                assert int(ex["firstpos"][st[b]]) == naive.first_end_position(sam.corpus, suffix)
                assert ex["len"][ex["link"][st[b]]] < L <= ex["len"][st[b]]

    for rnd in range(12):
        for b in range(n_streams):
            for _ in range(int(rng.integers(1, 5))):
                if hist[b] and rng.random() < 0.7:
                    occ = np.nonzero(sam.corpus[:-1] == hist[b][-1])[0]
                    tok = int(sam.corpus[rng.choice(occ) + 1]) if occ.shape[0] else int(rng.integers(0, sigma))
                else:
                    tok = int(rng.integers(0, sigma + 1))
                hist[b].append(tok)
                s, L = sam.walk(int(st[b]), int(ml[b]), [tok])
                st[b], ml[b] = s, L
        check()
        # the text grows: sometimes by a stream's own recent tokens (its verified output), sometimes by new text
        if rng.random() < 0.5:
            b = int(rng.integers(0, n_streams))
            piece = np.array(hist[b][-int(rng.integers(1, 9)):], np.int32)
        else:
            piece = rng.integers(0, sigma, size=int(rng.integers(1, 12))).astype(np.int32)
        sam.extend(piece)
        before = st.copy()
        sam.renormalize(st, ml)
        moved += int((before != st).sum())
        check()
    assert moved > 0 or sigma > 8        # small alphabets split states all the time: the climb must have been needed


def test_renormalize_is_identity_without_growth():
    rng = np.random.default_rng(9)
    text = rng.integers(0, 3, size=80).astype(np.int32)
    sam = oracle.OracleSAM(text, [7])
    st = np.zeros(20, np.int32)
    ml = np.zeros(20, np.int32)
    for b in range(20):
        s, L = sam.walk(0, 0, rng.integers(0, 3, size=int(rng.integers(0, 15))).astype(np.int32))
        st[b], ml[b] = s, L
    ref = st.copy()
    sam.renormalize(st, ml)
    assert (st == ref).all()
