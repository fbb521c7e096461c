"""Pins for the oracle's composite drafting over several automata (CPU only): the slot that wins is the
one a naive scan of every member corpus says has the largest weight x longest-suffix length, and the
draft is that corpus' continuation."""
from __future__ import annotations

import numpy as np

import oracle
from tests import naive


def _members(rng, n, sigma, sep):
    corpora = [rng.integers(0, sigma, size=int(rng.integers(60, 140))).astype(np.int32) for _ in range(n)]
    return corpora, [oracle.OracleSAM(c, [sep]) for c in corpora]


def test_choice_equals_naive_scan_of_every_member():
    rng = np.random.default_rng(0)
    sigma, sep, B, M, K, mm = 3, 9, 10, 3, 4, 2
    corpora, members = _members(rng, 5, sigma, sep)
    slots = rng.integers(-1, 5, size=(B, M)).astype(np.int32)
    weights = rng.choice(np.array([0.25, 0.5, 1.0, 1.5], np.float32), size=(B, M)).astype(np.float32)
    st = np.zeros((B, M), np.int32); ml = np.zeros((B, M), np.int32)
    hist = [[] for _ in range(B)]
    picked = set()
    for step in range(12):
        ld = 5
        toks = rng.integers(0, sigma, size=(B, ld)).astype(np.int32)
        n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
        d, nd, ch = oracle.multi_draft(members, slots, weights, st, ml, toks, n_new, K, mm)
        for b in range(B):
            hist[b] += [int(x) for x in toks[b, :n_new[b]]]
            best, best_m, best_end = None, -1, -1
            for m in range(M):
                if slots[b, m] < 0:
                    continue
                L, end = naive.longest_suffix_match(corpora[slots[b, m]], hist[b])
                assert L == ml[b, m]
                if L >= mm:
                    score = np.float32(weights[b, m]) * np.float32(L)
                    if best is None or score > best:
                        best, best_m, best_end = score, m, end
            assert ch[b] == best_m
            if best_m >= 0:
                dn, ndn = naive.naive_draft(corpora[slots[b, best_m]], [sep], int(ml[b, best_m]), best_end, K, mm)
                assert nd[b] == ndn and (d[b] == dn).all()
                picked.add(best_m)
            else:
                assert nd[b] == 0 and (d[b] == -1).all()
    assert len(picked) > 1


def test_single_slot_is_plain_drafting_and_weights_break_length_ties():
    rng = np.random.default_rng(1)
    corpora, members = _members(rng, 2, 3, 9)
    B, K, mm = 6, 3, 1
    toks = rng.integers(0, 3, size=(B, 4)).astype(np.int32)
    n_new = np.full(B, 4, np.int32)
    st = np.zeros((B, 1), np.int32); ml = np.zeros((B, 1), np.int32)
    d, nd, ch = oracle.multi_draft(members, np.zeros((B, 1), np.int32), np.ones((B, 1), np.float32), st, ml, toks, n_new, K, mm)
    s1 = np.zeros(B, np.int32); l1 = np.zeros(B, np.int32)
    d1, nd1 = members[0].draft_batch(s1, l1, toks, n_new, K, mm)
    assert (d == d1).all() and (nd == nd1).all() and (st[:, 0] == s1).all() and (ch == np.where(l1 >= mm, 0, -1)).all()
    # the same automaton in two slots: equal lengths, so the heavier slot wins; equal weights, the lower slot
    st = np.zeros((B, 2), np.int32); ml = np.zeros((B, 2), np.int32)
    w = np.tile(np.array([[1.0, 2.0]], np.float32), (B, 1))
    _, _, ch = oracle.multi_draft(members, np.zeros((B, 2), np.int32), w, st, ml, toks, n_new, K, mm)
    assert (ch[l1 >= mm] == 1).all()
    st[:] = 0; ml[:] = 0
    _, _, ch = oracle.multi_draft(members, np.zeros((B, 2), np.int32), np.ones((B, 2), np.float32), st, ml, toks, n_new, K, mm)
    assert (ch[l1 >= mm] == 0).all()
