"""Brute-force definitions used to pin the oracle (tiny inputs only).

Nothing here builds an automaton: substrings are enumerated or searched directly.
"""
from __future__ import annotations

import numpy as np


def all_substrings(corpus) -> set:
    c = tuple(int(x) for x in corpus)
    n = len(c)
    return {c[i:j] for i in range(n) for j in range(i + 1, n + 1)}


def first_end_position(corpus, pattern) -> int:
    """Index of the last token of the first occurrence of pattern, or -1."""
    c = [int(x) for x in corpus]
    p = [int(x) for x in pattern]
    m = len(p)
    for i in range(len(c) - m + 1):
        if c[i:i + m] == p:
            return i + m - 1
    return -1


def longest_suffix_match(corpus: np.ndarray, history) -> tuple[int, int]:
    """(L, end) where L is the length of the longest suffix of history that occurs
    contiguously in corpus and end is the index of the last token of its FIRST
    occurrence (end = -1 when L = 0).  Candidate filtering, vectorised."""
    corpus = np.asarray(corpus)
    h = np.asarray(history)
    n = corpus.shape[0]
    if h.shape[0] == 0:
        return 0, -1
    cand = np.nonzero(corpus == h[-1])[0]  # end positions of matches of length 1
    if cand.shape[0] == 0:
        return 0, -1
    L = 1
    while L < h.shape[0]:
        prev = cand - L
        ok = prev >= 0
        ok[ok] = corpus[prev[ok]] == h[-1 - L]
        nxt = cand[ok]
        if nxt.shape[0] == 0:
            break
        cand = nxt
        L += 1
    return L, int(cand.min())


def naive_draft(corpus: np.ndarray, separators, L: int, end: int, K: int, min_match: int):
    """Continuation after the first occurrence: up to K tokens after index end,
    cut before a separator or the corpus end; nothing if L < min_match."""
    out = np.full(K, -1, dtype=np.int32)
    if L < min_match:
        return out, 0
    seps = set(int(s) for s in np.atleast_1d(separators))
    n = 0
    for j in range(K):
        p = end + 1 + j
        if p >= corpus.shape[0] or int(corpus[p]) in seps:
            break
        out[j] = corpus[p]
        n += 1
    return out, n


def naive_accept(drafts, n_draft: int, argmax_row, K: int):
    acc = [-1] * (K + 1)
    a = 0
    for j in range(n_draft):
        if int(drafts[j]) != int(argmax_row[j]):
            break
        a += 1
    acc[:a] = [int(x) for x in drafts[:a]]
    acc[a] = int(argmax_row[a])
    return np.array(acc, dtype=np.int32), a + 1
