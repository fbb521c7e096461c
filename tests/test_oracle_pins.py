"""Pins of the CPU oracle against things that are not the oracle: brute force,
closed forms, textbook bounds, a hand-derived example, library routines on the
cases where they are unambiguous.  CPU only."""
from __future__ import annotations

import os

import numpy as np
import pytest

import oracle
from tests import naive
from workload import f32_to_bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example_abcbc.txt")


def _rand_corpora():
    rng = np.random.default_rng(123)
    out = []
    for sigma in (1, 2, 3, 4):
        for n in (1, 2, 3, 7, 20, 60, 150):
            out.append(rng.integers(0, sigma, size=n).astype(np.int32))
    # Zipf-like tokens over a larger alphabet, with a copied span (forces long repeats)
    for n in (50, 200):
        z = np.minimum(rng.zipf(1.3, size=n), 40).astype(np.int32)
        z[n // 2:n // 2 + 10] = z[3:13]
        out.append(z)
    return out


def _check_structure(ex, n):
    ln, link, fp = ex["len"], ex["link"], ex["firstpos"]
    rp, et, ed = ex["row_ptr"], ex["edge_tok"], ex["edge_dst"]
    S = ln.shape[0]
    assert ln[0] == 0 and link[0] == -1 and fp[0] == -1
    assert (link[1:] >= 0).all() and (link[1:] < S).all()
    assert (ln[link[1:]] < ln[1:]).all()                    # link strictly shortens
    assert (fp[1:] >= 0).all() and (fp[1:] < n).all()
    for s in range(S):
        row = et[rp[s]:rp[s + 1]]
        assert (np.diff(row) > 0).all()                    # strictly ascending tokens
        dst = ed[rp[s]:rp[s + 1]]
        assert (ln[dst] >= ln[s] + 1).all()
    # every state reaches the root through links (tree): len strictly decreases, so it ends
    if n >= 2:
        assert S <= 2 * n - 1
    if n >= 3:
        assert et.shape[0] <= 3 * n - 4


@pytest.mark.parametrize("idx", range(len(_rand_corpora())))
def test_substring_count_membership_firstpos(idx):
    corpus = _rand_corpora()[idx]
    n = corpus.shape[0]
    sam = oracle.OracleSAM(corpus, [10 ** 6])
    ex = sam.export()
    _check_structure(ex, n)
    subs = naive.all_substrings(corpus)
    # distinct substrings = sum over non-root states of len(s) - len(link(s))
    assert int((ex["len"][1:] - ex["len"][ex["link"][1:]]).sum()) == len(subs)
    # every substring is accepted from the root with matched length == its length
    sample = sorted(subs)
    rng = np.random.default_rng(idx)
    if len(sample) > 400:
        sample = [sample[i] for i in rng.choice(len(sample), 400, replace=False)]
    for sub in sample:
        s, L = sam.walk(0, 0, np.array(sub, np.int32))
        assert L == len(sub)
        # the state's first end position is the first occurrence of this very substring
        assert ex["firstpos"][s] == naive.first_end_position(corpus, sub)
    # strings that are not substrings are not fully matched
    sigma = int(corpus.max()) + 1
    misses = 0
    for _ in range(200):
        m = int(rng.integers(1, min(n, 6) + 1))
        cand = tuple(int(x) for x in rng.integers(0, sigma + 1, size=m))
        if cand in subs:
            continue
        _, L = sam.walk(0, 0, np.array(cand, np.int32))
        assert L < m
        misses += 1
    assert misses > 0 or sigma == 1
    # the longest string of each state ends at firstpos, and firstpos is its first occurrence
    for s in range(1, ex["len"].shape[0]):
        e, ln = int(ex["firstpos"][s]), int(ex["len"][s])
        w = corpus[e - ln + 1:e + 1]
        assert w.shape[0] == ln
        s2, L2 = sam.walk(0, 0, w)
        assert (s2, L2) == (s, ln)
        assert naive.first_end_position(corpus, w) == e


@pytest.mark.parametrize("n", [1, 2, 5, 33])
def test_closed_form_all_distinct(n):
    corpus = np.arange(n, dtype=np.int32)[::-1].copy()     # descending ids: sorting must reorder the root row
    sam = oracle.OracleSAM(corpus, [10 ** 6])
    ex = sam.export()
    assert sam.n_states == n + 1 and sam.n_edges == 2 * n - 1
    assert (ex["len"] == np.arange(n + 1)).all()
    assert (ex["link"][1:] == 0).all()
    assert (ex["firstpos"][1:] == np.arange(n)).all()
    root = ex["edge_tok"][ex["row_ptr"][0]:ex["row_ptr"][1]]
    assert (root == np.arange(n)).all()
    root_dst = ex["edge_dst"][ex["row_ptr"][0]:ex["row_ptr"][1]]
    assert (root_dst == n - np.arange(n)).all()             # token t sits at position n-1-t -> state n-t
    assert int((ex["len"][1:] - ex["len"][ex["link"][1:]]).sum()) == n * (n + 1) // 2


@pytest.mark.parametrize("n", [1, 2, 6, 40])
def test_closed_form_single_letter(n):
    sam = oracle.OracleSAM(np.full(n, 7, np.int32), [10 ** 6])
    ex = sam.export()
    assert sam.n_states == n + 1 and sam.n_edges == n
    assert (ex["link"][1:] == np.arange(n)).all()
    assert (ex["firstpos"][1:] == np.arange(n)).all()
    assert int((ex["len"][1:] - ex["len"][ex["link"][1:]]).sum()) == n


@pytest.mark.parametrize("n", [3, 5, 8, 21])
def test_extremal_families(n):
    """Textbook extremal inputs: a b^(n-1) reaches 2n-1 states, a b^(n-2) c reaches 3n-4 transitions."""
    abn = np.array([0] + [1] * (n - 1), np.int32)
    assert oracle.OracleSAM(abn, [99]).n_states == 2 * n - 1
    abc = np.array([0] + [1] * (n - 2) + [2], np.int32)
    assert oracle.OracleSAM(abc, [99]).n_edges == 3 * n - 4


def _read_golden():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            s, ln, link, fp, edges = line.split()
            e = [] if edges == "-" else [tuple(int(x) for x in kv.split(":")) for kv in edges.split(",")]
            rows.append((int(s), int(ln), int(link), int(fp), e))
    return rows


def test_worked_example():
    corpus = np.array([0, 1, 2, 1, 2], np.int32)
    sam = oracle.OracleSAM(corpus, [99])
    ex = sam.export()
    rows = _read_golden()
    assert sam.n_states == len(rows) == 8 and sam.n_edges == 9
    for s, ln, link, fp, edges in rows:
        assert (ex["len"][s], ex["link"][s], ex["firstpos"][s]) == (ln, link, fp)
        lo, hi = ex["row_ptr"][s], ex["row_ptr"][s + 1]
        assert list(zip(ex["edge_tok"][lo:hi].tolist(), ex["edge_dst"][lo:hi].tolist())) == edges
    assert sam.walk(0, 0, [1]) == (5, 1)
    assert sam.walk(0, 0, [1, 2]) == (7, 2)
    d, nd = sam.draft(7, 2, 3, 2)
    assert nd == 2 and d.tolist() == [1, 2, -1]
    assert sam.walk(0, 0, [2]) == (7, 1)
    assert sam.walk(0, 0, [2, 0]) == (1, 1)
    d, nd = sam.draft(1, 1, 3, 2)
    assert nd == 0 and d.tolist() == [-1, -1, -1]
    d, nd = sam.draft(1, 1, 3, 1)
    assert nd == 3 and d.tolist() == [1, 2, 1]
    assert sam.walk(7, 2, [9]) == (0, 0)


def _sep_corpus(rng, sessions, ln, sigma, sep):
    parts = []
    for i in range(sessions):
        parts.append(rng.integers(0, sigma, size=ln).astype(np.int32))
        if i + 1 < sessions:
            parts.append(np.array([sep], np.int32))
    return np.concatenate(parts)


@pytest.mark.parametrize("seed,sigma", [(0, 2), (1, 3), (2, 6), (3, 30)])
def test_walk_and_draft_equal_naive_scan(seed, sigma):
    """After every fed token, matched_len is the longest suffix of the whole history that
    occurs in the corpus, the state's firstpos is the end of its first occurrence, and the
    draft is the continuation after that occurrence, cut at a separator / the end."""
    rng = np.random.default_rng(seed)
    sep = sigma
    corpus = _sep_corpus(rng, 4, 40, sigma, sep)
    sam = oracle.OracleSAM(corpus, [sep])
    ex = sam.export()
    for stream in range(6):
        hist = []
        s, L = 0, 0
        for step in range(60):
            r = rng.random()
            if r < 0.6 and len(hist) > 0:
                # follow the corpus after a random occurrence of the last token (keeps matches long)
                occ = np.nonzero(corpus[:-1] == hist[-1])[0]
                tok = int(corpus[rng.choice(occ) + 1]) if occ.shape[0] else int(rng.integers(0, sigma))
            elif r < 0.9:
                tok = int(rng.integers(0, sigma + 1))      # may be the separator itself
            else:
                tok = sigma + 5                             # never in the corpus
            hist.append(tok)
            s, L = sam.walk(s, L, [tok])
            Ln, end = naive.longest_suffix_match(corpus, hist)
            assert L == Ln
            assert int(ex["firstpos"][s]) == end
            if s != 0:
                assert ex["len"][ex["link"][s]] < L <= ex["len"][s]
            for K, mm in ((1, 1), (4, 2), (9, 3)):
                d, nd = sam.draft(s, L, K, mm)
                dn, ndn = naive.naive_draft(corpus, [sep], Ln, end, K, mm)
                assert nd == ndn and (d == dn).all()


def test_multi_token_walk_equals_single_token_walks():
    rng = np.random.default_rng(5)
    corpus = _sep_corpus(rng, 3, 50, 3, 3)
    sam = oracle.OracleSAM(corpus, [3])
    toks = rng.integers(0, 4, size=40).astype(np.int32)
    s, L = 0, 0
    for t in toks:
        s, L = sam.walk(s, L, [t])
    assert sam.walk(0, 0, toks) == (s, L)
    assert sam.walk(4, 2, np.zeros(0, np.int32)) == (4, 2)   # no tokens: unchanged


# ------------------------------------------------------------------ argmax / accept
def _bits(x):
    return f32_to_bf16_bits(np.asarray(x, np.float32))


def test_argmax_matches_library_on_unique_max_rows():
    rng = np.random.default_rng(0)
    rows = _bits(rng.standard_normal((64, 5000)))
    f = (rows.astype(np.uint32) << 16).view(np.float32)
    got = oracle.argmax_batch(rows)
    checked = 0
    for r in range(rows.shape[0]):
        m = f[r].max()
        if (f[r] == m).sum() == 1:
            assert got[r] == int(np.argmax(f[r]))
            checked += 1
        else:
            assert got[r] == int(np.nonzero(f[r] == m)[0][0])
    assert checked > 32


def test_argmax_special_rows():
    assert oracle.argmax_row(_bits([-3.0, -1.5, -2.0, -1.5])) == 1        # negatives, tie -> lowest
    assert oracle.argmax_row(_bits([1.0])) == 0
    assert oracle.argmax_row(_bits([2.0, 2.0, 2.0])) == 0
    assert oracle.argmax_row(np.array([0x8000, 0x0000, 0x8000], np.uint16)) == 0   # -0 == +0
    assert oracle.argmax_row(np.array([0xBF80, 0x8000, 0x0000], np.uint16)) == 1   # -1, -0, +0
    assert oracle.argmax_row(_bits([-np.inf, -np.inf])) == 0
    assert oracle.argmax_row(_bits([0.5, np.inf, 3.0, np.inf])) == 1
    assert oracle.argmax_row(np.array([0x3F80, 0x7FC0, 0x4000], np.uint16)) == 2   # NaN never wins
    assert oracle.argmax_row(np.array([0x7FC0, 0x3F80, 0x4000], np.uint16)) == 0   # NaN first: nothing beats it
    # planted unique maximum at a known place, last / first / middle column
    rng = np.random.default_rng(1)
    base = rng.standard_normal(3001).astype(np.float32)
    for col in (0, 1499, 3000):
        x = base.copy()
        x[col] = 9.0
        assert oracle.argmax_row(_bits(x)) == col
    # planted tie: the lower column wins wherever the pair sits
    for lo, hi in ((0, 3000), (17, 18), (2999, 3000)):
        x = base.copy()
        x[lo] = x[hi] = 9.0
        assert oracle.argmax_row(_bits(x)) == lo


def test_argmax_batch_respects_row_stride_and_V():
    rng = np.random.default_rng(2)
    buf = _bits(rng.standard_normal((5, 300)))
    buf[:, 200:] = _bits(np.float32(50.0))     # beyond V: must be ignored
    got = oracle.argmax_batch(buf, V=200)
    f = (buf[:, :200].astype(np.uint32) << 16).view(np.float32)
    for r in range(5):
        assert got[r] == int(np.nonzero(f[r] == f[r].max())[0][0])


def test_accept_equals_prefix_compare():
    rng = np.random.default_rng(3)
    for _ in range(500):
        K = int(rng.integers(1, 9))
        nd = int(rng.integers(0, K + 1))
        am = rng.integers(0, 4, size=K + 1).astype(np.int32)
        dr = np.full(K, -1, np.int32)
        dr[:nd] = np.where(rng.random(nd) < 0.7, am[:nd], rng.integers(0, 4, size=nd))
        acc, n = oracle.accept(dr, nd, am)
        acc2, n2 = naive.naive_accept(dr, nd, am, K)
        assert n == n2 and (acc == acc2).all()
        assert 1 <= n <= nd + 1
    # full accept takes the bonus from row n_draft; empty draft commits the model's token
    acc, n = oracle.accept(np.array([4, 5], np.int32), 2, np.array([4, 5, 6], np.int32))
    assert n == 3 and acc.tolist() == [4, 5, 6]
    acc, n = oracle.accept(np.array([-1, -1], np.int32), 0, np.array([8, 1, 2], np.int32))
    assert n == 1 and acc.tolist() == [8, -1, -1]
    acc, n = oracle.accept(np.array([4, 5], np.int32), 2, np.array([4, 9, 6], np.int32))
    assert n == 2 and acc.tolist() == [4, 9, -1]
