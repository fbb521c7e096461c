"""Seeded random sweeps of the CUDA path against the oracle: shapes nobody picked by hand.

Verification over random (B, K, V, row padding) with special values sprinkled in, and closed loops over
corpora with two to a few dozen distinct tokens, where almost every state is a clone or has a long chain of
suffix links and every miss follows many of them.
"""
import numpy as np
import pytest
import torch

import oracle
import workload as W
from harness.cuda_backend import CudaBackend, bits_to_device
from oracle.backend import OracleBackend
import paper_2512_18337_b200 as S

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SPECIAL = np.array([0x0000, 0x8000, 0x7F80, 0xFF80, 0x7FC0, 0xFFC0, 0x7F7F, 0xFF7F, 0x0001, 0x8001], np.uint16)


def _i32(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)


def _random_case(rng):
    V = int(np.exp(rng.uniform(0, np.log(300000))))
    if rng.random() < 0.3:
        V = max(1, (V // 8) * 8)                       # rows that qualify for the bulk-copy kernel
    pad = int(rng.choice([0, 0, 1, 3, 8, 9]))
    K = int(rng.integers(1, 33))
    B = int(rng.integers(1, 24))
    while B * (K + 1) * (V + pad) > 6_000_000 and B > 1:
        B //= 2
    while (K + 1) * (V + pad) * B > 6_000_000 and K > 1:
        K //= 2
    return V, pad, B, K


@pytest.mark.parametrize("seed", range(24))
def test_verify_random_shapes_and_values(seed):
    rng = np.random.default_rng(1000 + seed)
    V, pad, B, K = _random_case(rng)
    R = B * (K + 1)
    bits = W.f32_to_bf16_bits(rng.standard_normal((R, V + pad), dtype=np.float32))
    # coarse values in some rows: many equal maxima
    coarse = rng.random(R) < 0.3
    bits[coarse] &= np.uint16(0xFFC0)
    # special bit patterns anywhere, the row ends included
    n_sp = int(rng.integers(0, 4 * R + 1))
    rr = rng.integers(0, R, size=n_sp)
    cc = np.where(rng.random(n_sp) < 0.3, rng.choice(np.array([0, V - 1]), size=n_sp), rng.integers(0, V, size=n_sp))
    bits[rr, cc] = rng.choice(SPECIAL, size=n_sp)
    if pad:
        bits[:, V:] = rng.choice(np.array([0x7F00, 0x7F80, 0x7FC0], np.uint16))    # beyond V: never read as a value
    am_o = oracle.argmax_batch(bits, V=V, threads=oracle.host_threads()).reshape(B, K + 1)
    n_draft = rng.integers(0, K + 1, size=B).astype(np.int32)
    drafts = np.full((B, K), -1, np.int32)
    for b in range(B):
        nd = n_draft[b]
        drafts[b, :nd] = np.where(rng.random(nd) < 0.8, am_o[b, :nd], rng.integers(0, V, size=nd))
    acc_o, nacc_o = oracle.accept_batch(drafts, n_draft, am_o)
    lg = bits_to_device(bits)
    wsb = S.sam_workspace_bytes(B, K)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    S.sam_workspace_init(ws, wsb)
    d, nd_t = _i32(drafts), _i32(n_draft)
    for variant in (0, 1, 2, 3):
        am = torch.full((B, K + 1), -9, dtype=torch.int32, device=DEV)
        acc = torch.full((B, K + 1), -9, dtype=torch.int32, device=DEV)
        nacc = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        S.sam_set_argmax_variant(variant)
        try:
            S.sam_verify(lg, V + pad, B, K, V, d, nd_t, am, acc, nacc, ws, wsb)
            torch.cuda.synchronize()
        finally:
            S.sam_set_argmax_variant(0)
        assert S.sam_workspace_status(ws, B, K) == 0
        assert (am.cpu().numpy() == am_o).all(), (V, pad, B, K, variant)
        assert (nacc.cpu().numpy() == nacc_o).all() and (acc.cpu().numpy() == acc_o).all(), (V, pad, B, K, variant)


@pytest.mark.parametrize("vocab,K,mm,variant", [
    (2, 4, 1, 0), (3, 32, 2, 0), (5, 8, 3, 1), (17, 16, 2, 0),
    (8, 8, 2, 3), (8, 8, 2, 2), (16, 32, 1, 0), (24, 5, 4, 2), (32, 16, 2, 3),
])
def test_closed_loop_small_alphabets(vocab, K, mm, variant):
    """Two to thirty-two distinct tokens: long runs, clones everywhere, suffix-link chains dozens deep.
    Alphabets of 8, 16, 24, 32 give rows of whole 16-byte units (bulk-copy kernel, thousands of rows per tile)."""
    cfg = W.CONFIGS[0].scaled(vocab=vocab, B=96, K=K, steps=10, min_match=mm, sessions=8)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    tr_o = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax),
                             OracleBackend(cfg, corpus, noise.copy(), oracle.host_threads()), None)
    S.sam_set_argmax_variant(variant)
    try:
        tr_g = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax),
                                 CudaBackend(cfg, corpus, bits_to_device(noise)), None)
    finally:
        S.sam_set_argmax_variant(0)
    assert len(tr_o) == len(tr_g)
    for t, (o, g) in enumerate(zip(tr_o, tr_g)):
        for k in ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft"):
            assert (o[k] == g[k]).all(), (t, k)
    assert max(int(t["matched_len"].max()) for t in tr_o) >= 20


@pytest.mark.parametrize("alphabet,start_len", [(2, 0), (2, 600), (3, 600), (4, 50), (6, 1500)])
def test_growing_index_small_alphabets(alphabet, start_len):
    """Growth over a handful of distinct tokens: every appended token splits states (clones that take over
    existing transitions), rows change from inline to sorted, and matched states move under the streams."""
    rng = np.random.default_rng(alphabet * 100 + start_len)
    sep, K, mm, B, ld = 9, 7, 1, 40, 10

    def text_piece(n):
        t = rng.integers(0, alphabet, size=n).astype(np.int32)
        runs = rng.integers(0, max(1, n), size=max(1, n // 30))
        for r in runs:                                   # long runs of one token: deep suffix-link chains
            t[r:r + int(rng.integers(2, 25))] = t[r] if n else 0
        if n > 20:
            t[rng.integers(0, n, size=n // 40 + 1)] = sep
        return t

    text = text_piece(start_len)
    index = S.SamIndex(text, [sep], max_tokens=8000, max_token_id=sep + 1)
    osam = oracle.OracleSAM(text, [sep])
    st = torch.zeros(B, dtype=torch.int32, device=DEV)
    ml = torch.zeros(B, dtype=torch.int32, device=DEV)
    st_o = np.zeros(B, np.int32)
    ml_o = np.zeros(B, np.int32)
    moved = 0
    for rnd in range(20):
        piece = text_piece(int(rng.integers(1, 250)))
        osam.extend(piece)
        S.sam_extend(index.handle, piece)
        before = st_o.copy()
        osam.renormalize(st_o, ml_o)
        moved += int((before != st_o).sum())
        if rnd % 2 == 0:
            assert S.sam_sync(index.handle) == osam.n
            S.sam_renormalize(index.handle, B, st, ml)
        else:
            assert S.sam_sync_renormalize(index.handle, B, st, ml) == osam.n
        torch.cuda.synchronize()
        assert (st.cpu().numpy() == st_o).all() and (ml.cpu().numpy() == ml_o).all()
        toks = rng.integers(0, alphabet, size=(B, ld)).astype(np.int32)
        if osam.n > ld:
            for b in range(0, B, 2):                     # half the streams re-read the text, half are random
                s0 = int(rng.integers(0, osam.n - ld))
                toks[b] = osam.corpus[s0:s0 + ld]
        toks[rng.random((B, ld)) < 0.03] = alphabet + 1   # a token the text never has
        n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
        d = torch.full((B, K), -9, dtype=torch.int32, device=DEV)
        nd = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        S.sam_draft(index.handle, B, st, ml, _i32(toks), ld, _i32(n_new), K, mm, d, nd)
        torch.cuda.synchronize()
        d_o, nd_o = osam.draft_batch(st_o, ml_o, toks, n_new, K, mm)
        assert (st.cpu().numpy() == st_o).all() and (ml.cpu().numpy() == ml_o).all(), rnd
        assert (nd.cpu().numpy() == nd_o).all() and (d.cpu().numpy() == d_o).all(), rnd
    assert moved > 0
    ex, oe = S.sam_export(index.handle), osam.export()
    for k in oe:
        assert (ex[k] == oe[k]).all(), k
