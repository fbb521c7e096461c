"""Parity of the growing index on the GPU with the oracle's growing automaton, tolerance 0.

The text grows between decoding steps (new sessions, and the streams' own verified tokens); after
every growth both sides renormalise the stream states, and every later output must still agree."""
from __future__ import annotations

import time

import numpy as np
import pytest
import torch

import oracle
import paper_2512_18337_b200 as S
import workload as W
from harness.cuda_backend import CudaBackend, bits_to_device
from oracle.backend import OracleBackend

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _i32(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)


def _hub_text(rng, n, sep):
    body = rng.integers(0, 400, size=n).astype(np.int32)
    body[::3] = rng.integers(0, 3, size=body[::3].shape[0])      # hubs: rows that keep growing
    body[5::97] = sep
    return body


def _draft_both(index, osam, B, st, ml, st_o, ml_o, toks, n_new, K, mm):
    d = torch.full((B, K), -9, dtype=torch.int32, device=DEV)
    nd = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    S.sam_draft(index.handle, B, st, ml, _i32(toks), toks.shape[1], _i32(n_new), K, mm, d, nd)
    torch.cuda.synchronize()
    d_o, nd_o = osam.draft_batch(st_o, ml_o, toks, n_new, K, mm)
    assert (st.cpu().numpy() == st_o).all() and (ml.cpu().numpy() == ml_o).all()
    assert (nd.cpu().numpy() == nd_o).all() and (d.cpu().numpy() == d_o).all()
    return d_o, nd_o


@pytest.mark.parametrize("seed,compact_every", [(0, None), (1, 4)])
def test_draft_parity_while_the_text_grows(seed, compact_every):
    """With sam_growing_set_relayout_every(4), every fourth update lays the wide rows out afresh and is sent as a
    whole image (what happens by itself when the wide area fills up); the default keeps every update incremental."""
    rng = np.random.default_rng(seed)
    sep, K, mm, B, ld = 1000, 6, 2, 48, 12
    text = _hub_text(rng, 3000, sep)
    index = S.SamIndex(text, [sep], max_tokens=12000, max_token_id=sep + 50)
    if compact_every is not None:
        S.sam_growing_set_relayout_every(index.handle, compact_every)
    osam = oracle.OracleSAM(text, [sep])
    st = torch.zeros(B, dtype=torch.int32, device=DEV)
    ml = torch.zeros(B, dtype=torch.int32, device=DEV)
    st_o = np.zeros(B, np.int32)
    ml_o = np.zeros(B, np.int32)
    hist = [[] for _ in range(B)]
    moved = 0
    for rnd in range(14):
        toks = np.empty((B, ld), np.int32)
        n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
        for b in range(B):
            start = int(rng.integers(0, osam.n - ld))
            toks[b] = osam.corpus[start:start + ld]
            noise = rng.random(ld) < 0.08
            toks[b, noise] = rng.integers(0, sep + 40, size=int(noise.sum()))
            hist[b] += [int(x) for x in toks[b, :n_new[b]]]
        _draft_both(index, osam, B, st, ml, st_o, ml_o, toks, n_new, K, mm)
        # growth: a stream's own recent tokens as a new session, then fresh text with new token ids
        b = int(rng.integers(0, B))
        piece = np.concatenate([[sep], np.array(hist[b][-40:], np.int32), [sep],
                                _hub_text(rng, int(rng.integers(50, 400)), sep),
                                rng.integers(sep + 1, sep + 50, size=5).astype(np.int32)]).astype(np.int32)
        osam.extend(piece)
        S.sam_extend(index.handle, piece)
        before = st_o.copy()
        osam.renormalize(st_o, ml_o)
        moved += int((before != st_o).sum())
        if rnd % 2 == 0:
            assert S.sam_sync(index.handle) == osam.n
            S.sam_renormalize(index.handle, B, st, ml)
        else:                                   # the same in one call (one kernel when the update is small)
            assert S.sam_sync_renormalize(index.handle, B, st, ml) == osam.n
        torch.cuda.synchronize()
        assert (st.cpu().numpy() == st_o).all()
        # n_new = 0: the draft is re-emitted from the (moved) state over the grown text
        _draft_both(index, osam, B, st, ml, st_o, ml_o, toks, np.zeros(B, np.int32), K, mm)
    assert moved > 0
    inc, full, nbytes = S.sam_update_stats(index.handle)
    assert inc + full == 14 and nbytes > 0
    assert full == (3 if compact_every is not None else 0)
    ex, oe = S.sam_export(index.handle), osam.export()
    for k in oe:
        assert (ex[k] == oe[k]).all(), k


def test_closed_loop_with_committed_tokens_appended():
    """The fused step on a growing index: after every step the tokens some streams committed are appended
    as new sessions, the device copy is synced, the states renormalised."""
    cfg = W.CONFIGS[0].scaled(B=24, steps=12, sessions=6)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    index = S.SamIndex(corpus, [cfg.separator], max_tokens=corpus.shape[0] + 4000, max_token_id=cfg.separator)
    gpu = CudaBackend(cfg, corpus, bits_to_device(noise), index=index)
    cpu = OracleBackend(cfg, corpus, noise.copy())
    f_g, f_o = W.ClosedLoopFeeder(cfg, scripts, rowmax), W.ClosedLoopFeeder(cfg, scripts, rowmax)
    toks, n = f_g.prime_tokens()
    dg, ndg = gpu.prime(toks, n)
    do, ndo = cpu.prime(toks, n)
    assert (dg == do).all() and (ndg == ndo).all()
    committed = [[] for _ in range(cfg.B)]
    for t in range(cfg.steps):
        outs = []
        for be, f, (d, nd) in ((gpu, f_g, (dg, ndg)), (cpu, f_o, (do, ndo))):
            ow = f.overwrites(t, d, nd)
            keep = np.arange(ow["row"].shape[0])
            saved = be.poke(ow["row"], ow["col"], ow["bits"], keep)
            out = be.step(d, nd)
            be.unpoke(ow["row"], ow["col"], saved)
            f.advance(out["n_accepted"])
            outs.append(out)
        g, o = outs
        for k in ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft"):
            assert (g[k] == o[k]).all(), (t, k)
        for b in range(cfg.B):
            committed[b] += [int(x) for x in o["accepted"][b, :o["n_accepted"][b]]]
        # every third step: two streams' output so far becomes part of the shared memory
        if t % 3 == 2:
            piece = []
            for b in (t % cfg.B, (5 * t + 1) % cfg.B):
                piece += [cfg.separator] + committed[b]
            piece = np.array(piece, np.int32)
            cpu.sam.extend(piece)
            cpu.sam.renormalize(cpu.state, cpu.mlen)
            S.sam_extend(index.handle, piece)
            S.sam_sync_renormalize(index.handle, cfg.B, gpu.state, gpu.mlen)
            # the pending drafts came from the text before it grew; both sides re-emit them
            z = np.zeros((cfg.B, 1), np.int32)
            nz = np.zeros(cfg.B, np.int32)
            dg, ndg = gpu.prime(z, nz)
            do, ndo = cpu.prime(z, nz)
            assert (dg == do).all() and (ndg == ndo).all()
        else:
            dg, ndg, do, ndo = g["drafts"], g["n_draft"], o["drafts"], o["n_draft"]


def test_builder_thread_and_empty_start():
    """An index that starts empty drafts nothing; text queued for the builder thread becomes visible only
    after sam_sync; once everything is built and synced the drafts equal the oracle's."""
    rng = np.random.default_rng(3)
    sep, K, mm, B, ld = 500, 5, 2, 16, 10
    index = S.SamIndex(np.zeros(0, np.int32), [sep], max_tokens=50000, max_token_id=sep)
    text = _hub_text(rng, 20000, sep)
    st = torch.zeros(B, dtype=torch.int32, device=DEV)
    ml = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = np.stack([text[s:s + ld] for s in rng.integers(0, text.shape[0] - ld, size=B)]).astype(np.int32)
    n_new = np.full(B, ld, np.int32)
    d = torch.full((B, K), -9, dtype=torch.int32, device=DEV)
    nd = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    S.sam_draft(index.handle, B, st, ml, _i32(toks), ld, _i32(n_new), K, mm, d, nd)
    torch.cuda.synchronize()
    assert int(nd.abs().sum()) == 0 and int(st.abs().sum()) == 0          # nothing indexed yet: no speculation
    for piece in np.array_split(text, 23):
        S.sam_extend(index.handle, piece, wait=False)
    assert S.sam_pending(index.handle)[0] == text.shape[0]
    assert S.sam_pending(index.handle)[2] == 0                            # the device has seen nothing so far
    deadline = time.time() + 60
    seen = 0
    while seen < text.shape[0]:
        seen = S.sam_sync(index.handle)                                   # whatever is finished so far
        assert time.time() < deadline
        time.sleep(0.002)
    osam = oracle.OracleSAM(text, [sep])
    st_o = np.zeros(B, np.int32)
    ml_o = np.zeros(B, np.int32)
    st.zero_(); ml.zero_()
    _draft_both(index, osam, B, st, ml, st_o, ml_o, toks, n_new, K, mm)
    assert (ml_o == ld).all()


def test_updates_pile_up_and_ring_slots_are_reused():
    """The builder thread sends every small update to one of eight slots of the device blob ahead of time.  Twenty
    updates between two syncs overflow the ring: the first eight wait in their slots, the others travel on the
    caller's stream when sam_sync comes, all applied in order.  Then many rounds of a few updates each make every
    slot be used again and again.  After every sync the device copy drafts like the oracle's automaton."""
    rng = np.random.default_rng(23)
    sep, K, mm, B, ld = 1000, 6, 2, 48, 10
    text = _hub_text(rng, 1500, sep)
    index = S.SamIndex(text, [sep], max_tokens=60000, max_token_id=sep + 50)
    osam = oracle.OracleSAM(text, [sep])
    st = torch.zeros(B, dtype=torch.int32, device=DEV)
    ml = torch.zeros(B, dtype=torch.int32, device=DEV)
    st_o = np.zeros(B, np.int32)
    ml_o = np.zeros(B, np.int32)
    bursts = [20] + [3, 1, 5, 2] * 6
    for rnd, n_updates in enumerate(bursts):
        inc0, full0, _ = S.sam_update_stats(index.handle)
        for _ in range(n_updates):
            piece = np.concatenate([[sep], _hub_text(rng, int(rng.integers(5, 120)), sep)]).astype(np.int32)
            osam.extend(piece)
            S.sam_extend(index.handle, piece)              # waits for the builder thread: one update per piece
        osam.renormalize(st_o, ml_o)
        if rnd % 2 == 0:
            assert S.sam_sync_renormalize(index.handle, B, st, ml) == osam.n
        else:
            assert S.sam_sync(index.handle) == osam.n
            S.sam_renormalize(index.handle, B, st, ml)
        inc1, full1, _ = S.sam_update_stats(index.handle)
        assert (inc1 - inc0) + (full1 - full0) == n_updates
        toks = np.empty((B, ld), np.int32)
        for b in range(B):
            start = int(rng.integers(0, osam.n - ld))
            toks[b] = osam.corpus[start:start + ld]
        toks[rng.random((B, ld)) < 0.05] = sep + 9
        n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
        _draft_both(index, osam, B, st, ml, st_o, ml_o, toks, n_new, K, mm)
    ex, oe = S.sam_export(index.handle), osam.export()
    for k in oe:
        assert (ex[k] == oe[k]).all(), k


def test_sync_without_pending_updates_launches_nothing():
    rng = np.random.default_rng(4)
    sep = 500
    index = S.SamIndex(_hub_text(rng, 800, sep), [sep], max_tokens=4000, max_token_id=sep)
    st = torch.zeros(8, dtype=torch.int32, device=DEV)
    ml = torch.zeros(8, dtype=torch.int32, device=DEV)
    n0 = S.sam_launch_count()
    assert S.sam_sync_renormalize(index.handle, 8, st, ml) == 800
    assert S.sam_launch_count() == n0


def test_small_and_large_updates_take_their_own_paths():
    """Updates of a few hundred tokens go through one page-locked buffer, one copy and one kernel; an update of
    tens of thousands of tokens is too large for that buffer and is applied section by section.  Both leave the
    device copy equal to the oracle's automaton (drafts, states and matched lengths of streams that read all over
    the grown text), whichever order they come in."""
    rng = np.random.default_rng(11)
    sep, K, mm, B, ld = 1000, 6, 2, 64, 12
    text = _hub_text(rng, 2000, sep)
    index = S.SamIndex(text, [sep], max_tokens=120000, max_token_id=sep + 50)
    osam = oracle.OracleSAM(text, [sep])
    st = torch.zeros(B, dtype=torch.int32, device=DEV)
    ml = torch.zeros(B, dtype=torch.int32, device=DEV)
    st_o = np.zeros(B, np.int32)
    ml_o = np.zeros(B, np.int32)
    sizes = [300, 40000, 150, 25000, 60, 1]
    for rnd, n in enumerate(sizes):
        piece = _hub_text(rng, n, sep)
        osam.extend(piece)
        inc0, full0, bytes0 = S.sam_update_stats(index.handle)
        S.sam_extend(index.handle, piece)
        if rnd < 3:
            assert S.sam_sync(index.handle) == osam.n
            S.sam_renormalize(index.handle, B, st, ml)
        else:                                   # one call; after a large update the states get a kernel of their own
            assert S.sam_sync_renormalize(index.handle, B, st, ml) == osam.n
        inc1, full1, bytes1 = S.sam_update_stats(index.handle)
        assert inc1 + full1 > inc0 + full0
        if n >= 25000:
            assert bytes1 - bytes0 > (1 << 20)          # more than the page-locked buffer holds
        elif full1 == full0:
            assert bytes1 - bytes0 < (1 << 20)
        osam.renormalize(st_o, ml_o)
        toks = np.empty((B, ld), np.int32)
        for b in range(B):
            start = int(rng.integers(0, osam.n - ld))
            toks[b] = osam.corpus[start:start + ld]
        toks[rng.random((B, ld)) < 0.05] = sep + 7
        n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
        _draft_both(index, osam, B, st, ml, st_o, ml_o, toks, n_new, K, mm)
    ex, oe = S.sam_export(index.handle), osam.export()
    for k in oe:
        assert (ex[k] == oe[k]).all(), k
