"""Composite drafting over several automata on the GPU against the oracle, tolerance 0 (the choice
between slots compares float32 products on both sides)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import paper_2512_18337_b200 as S
import workload as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(x, dtype):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=dtype)).to(DEV)


def _corpus(rng, n, sep):
    body = rng.integers(0, 300, size=n).astype(np.int32)
    body[::4] = rng.integers(0, 4, size=body[::4].shape[0])
    body[7::61] = sep
    return body


def test_multi_draft_parity_with_growth_and_verification():
    rng = np.random.default_rng(4)
    sep, B, M, K, mm, ld = 999, 60, 4, 6, 2, 9
    corpora = [_corpus(rng, n, sep) for n in (4000, 2500, 6000, 1500, 3000)]
    members_o = [oracle.OracleSAM(c, [sep]) for c in corpora]
    members_g = [S.SamIndex(c, [sep]) for c in corpora[:4]]
    members_g.append(S.SamIndex(corpora[4], [sep], max_tokens=20000, max_token_id=sep))       # this one grows
    sset = S.SamSet(members_g)
    slots = rng.integers(-1, 5, size=(B, M)).astype(np.int32)
    slots[0] = -1                                                        # a stream without any automaton
    slots[1] = [4, 4, -1, 0]                                             # the same member twice
    weights = rng.choice(np.array([0.2, 0.5, 1.0, 1.0, 1.3], np.float32), size=(B, M)).astype(np.float32)
    st_o = np.zeros((B, M), np.int32); ml_o = np.zeros((B, M), np.int32)
    st = torch.zeros((B, M), dtype=torch.int32, device=DEV)
    ml = torch.zeros((B, M), dtype=torch.int32, device=DEV)
    d = torch.full((B, K), -9, dtype=torch.int32, device=DEV)
    nd = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    ch = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    sl_d, w_d = _dev(slots, np.int32), _dev(weights, np.float32)
    V = 1000
    wsb = S.sam_workspace_bytes(B, K)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    S.sam_workspace_init(ws, wsb)
    am = torch.zeros((B, K + 1), dtype=torch.int32, device=DEV)
    acc = torch.zeros((B, K + 1), dtype=torch.int32, device=DEV)
    nacc = torch.zeros((B,), dtype=torch.int32, device=DEV)
    toks = np.empty((B, ld), np.int32)
    n_new = np.empty(B, np.int32)
    seen_slots = set()
    for step in range(16):
        if step % 2 == 0 or step < 3:
            # feed spans of a random member (so that different slots lead), a few unknown tokens mixed in
            for b in range(B):
                c = members_o[int(rng.integers(0, 5))].corpus
                s0 = int(rng.integers(0, c.shape[0] - ld))
                toks[b] = c[s0:s0 + ld]
                noise = rng.random(ld) < 0.06
                toks[b, noise] = rng.integers(0, 1200, size=int(noise.sum()))
            n_new[:] = rng.integers(0, ld + 1, size=B)
            t_d, n_d, cur_ld = _dev(toks, np.int32), _dev(n_new, np.int32), ld
            t_o, n_o = toks.copy(), n_new.copy()
        else:
            # verification round: logits that accept a random prefix of the draft, then the accepted tokens are fed
            bits = W.f32_to_bf16_bits(rng.standard_normal((B * (K + 1), V), dtype=np.float32))
            for b in range(B):
                for j in range(int(nd_o[b])):
                    if rng.random() < 0.7:
                        bits[b * (K + 1) + j, d_o[b, j]] = 0x4200
            lg = torch.from_numpy(bits.view(np.int16)).to(DEV).view(torch.bfloat16)
            S.sam_verify(lg, V, B, K, V, d, nd, am, acc, nacc, ws, wsb)
            torch.cuda.synchronize()
            am_o = oracle.argmax_batch(bits).reshape(B, K + 1)
            acc_o, nacc_o = oracle.accept_batch(d_o, nd_o, am_o)
            assert (acc.cpu().numpy() == acc_o).all() and (nacc.cpu().numpy() == nacc_o).all()
            t_d, n_d, cur_ld = acc, nacc, K + 1
            t_o, n_o = acc_o, nacc_o
        S.sam_multi_draft(sset.handle, B, M, sl_d, w_d, st, ml, t_d, cur_ld, n_d, K, mm, d, nd, ch)
        torch.cuda.synchronize()
        d_o, nd_o, ch_o = oracle.multi_draft(members_o, slots, weights, st_o, ml_o, t_o, n_o, K, mm)
        assert (st.cpu().numpy() == st_o).all() and (ml.cpu().numpy() == ml_o).all()
        assert (ch.cpu().numpy() == ch_o).all()
        assert (nd.cpu().numpy() == nd_o).all() and (d.cpu().numpy() == d_o).all()
        seen_slots |= set(int(x) for x in ch_o)
        if step == 7:
            # the fifth member grows; its view in the table is refreshed and its slots' states renormalised
            piece = np.concatenate([[sep], _corpus(rng, 1500, sep)]).astype(np.int32)
            members_o[4].extend(piece)
            S.sam_extend(members_g[4].handle, piece)
            S.sam_sync(members_g[4].handle)
            sset.refresh()
            for m in range(M):
                own = np.nonzero(slots[:, m] == 4)[0]          # only these states belong to the member that grew
                col_o = np.ascontiguousarray(st_o[own, m])
                members_o[4].renormalize(col_o, np.ascontiguousarray(ml_o[own, m]))
                st_o[own, m] = col_o
            sset.renormalize(4, B, M, sl_d, st, ml)
            torch.cuda.synchronize()
            assert (st.cpu().numpy() == st_o).all()
    assert seen_slots >= {-1, 0, 1, 2, 3}


def test_multi_draft_argument_checks():
    lib = S.binding._load()
    assert lib.sam_set_bytes(0) == -1 and lib.sam_set_bytes(3) % 256 == 0
    ix = S.SamIndex(np.array([1, 2, 3, 1, 2], np.int32), [9])
    sset = S.SamSet([ix])
    z = torch.zeros(8, dtype=torch.int32, device=DEV)
    f = torch.ones(8, dtype=torch.float32, device=DEV)
    args = (z.data_ptr(), f.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), 1, z.data_ptr())
    assert lib.sam_multi_draft(sset.handle, 1, 9, *args, 2, 1, z.data_ptr(), z.data_ptr(), z.data_ptr(), None) == -1   # M > 8
    assert lib.sam_multi_draft(sset.handle, 0, 1, *args, 2, 1, z.data_ptr(), z.data_ptr(), z.data_ptr(), None) == 0    # B = 0


@pytest.mark.parametrize("variant", [0, 1])
def test_multi_step_closed_loop(variant):
    """The fused composite step (argmax with every slot's walk-ahead riding along, accept, per-slot resume,
    slot choice, next draft) against the oracle's accept followed by its composite drafting.  Variant 1 takes
    the direct-load argmax kernel, which has no walk-ahead: the slots then walk the whole accepted run."""
    rng = np.random.default_rng(11)
    sep, B, M, K, mm, V = 999, 70, 3, 7, 2, 4096
    corpora = [_corpus(rng, n, sep) for n in (5000, 3000, 4000, 2000)]
    members_o = [oracle.OracleSAM(c, [sep]) for c in corpora]
    sset = S.SamSet([S.SamIndex(c, [sep]) for c in corpora])
    slots = rng.integers(-1, 4, size=(B, M)).astype(np.int32)
    slots[0] = -1
    weights = rng.choice(np.array([0.5, 1.0, 1.0, 2.0], np.float32), size=(B, M)).astype(np.float32)
    st_o = np.zeros((B, M), np.int32); ml_o = np.zeros((B, M), np.int32)
    i32 = dict(dtype=torch.int32, device=DEV)
    st, ml = torch.zeros((B, M), **i32), torch.zeros((B, M), **i32)
    d, nd, ch = torch.full((B, K), -9, **i32), torch.full((B,), -9, **i32), torch.full((B,), -9, **i32)
    am, acc, nacc = torch.zeros((B, K + 1), **i32), torch.zeros((B, K + 1), **i32), torch.zeros(B, **i32)
    sl_d, w_d = _dev(slots, np.int32), _dev(weights, np.float32)
    wsb = S.sam_multi_workspace_bytes(B, K, M)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    S.sam_workspace_init(ws, wsb)
    # prime every stream with a span of some member
    toks = np.stack([members_o[int(rng.integers(0, 4))].corpus[s0:s0 + 10] for s0 in rng.integers(0, 1900, size=B)]).astype(np.int32)
    n_new = np.full(B, 10, np.int32)
    S.sam_multi_draft(sset.handle, B, M, sl_d, w_d, st, ml, _dev(toks, np.int32), 10, _dev(n_new, np.int32), K, mm, d, nd, ch)
    d_o, nd_o, ch_o = oracle.multi_draft(members_o, slots, weights, st_o, ml_o, toks, n_new, K, mm)
    torch.cuda.synchronize()
    assert (d.cpu().numpy() == d_o).all() and (nd.cpu().numpy() == nd_o).all()
    S.sam_set_argmax_variant(variant)
    try:
        full_accepts = 0
        for step in range(10):
            bits = W.f32_to_bf16_bits(rng.standard_normal((B * (K + 1), V), dtype=np.float32))
            for b in range(B):
                for j in range(int(nd_o[b]) + 1):
                    # the "model" mostly continues the winning member's text, sometimes goes its own way
                    if j < nd_o[b] and rng.random() < 0.8:
                        bits[b * (K + 1) + j, d_o[b, j]] = 0x4200
                    elif rng.random() < 0.5:
                        c = members_o[int(rng.integers(0, 4))].corpus
                        bits[b * (K + 1) + j, int(c[int(rng.integers(0, c.shape[0]))])] = 0x4200
            lg = torch.from_numpy(bits.view(np.int16)).to(DEV).view(torch.bfloat16)
            S.sam_multi_step(sset.handle, lg, V, B, K, V, d, nd, am, acc, nacc, M, sl_d, w_d, st, ml, mm, d, nd, ch, ws, wsb)
            torch.cuda.synchronize()
            am_o = oracle.argmax_batch(bits).reshape(B, K + 1)
            acc_o, nacc_o = oracle.accept_batch(d_o, nd_o, am_o)
            full_accepts += int(((nacc_o - 1 == nd_o) & (nd_o > 0)).sum())
            d_o, nd_o, ch_o = oracle.multi_draft(members_o, slots, weights, st_o, ml_o, acc_o, nacc_o, K, mm)
            assert (am.cpu().numpy() == am_o).all(), step
            assert (acc.cpu().numpy() == acc_o).all() and (nacc.cpu().numpy() == nacc_o).all(), step
            assert (st.cpu().numpy() == st_o).all() and (ml.cpu().numpy() == ml_o).all(), step
            assert (ch.cpu().numpy() == ch_o).all(), step
            assert (nd.cpu().numpy() == nd_o).all() and (d.cpu().numpy() == d_o).all(), step
        assert full_accepts > 0
    finally:
        S.sam_set_argmax_variant(0)
