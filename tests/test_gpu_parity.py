"""Parity of the CUDA path (through the C ABI) with the CPU oracle, tolerance 0.

Everything here needs a GPU.  bf16 values are compared as bit patterns / exact indices."""
from __future__ import annotations

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


def _verify_gpu(bits: np.ndarray, V, B, K, drafts, n_draft, dev_tensor=None, variant=0):
    """bits: [B*(K+1), stride] uint16 host. Returns argmax, accepted, n_accepted (numpy)."""
    lg = bits_to_device(bits) if dev_tensor is None else dev_tensor
    stride = bits.shape[1]
    am = torch.full((B, K + 1), -9, dtype=torch.int32, device=DEV)
    acc = torch.full((B, K + 1), -9, dtype=torch.int32, device=DEV)
    nacc = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    wsb = S.sam_workspace_bytes(B, K)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    S.sam_workspace_init(ws, wsb)
    d, nd = _i32(drafts), _i32(n_draft)
    S.sam_set_argmax_variant(variant)
    try:
        for _ in range(2):   # twice: the scratch must come back ready for the next call
            S.sam_verify(lg, stride, B, K, V, d, nd, am, acc, nacc, ws, wsb)
        torch.cuda.synchronize()
    finally:
        S.sam_set_argmax_variant(0)
    assert S.sam_workspace_status(ws, B, K) == 0
    # the per-row words (first in the scratch) are zero again; the rest may hold bookkeeping that outlives a call (a row
    # list for the next step, the count of launches)
    assert int(ws[:B * (K + 1) * 8].to(torch.int32).abs().sum()) == 0
    return am.cpu().numpy(), acc.cpu().numpy(), nacc.cpu().numpy()


def _check_verify(bits, V, B, K, rng):
    am_o = oracle.argmax_batch(bits, V=V, threads=oracle.host_threads()).reshape(B, K + 1)
    n_draft = rng.integers(0, K + 1, size=B).astype(np.int32)
    drafts = np.full((B, K), -1, np.int32)
    for b in range(B):
        nd = n_draft[b]
        keep = rng.random(nd) < 0.8
        drafts[b, :nd] = np.where(keep, am_o[b, :nd], rng.integers(0, V, size=nd))
    acc_o, nacc_o = oracle.accept_batch(drafts, n_draft, am_o)
    # 0: chosen by alignment and size (these small cases: direct loads); 1: direct loads always;
    # 2: bulk-copy pipeline (when rows are 16-byte aligned) with the accept step inside the same kernel;
    # 3: bulk-copy pipeline followed by the accept kernel
    for variant in (0, 1, 2, 3):
        am, acc, nacc = _verify_gpu(bits, V, B, K, drafts, n_draft, variant=variant)
        assert (am == am_o).all(), variant
        assert (nacc == nacc_o).all() and (acc == acc_o).all(), variant


@pytest.mark.parametrize("V,pad,B,K", [
    (1, 0, 3, 1), (7, 0, 3, 2), (8, 0, 2, 3), (9, 7, 5, 4), (1000, 0, 4, 8), (1000, 3, 4, 8),
    (4097, 0, 6, 5), (4097, 8, 6, 5), (50257, 0, 3, 7), (50257, 1, 3, 7), (151936, 0, 2, 8),
    (151936, 8, 3, 32), (8192 * 3, 0, 40, 16), (8191, 1, 33, 31), (8192 * 13 + 24, 0, 7, 3), (8192 * 12, 8, 9, 2),
    (3, 5, 300, 1), (8200, 0, 1, 1), (1000003, 5, 2, 3), (1 << 20, 0, 1, 1), (8192 * 25 + 5, 3, 2, 2), (32768 * 3, 0, 5, 2), (32768 * 2 + 8, 0, 4, 1), (32768 * 2 - 3, 3, 4, 1),
])
def test_verify_parity_shapes(V, pad, B, K):
    """Row lengths around vector/tile edges, misaligned row strides, every K edge."""
    rng = np.random.default_rng(V * 31 + pad)
    R = B * (K + 1)
    bits = W.f32_to_bf16_bits(rng.standard_normal((R, V + pad), dtype=np.float32))
    if pad:
        bits[:, V:] = 0x7F00      # huge finite values beyond V must be ignored
    _check_verify(bits, V, B, K, rng)


def test_verify_parity_special_values():
    """Ties at every distance, -0/+0, infinities, NaNs, all-equal rows, maxima at the row ends."""
    rng = np.random.default_rng(5)
    V, B, K = 20011, 8, 7
    R = B * (K + 1)
    f = rng.standard_normal((R, V)).astype(np.float32)
    bits = W.f32_to_bf16_bits(f)
    top = np.uint16(0x4120)   # 10.0
    bits[0, V - 1] = top
    bits[1, 0] = top
    bits[2, [5, V - 1]] = top
    bits[3, [8191, 8192]] = top
    bits[4, [7, 8]] = top
    bits[5, :] = 0x0000; bits[5, 3] = 0x8000                       # +0 everywhere, one -0
    bits[6, :] = 0x8000; bits[6, 100] = 0x0000                     # -0 everywhere, one +0 -> index 0 (equal)
    bits[7, :] = 0xFF80                                            # all -inf
    bits[8, :] = 0xFF80; bits[8, 777] = 0xC2C8                     # -inf and one -100
    bits[9, 4000] = 0x7F80; bits[9, 9000] = 0x7F80                 # two +inf
    bits[10, 17] = 0x7FC0; bits[10, 18] = 0xFFC0                   # NaNs inside the row
    bits[11, 0] = 0x7FC0                                           # NaN first: index 0
    bits[12, :] = 0x7FC0                                           # all NaN
    bits[13, :] = 0x7FC0; bits[13, 0] = 0xFF80                     # -inf then NaNs
    bits[14, :] = 0x7FC0; bits[14, 123] = 0x3F80; bits[14, 0] = 0xBF80   # numbers among NaNs
    bits[15, :] = 0x3F80                                           # all equal
    bits[16, :] = 0xBF80; bits[16, V - 1] = 0xBF00                 # all -1, last -0.5
    _check_verify(bits, V, B, K, rng)


def test_verify_parity_natural_and_planted_ties():
    """N(0,1) rows at full vocabulary: bf16 ties at the maximum are common; plus planted ties."""
    rng = np.random.default_rng(9)
    V, B, K = 151936, 8, 8
    bits = W.f32_to_bf16_bits(rng.standard_normal((B * (K + 1), V), dtype=np.float32))
    for r in range(0, bits.shape[0], 3):
        m = W.bf16_bits_to_f32(bits[r]).max()
        extra = rng.integers(0, V, size=2)
        bits[r, extra] = W.f32_to_bf16_bits(np.array([m], np.float32))[0]
    _check_verify(bits, V, B, K, rng)


def test_verify_on_a_strided_view():
    """Logits that are a column slice of a wider tensor (row stride > V, base not 16-byte aligned)."""
    rng = np.random.default_rng(11)
    V, B, K = 3001, 4, 3
    wide = W.f32_to_bf16_bits(rng.standard_normal((B * (K + 1), V + 37), dtype=np.float32))
    lg = bits_to_device(wide)
    view_ptr = lg.data_ptr() + 2 * 5          # start at column 5
    am_o = oracle.argmax_batch(wide[:, 5:], V=V).reshape(B, K + 1)
    drafts = am_o[:, :K].copy()
    n_draft = np.full(B, K, np.int32)
    am = torch.zeros((B, K + 1), dtype=torch.int32, device=DEV)
    acc = torch.zeros((B, K + 1), dtype=torch.int32, device=DEV)
    nacc = torch.zeros((B,), dtype=torch.int32, device=DEV)
    wsb = S.sam_workspace_bytes(B, K)
    ws = torch.zeros(wsb, dtype=torch.uint8, device=DEV)
    S.sam_verify(view_ptr, V + 37, B, K, V, _i32(drafts), _i32(n_draft), am, acc, nacc, ws, wsb)
    torch.cuda.synchronize()
    assert (am.cpu().numpy() == am_o).all()
    assert (nacc.cpu().numpy() == K + 1).all() and (acc.cpu().numpy() == am_o).all()


# ------------------------------------------------------------------ draft
def _draft_gpu(index, B, state, mlen, toks, n_new, K, mm):
    st, ml = _i32(state), _i32(mlen)
    d = torch.full((B, K), -9, dtype=torch.int32, device=DEV)
    nd = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    t = _i32(toks)
    S.sam_draft(index.handle, B, st, ml, t, toks.shape[1], _i32(n_new), K, mm, d, nd)
    torch.cuda.synchronize()
    return st.cpu().numpy(), ml.cpu().numpy(), d.cpu().numpy(), nd.cpu().numpy()


def test_draft_open_loop_tiny():
    """Tiny config as written: 16 steps of 1..9 tokens per stream, every output compared."""
    cfg = W.CONFIGS[0]
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    toks, n_new = W.make_open_loop_feed(cfg, scripts)
    index = S.SamIndex(corpus, [cfg.separator])
    osam = oracle.OracleSAM(corpus, [cfg.separator])
    st = np.zeros(cfg.B, np.int32); ml = np.zeros(cfg.B, np.int32)
    st_o = st.copy(); ml_o = ml.copy()
    for t in range(cfg.steps):
        d_o, nd_o = osam.draft_batch(st_o, ml_o, toks[t], n_new[t], cfg.K, cfg.min_match)
        st, ml, d, nd = _draft_gpu(index, cfg.B, st, ml, toks[t], n_new[t], cfg.K, cfg.min_match)
        assert (st == st_o).all() and (ml == ml_o).all()
        assert (nd == nd_o).all() and (d == d_o).all()


@pytest.mark.parametrize("K,mm", [(1, 1), (5, 2), (32, 1), (17, 4)])
def test_draft_random_feeds(K, mm):
    """Hub tokens (wide rows on every search depth), separators and unseen ids in the feed,
    empty feeds, feeds longer than a warp, drafts cut at separators and at the corpus end."""
    rng = np.random.default_rng(K)
    sep = 5000
    parts = []
    for s in range(6):
        body = rng.integers(0, 3000, size=3000).astype(np.int32)
        body[::3] = rng.integers(0, 3, size=body[::3].shape[0])         # three hub tokens with ~1000+ successors
        body[1::50] = 7                                                  # a medium hub (33..1024 successors)
        parts += [body, np.array([sep], np.int32)]
    corpus = np.concatenate(parts[:-1])
    index = S.SamIndex(corpus, [sep])
    osam = oracle.OracleSAM(corpus, [sep])
    B, ld = 64, 70
    st = np.zeros(B, np.int32); ml = np.zeros(B, np.int32)
    st_o = st.copy(); ml_o = ml.copy()
    for step in range(6):
        toks = np.empty((B, ld), np.int32)
        n_new = rng.integers(0, ld + 1, size=B).astype(np.int32)
        n_new[rng.random(B) < 0.15] = 0
        for b in range(B):
            pos = 0
            while pos < ld:
                span = int(rng.integers(1, 40))
                start = int(rng.integers(0, corpus.shape[0] - span))
                if rng.random() < 0.2:
                    start = corpus.shape[0] - span                      # spans that run into the corpus end
                take = min(span, ld - pos)
                toks[b, pos:pos + take] = corpus[start:start + take]
                pos += take
            noise = rng.random(ld) < 0.05
            toks[b, noise] = rng.choice(np.array([-1, -7, 4000, sep, 2 ** 30, 1], np.int32), size=int(noise.sum()))
        d_o, nd_o = osam.draft_batch(st_o, ml_o, toks, n_new, K, mm)
        st, ml, d, nd = _draft_gpu(index, B, st, ml, toks, n_new, K, mm)
        assert (st == st_o).all() and (ml == ml_o).all()
        assert (nd == nd_o).all() and (d == d_o).all()
    assert (nd_o == 0).any() and (nd_o == K).any()


@pytest.mark.parametrize("n_sep", [0, 1, 16])
def test_draft_with_no_one_and_sixteen_separators(n_sep):
    """The largest number of separator ids, a single one, and none at all (drafts then only end at the corpus end)."""
    rng = np.random.default_rng(40 + n_sep)
    corpus = rng.integers(0, 60, size=5000).astype(np.int32)
    seps = list(range(100, 100 + n_sep))
    if n_sep:
        corpus[rng.integers(0, 5000, size=400)] = rng.choice(np.array(seps, np.int32), size=400)
    index = S.SamIndex(corpus, seps)
    osam = oracle.OracleSAM(corpus, seps if n_sep else np.zeros(0, np.int32))
    B, ld, K, mm = 40, 8, 12, 1
    st = np.zeros(B, np.int32); ml = np.zeros(B, np.int32)
    st_o = st.copy(); ml_o = ml.copy()
    cut_short = 0
    for step in range(4):
        starts = rng.integers(0, 5000 - ld, size=B)
        starts[:4] = 5000 - ld                                   # runs into the corpus end
        toks = np.stack([corpus[s0:s0 + ld] for s0 in starts]).astype(np.int32)
        n_new = rng.integers(1, ld + 1, size=B).astype(np.int32)
        d_o, nd_o = osam.draft_batch(st_o, ml_o, toks, n_new, K, mm)
        st, ml, d, nd = _draft_gpu(index, B, st, ml, toks, n_new, K, mm)
        assert (st == st_o).all() and (ml == ml_o).all() and (nd == nd_o).all() and (d == d_o).all()
        cut_short += int(((nd_o < K) & (ml_o >= mm)).sum())
    assert cut_short > 0


def test_draft_rejects_foreign_state():
    """A (state, matched_len) pair outside the automaton restarts from the root instead of faulting."""
    corpus = np.array([1, 2, 3, 1, 2, 4], np.int32)
    index = S.SamIndex(corpus, [9])
    osam = oracle.OracleSAM(corpus, [9])
    toks = np.array([[1, 2], [1, 2]], np.int32)
    n_new = np.array([2, 2], np.int32)
    st, ml, d, nd = _draft_gpu(index, 2, np.array([10 ** 6, -5], np.int32), np.array([3, 3], np.int32), toks, n_new, 3, 1)
    so, lo = osam.walk(0, 0, [1, 2])
    do, ndo = osam.draft(so, lo, 3, 1)
    assert (st == so).all() and (ml == lo).all() and (nd == ndo).all() and (d == do[None, :]).all()


# ------------------------------------------------------------------ closed loop
def _closed_loop_pair(cfg, steps=None, threads=None):
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    threads = oracle.host_threads() if threads is None else threads
    tr_o = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax),
                             OracleBackend(cfg, corpus, noise.copy(), threads), steps)
    tr_g = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax),
                             CudaBackend(cfg, corpus, bits_to_device(noise)), steps)
    return tr_o, tr_g


def _assert_traces_equal(tr_o, tr_g):
    assert len(tr_o) == len(tr_g)
    for t, (o, g) in enumerate(zip(tr_o, tr_g)):
        for k in ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft"):
            assert (o[k] == g[k]).all(), (t, k)


def test_closed_loop_tiny():
    cfg = W.CONFIGS[0]
    tr_o, tr_g = _closed_loop_pair(cfg)
    _assert_traces_equal(tr_o, tr_g)
    st = W.trace_stats(cfg, tr_g)
    assert st["ote"] > 1.3


def test_closed_loop_cfg1_full():
    """Config 1 at its full size: 1M-token corpus, B=64, K=8, V=151,936, all 64 steps."""
    cfg = W.CONFIGS[1]
    tr_o, tr_g = _closed_loop_pair(cfg)
    _assert_traces_equal(tr_o, tr_g)


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_closed_loop_other_kernel_variants(variant):
    """The step with direct loads (full walk in the accept kernel) and with the accept step inside the
    bulk-copy argmax kernel gives the same trace as the oracle."""
    cfg = W.CONFIGS[2].scaled(sessions=64, B=300, steps=6)
    S.sam_set_argmax_variant(variant)
    try:
        tr_o, tr_g = _closed_loop_pair(cfg)
    finally:
        S.sam_set_argmax_variant(0)
    _assert_traces_equal(tr_o, tr_g)


def test_closed_loop_many_streams_per_cta():
    """Short rows and many streams: every CTA finishes dozens of streams inside the argmax kernel."""
    cfg = W.CONFIGS[0].scaled(B=3000, K=2, steps=5, vocab=1000)
    S.sam_set_argmax_variant(2)
    try:
        tr_o, tr_g = _closed_loop_pair(cfg)
    finally:
        S.sam_set_argmax_variant(0)
    _assert_traces_equal(tr_o, tr_g)


@pytest.mark.parametrize("i,kw", [
    (2, dict(sessions=256, B=48, steps=12)),
    (3, dict(sessions=128, B=40, steps=8)),
    (4, dict(sessions=64, B=24, steps=8)),
])
def test_closed_loop_scaled_configs(i, kw):
    """Configs 2-4 with their own K / min_match / vocabulary / span recipe, fewer sessions and streams."""
    cfg = W.CONFIGS[i].scaled(**kw)
    tr_o, tr_g = _closed_loop_pair(cfg)
    _assert_traces_equal(tr_o, tr_g)


def _colliding_tokens(log2cap, count, limit=1 << 20):
    """Token ids whose home slot in a hash row of 2^log2cap slots is the same (multiplicative hashing with the
    golden-ratio constant - the row layout documented for states with more than 32 transitions)."""
    tok = np.arange(1, limit, dtype=np.uint64)
    home = ((tok * np.uint64(0x9E3779B1)) & np.uint64(0xFFFFFFFF)) >> np.uint64(32 - log2cap)
    same = tok[home == home[0]][:count]
    assert same.shape[0] == count
    return same.astype(np.int32)


@pytest.mark.parametrize("growing", [False, True])
def test_hash_row_with_a_probe_run_longer_than_one_window(growing):
    """A hub state whose 40 successors all hash to the same slot: the lookup has to go on into a second
    32-slot window, both for successors that are there and for a token that is not."""
    log2cap = 8 if growing else 7            # 40 transitions: 128 slots in a fixed index, 256 in a growing one
    succ = _colliding_tokens(log2cap, 41)
    present, absent = succ[:40], int(succ[40])
    hub, sep = 5, 3
    corpus = np.empty(2 * 40, np.int32)
    corpus[0::2] = hub
    corpus[1::2] = present
    if growing:
        index = S.SamIndex(corpus[:20], [sep], max_tokens=1000, max_token_id=int(succ.max()))
        S.sam_extend(index.handle, corpus[20:])
        S.sam_sync(index.handle)
    else:
        index = S.SamIndex(corpus, [sep])
    osam = oracle.OracleSAM(corpus, [sep])
    ex = osam.export()
    s_hub, _ = osam.walk(0, 0, [hub])
    assert ex["row_ptr"][s_hub + 1] - ex["row_ptr"][s_hub] == 40
    B = 42
    toks = np.full((B, 2), hub, np.int32)
    toks[:40, 1] = present
    toks[40, 1] = absent                     # same home slot, not a successor: falls back through the suffix link
    toks[41, 1] = hub
    n_new = np.full(B, 2, np.int32)
    st = np.zeros(B, np.int32); ml = np.zeros(B, np.int32)
    st_o = st.copy(); ml_o = ml.copy()
    d_o, nd_o = osam.draft_batch(st_o, ml_o, toks, n_new, 4, 1)
    st, ml, d, nd = _draft_gpu(index, B, st, ml, toks, n_new, 4, 1)
    assert (st == st_o).all() and (ml == ml_o).all() and (nd == nd_o).all() and (d == d_o).all()
    assert (ml_o[:40] == 2).all() and ml_o[40] == 0


def test_two_host_threads_on_two_streams():
    """Two host threads drive two independent closed loops at once, each on a stream and a scratch of its own, over
    one shared automaton: calls from several threads are allowed as long as they do not share scratch or outputs."""
    import threading
    cfgs = [W.CONFIGS[2].scaled(sessions=64, B=40, steps=10), W.CONFIGS[2].scaled(sessions=64, B=24, steps=10, seed=77)]
    corpus = W.make_corpus(cfgs[0])                      # one text; the second loop differs in streams, scripts and logits
    index = S.SamIndex(corpus, [cfgs[0].separator])
    want, got, errors = [None, None], [None, None], []
    inputs = []
    for cfg in cfgs:
        scripts = W.make_scripts(cfg, corpus)
        noise = W.make_noise_logits(cfg)
        rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
        inputs.append((scripts, noise, rowmax))
    for i, cfg in enumerate(cfgs):
        scripts, noise, rowmax = inputs[i]
        want[i] = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax),
                                    OracleBackend(cfg, corpus, noise.copy(), oracle.host_threads()), None)

    def worker(i):
        try:
            cfg = cfgs[i]
            scripts, noise, rowmax = inputs[i]
            with torch.cuda.stream(torch.cuda.Stream()):
                be = CudaBackend(cfg, corpus, bits_to_device(noise), index=index)
                for _ in range(3):                       # several loops per thread: more chances to collide
                    be.state.zero_(); be.mlen.zero_()
                    got[i] = W.run_closed_loop(cfg, W.ClosedLoopFeeder(cfg, scripts, rowmax), be, None)
                    assert be.status() == 0
                    _assert_traces_equal(want[i], got[i])
        except BaseException as e:                       # reported by the main thread
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
