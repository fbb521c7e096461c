"""Step options on the GPU against the oracle, tolerance 0: speculation switched off for a step
(the adaptive switch), verification restricted to the rows a proposal uses, and the running
OTE / SHR counters."""
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
KEYS = ("argmax", "accepted", "n_accepted", "state", "matched_len", "drafts", "n_draft")


def _i32(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)


@pytest.mark.parametrize("V,pad,B,K", [(1000, 0, 5, 8), (4097, 3, 7, 4), (151936, 0, 3, 16), (151936, 8, 40, 2),
                                       (8192 * 13 + 24, 0, 9, 5), (7, 0, 300, 1), (65536, 0, 2, 32)])
@pytest.mark.parametrize("variant", [0, 1, 3])
def test_verify_skipping_unused_rows(V, pad, B, K, variant):
    rng = np.random.default_rng(V + B + K)
    R = B * (K + 1)
    bits = W.f32_to_bf16_bits(rng.standard_normal((R, V + pad), dtype=np.float32))
    if pad:
        bits[:, V:] = 0x7F00
    am_all = oracle.argmax_batch(bits, V=V, threads=oracle.host_threads()).reshape(B, K + 1)
    n_draft = rng.integers(-1, K + 2, size=B).astype(np.int32)          # out-of-range counts are clamped
    n_draft[0] = 0
    nd = np.clip(n_draft, 0, K)
    drafts = np.where(rng.random((B, K)) < 0.8, am_all[:, :K], rng.integers(0, V, size=(B, K))).astype(np.int32)
    acc_o, nacc_o = oracle.accept_batch(drafts, nd, am_all)
    lg = bits_to_device(bits)
    outs = [torch.full(s, -9, dtype=torch.int32, device=DEV) for s in ((B, K + 1), (B, K + 1), (B,))]
    cnt = torch.zeros(S.SAM_N_COUNTERS, dtype=torch.int64, device=DEV)
    wsb = S.sam_workspace_bytes(B, K)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    S.sam_workspace_init(ws, wsb)
    S.sam_set_argmax_variant(variant)
    try:
        for _ in range(2):
            S.sam_verify_ex(lg, V + pad, B, K, V, _i32(drafts), _i32(n_draft), *outs,
                            S.SAM_STEP_SKIP_UNUSED_ROWS, cnt, ws, wsb)
        torch.cuda.synchronize()
    finally:
        S.sam_set_argmax_variant(0)
    am, acc, nacc = (o.cpu().numpy() for o in outs)
    used = np.arange(K + 1)[None, :] <= nd[:, None]
    assert (am[used] == am_all[used]).all() and (am[~used] == -1).all()
    assert (acc == acc_o).all() and (nacc == nacc_o).all()
    a = nacc_o - 1
    assert cnt.cpu().numpy().tolist() == [2 * B, 2 * int(nacc_o.sum()), 2 * int(nd.sum()), 2 * int(a.sum()),
                                          2 * int((nd > 0).sum()), 2 * int((nd + 1).sum())]
    assert S.sam_workspace_status(ws, B, K) == 0


@pytest.mark.parametrize("variant,skip", [(0, True), (0, False), (1, True), (2, False), (3, True), (3, False),
                                          (0, "chain"), (1, "chain"), (3, "chain")])
def test_closed_loop_with_the_adaptive_switch(variant, skip):
    """A schedule of context lengths drives the switch: steps over the threshold run without speculation.
    Every output of every step and the final counters equal the oracle's.  skip = "chain": rows beyond the
    proposal are skipped and, from the second step on, the rows to read come from the list the previous step's
    accept kernel left in the workspace (SAM_STEP_ROW_LIST_READY) instead of a listing kernel."""
    chain, skip = skip == "chain", bool(skip)
    cfg = W.CONFIGS[1].scaled(sessions=24, B=40, steps=14, vocab=20000)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    gpu = CudaBackend(cfg, corpus, bits_to_device(noise))
    cpu = OracleBackend(cfg, corpus, noise.copy())
    f_g, f_o = W.ClosedLoopFeeder(cfg, scripts, rowmax), W.ClosedLoopFeeder(cfg, scripts, rowmax)
    toks, n = f_g.prime_tokens()
    dg, ndg = gpu.prime(toks, n)
    do, ndo = cpu.prime(toks, n)
    cnt_g = torch.zeros(S.SAM_N_COUNTERS, dtype=torch.int64, device=DEV)
    cnt_o = np.zeros(6, np.int64)
    ctx_schedule = [1000, 2000, 40000, 50000, 3000, 4000, 5000, 70000, 6000, 7000, 8000, 9000, 90000, 100]
    off_steps = 0
    S.sam_set_argmax_variant(variant)
    try:
        for t in range(cfg.steps):
            on = S.sam_adaptive_switch(ctx_schedule[t], cfg.B, 32768, 64)
            assert on == oracle.speculation_enabled(ctx_schedule[t], cfg.B, 32768, 64)
            flags = (0 if on else S.SAM_STEP_NO_SPECULATION) | (S.SAM_STEP_SKIP_UNUSED_ROWS if skip else 0)
            oracle_flags = flags
            if chain and t > 0:
                flags |= S.SAM_STEP_ROW_LIST_READY
            launches0 = S.sam_launch_count()
            off_steps += not on
            zero = np.zeros(cfg.B, np.int32)
            ow_g = f_g.overwrites(t, dg, ndg if on else zero)
            ow_o = f_o.overwrites(t, do, ndo if on else zero)
            keep = np.arange(ow_g["row"].shape[0])
            sv_g = gpu.poke(ow_g["row"], ow_g["col"], ow_g["bits"], keep)
            sv_o = cpu.poke(ow_o["row"], ow_o["col"], ow_o["bits"], keep)
            c = cfg
            S.sam_step_ex(gpu.index.handle, gpu.logits, gpu.stride, c.B, c.K, c.vocab, gpu.drafts, gpu.n_draft,
                          gpu.argmax, gpu.accepted, gpu.n_accepted, gpu.state, gpu.mlen, c.min_match,
                          gpu.drafts, gpu.n_draft, flags, cnt_g, gpu.ws, gpu.ws_bytes)
            torch.cuda.synchronize()
            g = dict(argmax=gpu.argmax.cpu().numpy(), accepted=gpu.accepted.cpu().numpy(),
                     n_accepted=gpu.n_accepted.cpu().numpy(), drafts=gpu.drafts.cpu().numpy(),
                     n_draft=gpu.n_draft.cpu().numpy(), state=gpu.state.cpu().numpy(), matched_len=gpu.mlen.cpu().numpy())
            if chain and t > 0 and on:
                assert S.sam_launch_count() - launches0 == 2       # argmax + accept, no listing kernel
            o = cpu.sam.step_ex(cpu.bits, c.B, c.K, c.vocab, do, ndo, cpu.state, cpu.mlen, c.min_match, oracle_flags, cnt_o)
            o["state"], o["matched_len"] = cpu.state.copy(), cpu.mlen.copy()
            gpu.unpoke(ow_g["row"], ow_g["col"], sv_g)
            cpu.unpoke(ow_o["row"], ow_o["col"], sv_o)
            for k in KEYS:
                assert (g[k] == o[k]).all(), (t, k)
            f_g.advance(g["n_accepted"])
            f_o.advance(o["n_accepted"])
            dg, ndg, do, ndo = g["drafts"], g["n_draft"], o["drafts"], o["n_draft"]
    finally:
        S.sam_set_argmax_variant(0)
    assert off_steps == 4
    assert (cnt_g.cpu().numpy() == cnt_o).all()
    assert cnt_o[0] == cfg.B * cfg.steps and cnt_o[3] > 0
    assert gpu.status() == 0


def test_closed_loop_driven_by_the_counter_switch():
    """The switch decided from the device counters: after every window of two steps the counters of the window's
    speculating passes go to sam_speculation_pays together with the cost ratio of the moment (a schedule standing
    in for a load that changes: cheap verification, then a phase where a full pass costs 40 one-row passes, then
    cheap again).  While speculation is off every third window tries it again.  The library's decisions equal the
    oracle's, every output of every step equals the oracle's, and the switch goes off and comes back on."""
    cfg = W.CONFIGS[1].scaled(sessions=24, B=40, steps=24, vocab=20000)
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    gpu = CudaBackend(cfg, corpus, bits_to_device(noise))
    cpu = OracleBackend(cfg, corpus, noise.copy())
    f_g, f_o = W.ClosedLoopFeeder(cfg, scripts, rowmax), W.ClosedLoopFeeder(cfg, scripts, rowmax)
    toks, n = f_g.prime_tokens()
    dg, ndg = gpu.prime(toks, n)
    do, ndo = cpu.prime(toks, n)
    cnt_g = torch.zeros(S.SAM_N_COUNTERS, dtype=torch.int64, device=DEV)
    cnt_o = np.zeros(6, np.int64)
    ratio_of_window = [1.2, 1.2, 1.2, 40.0, 40.0, 40.0, 40.0, 40.0, 1.2, 1.2, 1.2, 1.2]
    on, windows_off, history = True, 0, []
    c = cfg
    for t in range(cfg.steps):
        w = t // 2
        flags = S.SAM_STEP_SKIP_UNUSED_ROWS | (0 if on else S.SAM_STEP_NO_SPECULATION)
        zero = np.zeros(cfg.B, np.int32)
        ow_g = f_g.overwrites(t, dg, ndg if on else zero)
        ow_o = f_o.overwrites(t, do, ndo if on else zero)
        keep = np.arange(ow_g["row"].shape[0])
        sv_g = gpu.poke(ow_g["row"], ow_g["col"], ow_g["bits"], keep)
        sv_o = cpu.poke(ow_o["row"], ow_o["col"], ow_o["bits"], keep)
        S.sam_step_ex(gpu.index.handle, gpu.logits, gpu.stride, c.B, c.K, c.vocab, gpu.drafts, gpu.n_draft,
                      gpu.argmax, gpu.accepted, gpu.n_accepted, gpu.state, gpu.mlen, c.min_match,
                      gpu.drafts, gpu.n_draft, flags, cnt_g, gpu.ws, gpu.ws_bytes)
        torch.cuda.synchronize()
        g = dict(argmax=gpu.argmax.cpu().numpy(), accepted=gpu.accepted.cpu().numpy(),
                 n_accepted=gpu.n_accepted.cpu().numpy(), drafts=gpu.drafts.cpu().numpy(),
                 n_draft=gpu.n_draft.cpu().numpy(), state=gpu.state.cpu().numpy(), matched_len=gpu.mlen.cpu().numpy())
        o = cpu.sam.step_ex(cpu.bits, c.B, c.K, c.vocab, do, ndo, cpu.state, cpu.mlen, c.min_match, flags, cnt_o)
        o["state"], o["matched_len"] = cpu.state.copy(), cpu.mlen.copy()
        gpu.unpoke(ow_g["row"], ow_g["col"], sv_g)
        cpu.unpoke(ow_o["row"], ow_o["col"], sv_o)
        for k in KEYS:
            assert (g[k] == o[k]).all(), (t, k)
        f_g.advance(g["n_accepted"])
        f_o.advance(o["n_accepted"])
        dg, ndg, do, ndo = g["drafts"], g["n_draft"], o["drafts"], o["n_draft"]
        if t % 2 == 1:                                    # end of a window
            host = cnt_g.cpu().numpy()
            assert (host == cnt_o).all()
            if on:                                        # only speculating passes say what speculation is worth
                on = S.sam_speculation_pays(host, c.K, ratio_of_window[w])
                assert on == oracle.speculation_pays(cnt_o, c.K, ratio_of_window[w])
                windows_off = 0
            else:
                windows_off += 1
                on = windows_off % 3 == 0                 # try again every third window
            history.append(on)
            cnt_g.zero_()
            cnt_o[:] = 0
    assert gpu.status() == 0
    # on through the cheap phase, off (with failed retries) through the expensive one, on again afterwards
    assert history[:2] == [True, True] and not any(history[3:5]) and history[-1] and history.count(False) >= 4
    k = history.index(False)
    assert True in history[k:], history


def test_row_list_ready_without_a_list_is_reported():
    """SAM_STEP_ROW_LIST_READY on a workspace that holds no list for this shape: nothing is read, the status word
    says so, and after re-initialising the workspace an ordinary call gives the oracle's result."""
    cfg = W.CONFIGS[0]
    corpus = W.make_corpus(cfg)
    noise = W.make_noise_logits(cfg)
    gpu = CudaBackend(cfg, corpus, bits_to_device(noise))
    cpu = OracleBackend(cfg, corpus, noise.copy())
    toks = np.ascontiguousarray(W.make_scripts(cfg, corpus)[:, :cfg.prime])
    n = np.full(cfg.B, cfg.prime, np.int32)
    gpu.prime(toks, n)
    do, ndo = cpu.prime(toks, n)
    st0, ml0, d0, nd0 = (x.clone() for x in (gpu.state, gpu.mlen, gpu.drafts, gpu.n_draft))
    both = S.SAM_STEP_SKIP_UNUSED_ROWS | S.SAM_STEP_ROW_LIST_READY
    for variant in (1, 3):
        S.sam_set_argmax_variant(variant)
        try:
            S.sam_workspace_init(gpu.ws, gpu.ws_bytes)        # whatever list an earlier call left is gone
            gpu.flags = both
            gpu.launch_step()
            torch.cuda.synchronize()
            assert gpu.status() == 3
            S.sam_workspace_init(gpu.ws, gpu.ws_bytes)
            for dst, src in ((gpu.state, st0), (gpu.mlen, ml0), (gpu.drafts, d0), (gpu.n_draft, nd0)):
                dst.copy_(src)
            gpu.flags = S.SAM_STEP_SKIP_UNUSED_ROWS
            g = gpu.step(None, None)
            assert gpu.status() == 0
        finally:
            S.sam_set_argmax_variant(0)
        o = cpu.sam.step_ex(cpu.bits, cfg.B, cfg.K, cfg.vocab, do, ndo, cpu.state.copy(), cpu.mlen.copy(), cfg.min_match,
                            S.SAM_STEP_SKIP_UNUSED_ROWS, np.zeros(6, np.int64))
        for k in ("argmax", "accepted", "n_accepted", "drafts", "n_draft"):
            assert (g[k] == o[k]).all(), (variant, k)
        for dst, src in ((gpu.state, st0), (gpu.mlen, ml0), (gpu.drafts, d0), (gpu.n_draft, nd0)):
            dst.copy_(src)


def test_flags_are_checked():
    lib = S.binding._load()
    assert lib.sam_verify_ex(None, 8, 1, 1, 8, None, None, None, None, None, 4, None, None, 0, None) == -1
    # the row-list flag belongs to sam_step_ex and needs the row-skipping flag beside it
    assert lib.sam_step_ex(None, None, 8, 1, 1, 8, None, None, None, None, None, None, None, 1, None, None, 4, None,
                           None, 0, None) == -1
    assert lib.sam_adaptive_switch(10, 10, 10, 10) == 1 and lib.sam_adaptive_switch(11, 10, 10, 10) == 0


@pytest.mark.parametrize("shards,multiple", [(4, 8), (3, 1), (8, 8)])
def test_vocabulary_shards_merge_to_the_full_row(shards, multiple):
    """The vocabulary split into column shards (aligned ones take the bulk-copy kernel, odd ones the
    direct-load kernel): per-shard words, elementwise maximum, then accept + walk + draft from the
    merged words equal the oracle's step on the whole rows - ties across shards and NaN rows included."""
    from paper_2512_18337_b200.parallel import shard_bounds
    cfg = W.CONFIGS[1].scaled(sessions=16, B=12, steps=4, vocab=50257)
    c = cfg
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    # exact ties that straddle shards, and NaNs at the start of the row and of a later shard
    noise[1, [100, 40000]] = 0x4140
    noise[2, [49000, 7]] = 0x4140
    noise[3, 0] = 0x7FC0
    noise[4, shard_bounds(c.vocab, 1, shards, multiple)[0]] = 0x7FC0
    gpu = CudaBackend(cfg, corpus, bits_to_device(noise))
    cpu = OracleBackend(cfg, corpus, noise.copy())
    f_g, f_o = W.ClosedLoopFeeder(cfg, scripts, rowmax), W.ClosedLoopFeeder(cfg, scripts, rowmax)
    toks, n = f_g.prime_tokens()
    dg, ndg = gpu.prime(toks, n)
    do, ndo = cpu.prime(toks, n)
    R = c.B * (c.K + 1)
    for t in range(c.steps):
        ow = f_g.overwrites(t, dg, ndg)
        f_o.overwrites(t, do, ndo)
        keep = np.arange(ow["row"].shape[0])
        sv_g = gpu.poke(ow["row"], ow["col"], ow["bits"], keep)
        sv_o = cpu.poke(ow["row"], ow["col"], ow["bits"], keep)
        merged = torch.zeros(R, dtype=torch.int64, device=DEV)
        for r in range(shards):
            lo, hi = shard_bounds(c.vocab, r, shards, multiple)
            keys = torch.full((R + 1,), -1, dtype=torch.int64, device=DEV)
            S.sam_argmax_partial(gpu.logits.data_ptr() + 2 * lo, gpu.stride, R, hi - lo, lo, keys)
            torch.cuda.synchronize()
            assert int(keys[R]) == 0
            merged = torch.maximum(merged, keys[:R])
        S.sam_step_from_keys(gpu.index.handle, merged, c.B, c.K, gpu.drafts, gpu.n_draft, gpu.argmax, gpu.accepted,
                             gpu.n_accepted, gpu.state, gpu.mlen, c.min_match, gpu.drafts, gpu.n_draft)
        torch.cuda.synchronize()
        assert int(merged.abs().sum()) == 0                      # the words are handed back zeroed
        g = dict(argmax=gpu.argmax.cpu().numpy(), accepted=gpu.accepted.cpu().numpy(),
                 n_accepted=gpu.n_accepted.cpu().numpy(), drafts=gpu.drafts.cpu().numpy(),
                 n_draft=gpu.n_draft.cpu().numpy(), state=gpu.state.cpu().numpy(), matched_len=gpu.mlen.cpu().numpy())
        o = cpu.step(do, ndo)
        gpu.unpoke(ow["row"], ow["col"], sv_g)
        cpu.unpoke(ow["row"], ow["col"], sv_o)
        for k in KEYS:
            assert (g[k] == o[k]).all(), (t, k)
        f_g.advance(g["n_accepted"])
        f_o.advance(o["n_accepted"])
        dg, ndg, do, ndo = g["drafts"], g["n_draft"], o["drafts"], o["n_draft"]


@pytest.mark.parametrize("flags", [0, 2, 3])
def test_host_buffer_step_with_options(flags):
    """sam_step_host_ex: everything in host memory; with SAM_STEP_SKIP_UNUSED_ROWS only the used rows are copied
    to the device, so the staging area is poisoned first to show that nothing else is read."""
    cfg = W.CONFIGS[0].scaled(B=9, steps=5)
    c = cfg
    corpus = W.make_corpus(cfg)
    scripts = W.make_scripts(cfg, corpus)
    noise = W.make_noise_logits(cfg)
    rowmax = W.f32_to_bf16_bits(W.bf16_bits_to_f32(noise).max(axis=1))
    index = S.SamIndex(corpus, [cfg.separator])
    cpu = OracleBackend(cfg, corpus, noise.copy())
    f_o = W.ClosedLoopFeeder(cfg, scripts, rowmax)
    toks, n = f_o.prime_tokens()
    do, ndo = cpu.prime(toks, n)
    h = dict(drafts=do.copy(), n_draft=ndo.copy(), argmax=np.zeros((c.B, c.K + 1), np.int32),
             accepted=np.zeros((c.B, c.K + 1), np.int32), n_accepted=np.zeros(c.B, np.int32),
             state=cpu.state.copy(), mlen=cpu.mlen.copy())
    sb = S.sam_step_host_staging_bytes(c.vocab, c.B, c.K, c.vocab)
    staging = torch.empty(sb, dtype=torch.uint8, device=DEV)
    host_bits = noise.copy()
    for t in range(c.steps):
        ow = f_o.overwrites(t, do, ndo if not (flags & 1) else np.zeros(c.B, np.int32))
        keep = np.arange(ow["row"].shape[0])
        sv = cpu.poke(ow["row"], ow["col"], ow["bits"], keep)
        sv_h = host_bits[ow["row"], ow["col"]].copy()
        host_bits[ow["row"], ow["col"]] = ow["bits"]
        staging.fill_(0x7F)          # 0x7F7F as bf16 is a huge number: a row that was not copied would win every argmax
        S.sam_step_host_ex(index.handle, host_bits, c.vocab, c.B, c.K, c.vocab, h["drafts"], h["n_draft"], h["argmax"],
                           h["accepted"], h["n_accepted"], h["state"], h["mlen"], c.min_match,
                           h["drafts"], h["n_draft"], flags, staging, sb)
        o = cpu.sam.step_ex(cpu.bits, c.B, c.K, c.vocab, do, ndo, cpu.state, cpu.mlen, c.min_match, flags)
        cpu.unpoke(ow["row"], ow["col"], sv)
        host_bits[ow["row"], ow["col"]] = sv_h
        assert (h["argmax"] == o["argmax"]).all() and (h["accepted"] == o["accepted"]).all(), t
        assert (h["n_accepted"] == o["n_accepted"]).all() and (h["state"] == cpu.state).all() and (h["mlen"] == cpu.mlen).all()
        assert (h["drafts"] == o["drafts"]).all() and (h["n_draft"] == o["n_draft"]).all()
        f_o.advance(o["n_accepted"])
        do, ndo = o["drafts"], o["n_draft"]
