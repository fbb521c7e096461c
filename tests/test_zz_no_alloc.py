"""sam_verify_static: the verification entry point for callers that cannot allocate device memory
(for instance a plugin inside a serving engine that has already claimed the whole GPU for its own
pools).  Its scratch is a fixed array inside the library, so the test checks that two calls in a
row - the second on different logits, so leftovers of the first would show - give exactly what
sam_verify gives with a caller-allocated workspace and what the CPU oracle computes from the same
bits, that the call leaves the amount of free device memory unchanged, that its status word reads
zero afterwards, and that oversize batches are refused.
Collected last on purpose: a failure here must not hide any other test."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
import paper_2512_18337_b200 as S
import workload as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, B, K, V, pad):
    rng = np.random.default_rng(seed)
    bits = W.f32_to_bf16_bits(rng.standard_normal((B * (K + 1), V + pad), dtype=np.float32))
    # planted ties and a few special rows so that the scratch sees every kind of candidate
    bits[0, [3, V - 1]] = 0x4120
    bits[1, :] = 0xFF80
    bits[2, 0] = 0x7FC0
    lg = torch.from_numpy(bits.view(np.int16)).to(DEV).view(torch.bfloat16)
    n_draft = torch.from_numpy(rng.integers(0, K + 1, size=B).astype(np.int32)).to(DEV)
    return lg, n_draft, rng, bits


def _outputs(B, K):
    return [torch.full(s, -3, dtype=torch.int32, device=DEV) for s in ((B, K + 1), (B, K + 1), (B,))]


def test_static_scratch_matches_workspace_twice():
    B, K, V, pad = 37, 9, 50257, 3
    wsb = S.sam_workspace_bytes(B, K)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    S.sam_workspace_init(ws, wsb)
    for call, seed in enumerate((21, 22)):
        lg, n_draft, rng, bits = _case(seed, B, K, V, pad)
        # reference run with a caller-owned workspace; drafts follow its argmax so accepts are non-trivial
        am0, acc0, n0 = _outputs(B, K)
        drafts = torch.zeros((B, K), dtype=torch.int32, device=DEV)
        S.sam_verify(lg, V + pad, B, K, V, drafts, n_draft, am0, acc0, n0, ws, wsb)
        torch.cuda.synchronize()
        d = am0[:, :K].clone()
        flip = torch.from_numpy(rng.random((B, K)) < 0.2).to(DEV)
        d[flip] = 1
        S.sam_verify(lg, V + pad, B, K, V, d, n_draft, am0, acc0, n0, ws, wsb)
        am1, acc1, n1 = _outputs(B, K)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        reserved_before = torch.cuda.memory_reserved()
        S.sam_verify_static(lg, V + pad, B, K, V, d, n_draft, am1, acc1, n1)
        torch.cuda.synchronize()
        if call > 0:
            # the first call on a device may load the module and looks up the array's address; from the second
            # call on nothing about the device's memory may move (neither the driver's nor torch's allocator)
            assert torch.cuda.mem_get_info()[0] == free_before
            assert torch.cuda.memory_reserved() == reserved_before
        assert S.sam_static_status() == 0
        assert torch.equal(am0, am1), f"call {call}: argmax differs"
        assert torch.equal(acc0, acc1) and torch.equal(n0, n1), f"call {call}: accept differs"
        assert int((n1 >= 1).all()) == 1
        # and against the oracle, from the same bits
        am_o = oracle.argmax_batch(bits, V=V, threads=oracle.host_threads()).reshape(B, K + 1)
        acc_o, n_o = oracle.accept_batch(d.cpu().numpy(), n_draft.cpu().numpy(), am_o)
        assert (am1.cpu().numpy() == am_o).all(), f"call {call}: argmax differs from the oracle"
        assert (acc1.cpu().numpy() == acc_o).all() and (n1.cpu().numpy() == n_o).all(), f"call {call}: accept differs from the oracle"


def test_static_scratch_rejects_oversize_and_bad_sizes():
    lib = S.binding._load()
    too_many = S.binding.SAM_STATIC_MAX_ROWS // 17 + 1
    assert lib.sam_verify_static(None, 8, too_many, 16, 8, None, None, None, None, None, None) == -6
    assert "limit" in S.sam_strerror(-6)
    assert lib.sam_verify_static(None, 8, 4, 0, 8, None, None, None, None, None, None) == -1
    assert lib.sam_verify_static(None, 8, 0, 4, 8, None, None, None, None, None, None) == 0   # B = 0: no-op
    # the largest admissible batch runs
    B, K, V = S.binding.SAM_STATIC_MAX_ROWS // 2, 1, 64
    lg, n_draft, _, bits = _case(5, B, K, V, 0)
    am, acc, n = _outputs(B, K)
    d = torch.zeros((B, K), dtype=torch.int32, device=DEV)
    S.sam_verify_static(lg, V, B, K, V, d, n_draft, am, acc, n)
    torch.cuda.synchronize()
    assert S.sam_static_status() == 0
    am_o = oracle.argmax_batch(bits, V=V, threads=oracle.host_threads()).reshape(B, K + 1)
    acc_o, n_o = oracle.accept_batch(d.cpu().numpy(), n_draft.cpu().numpy(), am_o)
    assert (am.cpu().numpy() == am_o).all()
    assert (acc.cpu().numpy() == acc_o).all() and (n.cpu().numpy() == n_o).all()
