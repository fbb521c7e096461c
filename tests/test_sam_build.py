"""Host-side setup of the CUDA library against the oracle, the C-ABI surface, error codes. CPU only."""
from __future__ import annotations

import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
import paper_2512_18337_b200 as S
import workload as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _cmp(corpus, seps):
    h = S.sam_build(corpus, seps)
    try:
        ex = S.sam_export(h)
        S_, E_, nbytes = S.sam_sizes(h)
    finally:
        S.sam_free(h)
    o = oracle.OracleSAM(corpus, seps)
    oe = o.export()
    assert (S_, E_) == (o.n_states, o.n_edges)
    for k in oe:
        assert ex[k].dtype == oe[k].dtype and (ex[k] == oe[k]).all(), k
    assert nbytes % 256 == 0 and nbytes >= 32 * S_ + 4 * corpus.shape[0]


def test_build_equals_oracle_small_alphabets():
    rng = np.random.default_rng(7)
    for sigma in (1, 2, 3, 5, 50):
        for n in (1, 2, 3, 10, 100, 3000):
            _cmp(rng.integers(0, sigma, size=n).astype(np.int32), [sigma])


def test_build_equals_oracle_heavy_rows():
    # one hub token followed by many distinct tokens: rows far wider than the chain/hash switch-over
    rng = np.random.default_rng(8)
    body = np.empty(4000, np.int32)
    body[0::2] = 0
    body[1::2] = rng.integers(1, 700, size=2000)
    _cmp(body, [1 << 20])


@pytest.mark.parametrize("i", [0, 1])
def test_build_equals_oracle_configs(i):
    cfg = W.CONFIGS[i]
    if i == 1:
        cfg = cfg.scaled(sessions=48)
    _cmp(W.make_corpus(cfg), [cfg.separator])


def test_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "sam.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(sam_[a-z_]+)\s*\(", text))
    assert declared == set(S.exported_symbols())
    lib = C.CDLL(str(S.library_path()))
    for name in declared:
        assert hasattr(lib, name), name


def test_error_codes_without_a_device():
    corpus = np.arange(10, dtype=np.int32)
    with pytest.raises(S.SamError) as e:
        S.sam_build(np.array([1, -2, 3], np.int32), [9])
    assert e.value.status == -1
    with pytest.raises(S.SamError):
        S.sam_build(np.zeros(0, np.int32), [9])
    with pytest.raises(S.SamError):
        S.sam_build(corpus, list(range(100, 100 + S.binding.SAM_MAX_SEPARATORS + 1)))
    h = S.sam_build(corpus, [])
    try:
        assert S.sam_sizes(h)[0] == 11
        lib = S.binding._load()
        # hot path before upload
        assert lib.sam_draft(h, 1, 8, 8, 8, 1, 8, 4, 1, 8, 8, None) == -3
        assert lib.sam_draft(h, 1, 8, 8, 8, 1, 8, 0, 1, 8, 8, None) == -1          # K < 1
        assert lib.sam_draft(h, 1, 8, 8, 8, 1, 8, 33, 1, 8, 8, None) == -1         # K > SAM_K_MAX
        assert lib.sam_draft(h, 1, 8, 8, 8, 1, 8, 4, 0, 8, 8, None) == -1          # min_match < 1
        assert lib.sam_verify(16, 10, 1, 4, 11, 8, 8, 8, 8, 8, 8, 1 << 20, None) == -1   # stride < V
        assert lib.sam_verify(17, 16, 1, 4, 11, 8, 8, 8, 8, 8, 8, 1 << 20, None) == -1   # odd logits address
        assert lib.sam_verify(16, 16, 1, 4, 11, 8, 8, 8, 8, 8, 8, 8, None) == -5         # workspace too small
        assert lib.sam_verify(None, 16, 1, 4, 11, 8, 8, 8, 8, 8, 8, 1 << 20, None) == -1
        assert lib.sam_verify(None, 16, 0, 4, 11, None, None, None, None, None, None, 0, None) == 0  # B = 0
        assert lib.sam_upload(h, None, 1 << 30, None) == -1
        assert lib.sam_upload(h, 256, 16, None) == -5
    finally:
        S.sam_free(h)
    assert S.sam_workspace_bytes(256, 16) >= 256 * 17 * 8
    with pytest.raises(S.SamError):
        S.sam_workspace_bytes(4, 33)
    assert "invalid" in S.sam_strerror(-1)
