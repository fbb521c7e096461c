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


# ------------------------------------------------------------------ growing index (host side)
def _grow_and_compare(text, cuts, sep, wait_each=True):
    parts = np.split(text, cuts)
    h = S.sam_build_growing(parts[0], [sep], max_tokens=text.shape[0] + 5, max_token_id=int(max(text.max(), sep)))
    try:
        for p in parts[1:]:
            S.sam_extend(h, p, wait=wait_each)
        if not wait_each:
            S.sam_extend(h, np.zeros(0, np.int32), wait=True)      # waits for the queue to drain
        queued, built, on_dev = S.sam_pending(h)
        assert queued == built == text.shape[0] and on_dev == 0
        ex = S.sam_export(h)
        S_, E_, nbytes = S.sam_sizes(h)
    finally:
        S.sam_free(h)
    o = oracle.OracleSAM(text, [sep])
    oe = o.export()
    assert (S_, E_) == (o.n_states, o.n_edges)
    for k in oe:
        assert (ex[k] == oe[k]).all(), k
    assert nbytes >= 32 * (2 * text.shape[0]) + 4 * text.shape[0]


@pytest.mark.parametrize("sigma,n", [(1, 40), (2, 500), (3, 2000), (50, 3000)])
def test_growing_index_equals_one_shot_build(sigma, n):
    """Text that arrives in pieces (synchronously and through the builder thread's queue) yields the very
    automaton, numbering included, that the oracle builds from the whole text."""
    rng = np.random.default_rng(sigma * 1000 + n)
    text = rng.integers(0, sigma, size=n).astype(np.int32)
    cuts = np.sort(rng.choice(np.arange(1, n), size=min(7, n - 1), replace=False))
    _grow_and_compare(text, cuts, sigma, wait_each=True)
    _grow_and_compare(text, cuts, sigma, wait_each=False)


def test_growing_index_from_empty_and_limits():
    h = S.sam_build_growing(np.zeros(0, np.int32), [9], max_tokens=10, max_token_id=9)
    try:
        assert S.sam_sizes(h)[0] == 1                               # the root alone
        S.sam_extend(h, np.array([1, 2, 1, 2, 9, 1], np.int32))
        assert S.sam_pending(h)[:2] == (6, 6)
        with pytest.raises(S.SamError) as e:
            S.sam_extend(h, np.array([10], np.int32))               # id above max_token_id
        assert e.value.status == -1
        with pytest.raises(S.SamError) as e:
            S.sam_extend(h, np.arange(5, dtype=np.int32))           # 6 + 5 > max_tokens
        assert e.value.status == -6
        ex = S.sam_export(h)
        oe = oracle.OracleSAM(np.array([1, 2, 1, 2, 9, 1], np.int32), [9]).export()
        for k in oe:
            assert (ex[k] == oe[k]).all(), k
    finally:
        S.sam_free(h)
    lib = S.binding._load()
    hs = S.sam_build(np.array([1, 2, 3], np.int32), [9])
    try:
        assert lib.sam_extend(hs, None, 0) == -1                    # a one-shot index cannot grow
        assert lib.sam_sync(hs, None, None) == -1
    finally:
        S.sam_free(hs)


def test_argument_checks_that_need_no_device():
    """Entry points reject bad sizes, flags and null pointers before they touch CUDA."""
    lib = S.binding._load()
    assert S.sam_workspace_bytes(4, 8) % 256 == 0
    assert S.sam_workspace_bytes(8, 8) > S.sam_workspace_bytes(4, 8) > S.sam_workspace_bytes(4, 1)
    assert lib.sam_workspace_bytes(-1, 4) == -1 and lib.sam_workspace_bytes(4, 0) == -1 and lib.sam_workspace_bytes(4, 33) == -1
    assert lib.sam_verify_ex(None, 8, 1, 1, 8, None, None, None, None, None, 8, None, None, 0, None) == -1     # unknown flag
    assert lib.sam_verify_ex(None, 8, 0, 1, 8, None, None, None, None, None, 0, None, None, 0, None) == 0      # B = 0
    assert lib.sam_verify_ex(None, 7, 1, 1, 8, None, None, None, None, None, 0, None, None, 0, None) == -1     # stride < V
    assert lib.sam_step_ex(None, None, 8, 1, 1, 8, None, None, None, None, None, None, None, 1, None, None, 0, None,
                           None, 0, None) == -1                                                                # no index
    assert lib.sam_argmax_partial(None, 8, 0, 8, 0, None, None) == 0                                           # no rows
    assert lib.sam_argmax_partial(None, 8, 1, 8, -1, None, None) == -1                                         # bad offset
    assert lib.sam_argmax_partial(None, 8, 1, 8, 0, None, None) == -1                                          # null pointers
    assert lib.sam_set_bytes(0) == -1 and lib.sam_set_bytes(2) % 256 == 0
    assert lib.sam_adaptive_switch(100, 4, 100, 4) == 1 and lib.sam_adaptive_switch(101, 4, 100, 4) == 0
    assert lib.sam_adaptive_switch(100, 5, 100, 4) == 0
    for ctx, bs in [(1, 1), (10 ** 6, 1), (1, 10 ** 4), (32768, 64), (32769, 64), (32768, 65)]:
        assert bool(lib.sam_adaptive_switch(ctx, bs, 32768, 64)) == oracle.speculation_enabled(ctx, bs, 32768, 64)
    h = S.sam_build(np.array([1, 2, 3], np.int32), [9])
    try:   # hot-path calls before sam_upload
        assert lib.sam_draft(h, 1, None, None, None, 0, None, 2, 1, None, None, None) == -3
        assert lib.sam_renormalize(h, 1, None, None, None) == -3
    finally:
        S.sam_free(h)
    assert S.sam_strerror(-3).startswith("automaton not uploaded")
    # the kernel-selection switch takes 0..3 and keeps its value on a refused call
    for v in (1, 2, 3, 0):
        assert lib.sam_set_argmax_variant(v) == 0
    assert lib.sam_set_argmax_variant(4) == -1 and lib.sam_set_argmax_variant(-1) == -1


def test_missing_library_fails_loudly(tmp_path):
    """There is no CPU fallback: with the shared library absent the first call raises, and nothing under
    the package imports the oracle."""
    import subprocess
    import sys
    code = (
        "import os, sys\n"
        f"sys.path.insert(0, {ROOT!r})\n"
        "import numpy as np\n"
        "import paper_2512_18337_b200 as S\n"
        f"S.use_library({str(tmp_path / 'nowhere.so')!r})\n"
        "try:\n"
        "    S.sam_build(np.array([1, 2, 3], np.int32), [9])\n"
        "except RuntimeError as e:\n"
        "    assert 'missing' in str(e) and 'no CPU fallback' in str(e), e\n"
        "    assert 'oracle' not in sys.modules\n"
        "    print('raised')\n"
    )
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and "raised" in out.stdout, out.stderr
    # the product sources never import the oracle package
    pkg = os.path.join(ROOT, "paper_2512_18337_b200")
    for name in os.listdir(pkg):
        if name.endswith(".py"):
            text = open(os.path.join(pkg, name)).read()
            assert "import oracle" not in text and "from oracle" not in text, name
