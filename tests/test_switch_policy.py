"""The library's counter-driven switch (a host function of the C ABI) against the oracle's.  CPU only."""
from __future__ import annotations

import numpy as np

import oracle
import paper_2512_18337_b200 as S


def test_library_decides_like_the_oracle():
    rng = np.random.default_rng(5)
    seen = set()
    for _ in range(3000):
        K = int(rng.integers(1, 33))
        passes = int(rng.integers(0, 5000))
        rows = passes + int(rng.integers(0, K * passes + 1))
        acc = int(rng.integers(0, rows - passes + 1))
        cnt = np.array([passes, passes + acc, int(rng.integers(acc, acc + 999)), acc, passes // 2, rows], np.int64)
        # ratios of every kind: dyadic, decimal, and ones that put the two sides close together
        ratio = float(rng.choice([0.5, 1.0, 1.1, 1.7, 2.0, 3.3, 1.0 + (acc * K) / max(1, rows - passes),
                                  np.nextafter(1.0 + (acc * K) / max(1, rows - passes), 9.0), float(rng.random() * 6 + 0.01)]))
        got = S.sam_speculation_pays(cnt, K, ratio)
        assert got == oracle.speculation_pays(cnt, K, ratio), (cnt.tolist(), K, ratio)
        seen.add(got)
    assert seen == {True, False}


def test_bad_arguments_are_refused():
    lib = S.binding._load()
    ok = np.array([10, 25, 30, 15, 8, 50], np.int64)
    assert lib.sam_speculation_pays(ok.ctypes.data, 4, 2.0) == 1
    assert lib.sam_speculation_pays(None, 4, 2.0) == -1
    assert lib.sam_speculation_pays(ok.ctypes.data, 0, 2.0) == -1 and lib.sam_speculation_pays(ok.ctypes.data, 33, 2.0) == -1
    assert lib.sam_speculation_pays(ok.ctypes.data, 4, 0.0) == -1 and lib.sam_speculation_pays(ok.ctypes.data, 4, float("nan")) == -1
    fewer_rows_than_passes = np.array([10, 25, 30, 15, 8, 9], np.int64)
    assert lib.sam_speculation_pays(fewer_rows_than_passes.ctypes.data, 4, 2.0) == -1
