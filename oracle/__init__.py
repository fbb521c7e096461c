"""ctypes front end of the CPU oracle (``sam_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline may import this; the CUDA product path never does, and this module
imports nothing from the CUDA package.  The arithmetic of the single-automaton
path lives in the C file, which this wrapper compiles with gcc and calls through
numpy arrays; only the composite-drafting rule (`multi_draft`) is stated here in
Python, on top of the C walk and draft.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_DIR = Path(__file__).resolve().parent
_SRC = _DIR / "sam_oracle.c"
_SO = _DIR / "libsam_oracle.so"
_lib = None

_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_u16p = C.POINTER(C.c_uint16)


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (rebuilds when the source is newer)."""
    if force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _SO.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-Wall", "-Wextra",
             "-o", str(tmp), str(_SRC)])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(str(build()))
        lib.oracle_sam_build.restype = C.c_void_p
        lib.oracle_sam_build.argtypes = [_i32p, C.c_int64]
        lib.oracle_sam_extend.restype = C.c_int
        lib.oracle_sam_extend.argtypes = [C.c_void_p, _i32p, C.c_int64]
        lib.oracle_renormalize.restype = C.c_int32
        lib.oracle_renormalize.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        lib.oracle_sam_free.restype = None
        lib.oracle_sam_free.argtypes = [C.c_void_p]
        lib.oracle_sam_states.restype = C.c_int64
        lib.oracle_sam_states.argtypes = [C.c_void_p]
        lib.oracle_sam_edges.restype = C.c_int64
        lib.oracle_sam_edges.argtypes = [C.c_void_p]
        lib.oracle_sam_export.restype = None
        lib.oracle_sam_export.argtypes = [C.c_void_p, _i32p, _i32p, _i32p, _i64p, _i32p, _i32p]
        lib.oracle_walk.restype = None
        lib.oracle_walk.argtypes = [C.c_void_p, _i32p, _i32p, _i32p, C.c_int32]
        lib.oracle_draft.restype = C.c_int32
        lib.oracle_draft.argtypes = [C.c_void_p, _i32p, C.c_int64, _i32p, C.c_int32,
                                     C.c_int32, C.c_int32, C.c_int32, C.c_int32, _i32p]
        lib.oracle_argmax_row.restype = C.c_int32
        lib.oracle_argmax_row.argtypes = [_u16p, C.c_int32]
        lib.oracle_accept.restype = C.c_int32
        lib.oracle_accept.argtypes = [_i32p, C.c_int32, _i32p, C.c_int32, _i32p]
        lib.oracle_draft_batch.restype = None
        lib.oracle_draft_batch.argtypes = [C.c_void_p, _i32p, C.c_int64, _i32p, C.c_int32, C.c_int32,
                                           _i32p, _i32p, _i32p, C.c_int32, _i32p,
                                           C.c_int32, C.c_int32, _i32p, _i32p, C.c_int32]
        lib.oracle_argmax_batch.restype = None
        lib.oracle_argmax_batch.argtypes = [_u16p, C.c_int64, C.c_int64, C.c_int32, _i32p, C.c_int32]
        lib.oracle_accept_batch.restype = None
        lib.oracle_accept_batch.argtypes = [C.c_int32, C.c_int32, _i32p, _i32p, _i32p, _i32p, _i32p]
        lib.oracle_step.restype = None
        lib.oracle_step.argtypes = [C.c_void_p, _i32p, C.c_int64, _i32p, C.c_int32,
                                    _u16p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                    _i32p, _i32p, _i32p, _i32p, _i32p, _i32p, _i32p, C.c_int32,
                                    _i32p, _i32p, C.c_int32]
        lib.oracle_step_ex.restype = None
        lib.oracle_step_ex.argtypes = [C.c_void_p, _i32p, C.c_int64, _i32p, C.c_int32,
                                       _u16p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                       _i32p, _i32p, _i32p, _i32p, _i32p, _i32p, _i32p, C.c_int32,
                                       _i32p, _i32p, C.c_uint32, _i64p]
        lib.oracle_speculation_enabled.restype = C.c_int32
        lib.oracle_speculation_enabled.argtypes = [C.c_int64] * 4
        lib.oracle_speculation_pays.restype = C.c_int32
        lib.oracle_speculation_pays.argtypes = [_i64p, C.c_int32, C.c_double]
        _lib = lib
    return _lib


def _i32(a: np.ndarray):
    assert a.dtype == np.int32 and a.flags.c_contiguous
    return a.ctypes.data_as(_i32p)


def _u16(a: np.ndarray):
    assert a.dtype == np.uint16 and a.flags.c_contiguous
    return a.ctypes.data_as(_u16p)


def host_threads() -> int:
    """Cores this process may run on."""
    return len(os.sched_getaffinity(0))


class OracleSAM:
    """Suffix automaton over a flat int32 corpus, plus per-stream walk/draft."""

    def __init__(self, corpus: np.ndarray, separators):
        self.lib = _load()
        self.corpus = np.ascontiguousarray(corpus, dtype=np.int32)
        self.seps = np.ascontiguousarray(np.atleast_1d(separators), dtype=np.int32)
        self.n = int(self.corpus.shape[0])
        self.h = self.lib.oracle_sam_build(_i32(self.corpus), self.n)
        if not self.h:
            raise MemoryError("oracle_sam_build failed")

    def __del__(self):
        h, self.h = getattr(self, "h", None), None
        if h:
            self.lib.oracle_sam_free(h)

    def extend(self, tokens) -> None:
        """Appends tokens to the indexed text (the corpus copy used for drafting grows with it)."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        if self.lib.oracle_sam_extend(self.h, _i32(t), t.shape[0]):
            raise MemoryError("oracle_sam_extend failed")
        self.corpus = np.concatenate([self.corpus, t])
        self.n = int(self.corpus.shape[0])

    def renormalize(self, state, matched_len) -> None:
        """In place: every (state[b], matched_len[b]) taken before the text grew is moved to the
        state that now holds its string."""
        for b in range(state.shape[0]):
            state[b] = self.lib.oracle_renormalize(self.h, int(state[b]), int(matched_len[b]))

    @property
    def n_states(self) -> int:
        return int(self.lib.oracle_sam_states(self.h))

    @property
    def n_edges(self) -> int:
        return int(self.lib.oracle_sam_edges(self.h))

    def export(self):
        """dict(len, link, firstpos [S] int32; row_ptr [S+1] int64; edge_tok, edge_dst [E] int32)."""
        S, E = self.n_states, self.n_edges
        out = dict(len=np.empty(S, np.int32), link=np.empty(S, np.int32),
                   firstpos=np.empty(S, np.int32), row_ptr=np.empty(S + 1, np.int64),
                   edge_tok=np.empty(E, np.int32), edge_dst=np.empty(E, np.int32))
        self.lib.oracle_sam_export(self.h, _i32(out["len"]), _i32(out["link"]), _i32(out["firstpos"]),
                                   out["row_ptr"].ctypes.data_as(_i64p),
                                   _i32(out["edge_tok"]), _i32(out["edge_dst"]))
        return out

    def walk(self, state: int, matched_len: int, tokens) -> tuple[int, int]:
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        s, L = C.c_int32(state), C.c_int32(matched_len)
        self.lib.oracle_walk(self.h, C.byref(s), C.byref(L), _i32(t), t.shape[0])
        return s.value, L.value

    def draft(self, state: int, matched_len: int, K: int, min_match: int):
        d = np.empty(K, np.int32)
        nd = self.lib.oracle_draft(self.h, _i32(self.corpus), self.n, _i32(self.seps), self.seps.shape[0],
                                   state, matched_len, K, min_match, _i32(d))
        return d, int(nd)

    def draft_batch(self, state, matched_len, new_tokens, n_new, K, min_match, threads=1):
        """In-place update of state/matched_len [B]; returns (drafts [B,K], n_draft [B])."""
        B, ld = new_tokens.shape
        drafts = np.empty((B, K), np.int32)
        n_draft = np.empty(B, np.int32)
        self.lib.oracle_draft_batch(self.h, _i32(self.corpus), self.n, _i32(self.seps), self.seps.shape[0], B,
                                    _i32(state), _i32(matched_len), _i32(new_tokens), ld, _i32(n_new),
                                    K, min_match, _i32(drafts), _i32(n_draft), threads)
        return drafts, n_draft

    def step(self, logits_bits, B, K, V, drafts, n_draft, state, matched_len, min_match, threads=1):
        """argmax -> accept -> walk -> next draft. logits_bits: [B*(K+1), >=V] uint16, row-major.
        state/matched_len updated in place. Returns dict of outputs."""
        lg = logits_bits.reshape(B * (K + 1), -1)
        stride = lg.shape[1]
        out = dict(argmax=np.empty((B, K + 1), np.int32), accepted=np.empty((B, K + 1), np.int32),
                   n_accepted=np.empty(B, np.int32), drafts=np.empty((B, K), np.int32),
                   n_draft=np.empty(B, np.int32))
        self.lib.oracle_step(self.h, _i32(self.corpus), self.n, _i32(self.seps), self.seps.shape[0],
                             _u16(lg), stride, B, K, V, _i32(drafts), _i32(n_draft),
                             _i32(out["argmax"]), _i32(out["accepted"]), _i32(out["n_accepted"]),
                             _i32(state), _i32(matched_len), min_match,
                             _i32(out["drafts"]), _i32(out["n_draft"]), threads)
        return out


NO_SPECULATION = 1
SKIP_UNUSED_ROWS = 2


def speculation_enabled(context_len: int, batch_size: int, max_context_len: int, max_batch_size: int) -> bool:
    return bool(_load().oracle_speculation_enabled(context_len, batch_size, max_context_len, max_batch_size))


def speculation_pays(counters: np.ndarray, K: int, cost_ratio: float) -> bool:
    """The counter-driven switch: does the window of passes behind `counters` (int64[6] as oracle_step_ex fills
    them) commit more tokens than it costs, a (K+1)-row pass costing cost_ratio one-row passes?"""
    c = np.ascontiguousarray(counters, dtype=np.int64)
    assert c.shape == (6,)
    return bool(_load().oracle_speculation_pays(c.ctypes.data_as(_i64p), K, float(cost_ratio)))


def argmax_row(row_bits: np.ndarray) -> int:
    r = np.ascontiguousarray(row_bits, dtype=np.uint16)
    return int(_load().oracle_argmax_row(_u16(r), r.shape[0]))


def _step_ex(self, logits_bits, B, K, V, drafts, n_draft, state, matched_len, min_match, flags=0, counters=None):
    """Step with options (NO_SPECULATION, SKIP_UNUSED_ROWS) and running counters (int64[6], updated in place)."""
    lg = logits_bits.reshape(B * (K + 1), -1)
    out = dict(argmax=np.empty((B, K + 1), np.int32), accepted=np.empty((B, K + 1), np.int32),
               n_accepted=np.empty(B, np.int32), drafts=np.empty((B, K), np.int32),
               n_draft=np.empty(B, np.int32))
    cp = counters.ctypes.data_as(_i64p) if counters is not None else None
    self.lib.oracle_step_ex(self.h, _i32(self.corpus), self.n, _i32(self.seps), self.seps.shape[0],
                            _u16(lg), lg.shape[1], B, K, V, _i32(drafts), _i32(n_draft),
                            _i32(out["argmax"]), _i32(out["accepted"]), _i32(out["n_accepted"]),
                            _i32(state), _i32(matched_len), min_match,
                            _i32(out["drafts"]), _i32(out["n_draft"]), flags, cp)
    return out


OracleSAM.step_ex = _step_ex


def argmax_batch(logits_bits: np.ndarray, V: int | None = None, threads: int = 1) -> np.ndarray:
    """[rows, stride] uint16 -> [rows] int32; V defaults to the row length."""
    lg = logits_bits
    assert lg.ndim == 2 and lg.dtype == np.uint16 and lg.strides[1] == 2
    rows, stride = lg.shape[0], lg.strides[0] // 2
    V = lg.shape[1] if V is None else V
    out = np.empty(rows, np.int32)
    _load().oracle_argmax_batch(lg.ctypes.data_as(_u16p), stride, rows, V, _i32(out), threads)
    return out


def accept(drafts: np.ndarray, n_draft: int, argmax: np.ndarray):
    K = drafts.shape[0]
    d = np.ascontiguousarray(drafts, np.int32)
    a = np.ascontiguousarray(argmax, np.int32)
    acc = np.empty(K + 1, np.int32)
    n = _load().oracle_accept(_i32(d), n_draft, _i32(a), K, _i32(acc))
    return acc, int(n)


def accept_batch(drafts: np.ndarray, n_draft: np.ndarray, argmax: np.ndarray):
    B, K = drafts.shape
    acc = np.empty((B, K + 1), np.int32)
    n_acc = np.empty(B, np.int32)
    _load().oracle_accept_batch(B, K, _i32(drafts), _i32(n_draft), _i32(argmax), _i32(acc), _i32(n_acc))
    return acc, n_acc


def multi_draft(members, slots, weights, state, matched_len, new_tokens, n_new, K, min_match):
    """Composite drafting over several automata (Section 5.4.2: the session's own context plus the
    top-K retrieved contexts, "the similarity scores determine the weights of each SAM").

    The paper names the ingredients but not the rule; the reading taken here: every stream b has M
    slots, slot m naming one member automaton (slots[b, m], -1 = empty) with a weight; each slot
    keeps its own (state, matched_len) and follows the new tokens in its own automaton; the draft
    comes from the slot with the largest weight * matched_len (float32 product) among the slots
    whose match reaches min_match, the lowest slot winning ties; no such slot, no draft.

    members: list of OracleSAM; slots [B, M] int32; weights [B, M] float32; state, matched_len
    [B, M] int32 (updated in place); new_tokens [B, ld], n_new [B].
    Returns (drafts [B, K], n_draft [B], chosen [B] slot or -1)."""
    B, M = slots.shape
    drafts = np.full((B, K), -1, np.int32)
    n_draft = np.zeros(B, np.int32)
    chosen = np.full(B, -1, np.int32)
    for b in range(B):
        best_score, best_m = None, -1
        for m in range(M):
            if slots[b, m] < 0:
                continue
            sam = members[int(slots[b, m])]
            s, L = sam.walk(int(state[b, m]), int(matched_len[b, m]), new_tokens[b, :max(0, int(n_new[b]))])
            state[b, m], matched_len[b, m] = s, L
            if L < min_match:
                continue
            score = np.float32(weights[b, m]) * np.float32(L)
            if best_score is None or score > best_score:
                best_score, best_m = score, m
        if best_m >= 0:
            sam = members[int(slots[b, best_m])]
            d, nd = sam.draft(int(state[b, best_m]), int(matched_len[b, best_m]), K, min_match)
            drafts[b], n_draft[b], chosen[b] = d, nd, best_m
    return drafts, n_draft, chosen
