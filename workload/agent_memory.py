"""Seeded generator of agent-memory-shaped inputs for the draft+verify path.

The paper measures on agent trajectories of a public browsing benchmark and a
cross-session corpus made of the generated sequences of all other questions
(Section 6.5, "Evaluation on AgentSAM").  Those are not available, so inputs
here are synthetic stand-ins with the same structure: Zipf-distributed token
sessions in which a fraction of every session is copied from earlier sessions
(the "frequently revisited" retrieved content of Section 5.4.1), one separator
token between sessions, request streams that replay mutated corpus spans, and
bf16 N(0,1) logits in which the drafted token is planted as the row maximum
with a given probability.

Everything is drawn from ``numpy.random.Generator(PCG64([seed, purpose]))`` so
each array depends only on (config, purpose), never on call order.

Nothing in this file implements the method (no automaton, no argmax, no accept
logic): it only produces inputs and applies/undoes the planted logits.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import numpy as np

# purposes for independent random streams
_P_CORPUS, _P_COPY, _P_SCRIPT, _P_NOISE, _P_PLANT, _P_TIE, _P_FEED = range(7)


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    sessions: int          # number of sessions in the corpus
    session_len: int       # tokens per session
    vocab: int             # V; token ids are in [0, V); the separator id is V
    zipf_s: float          # Zipf exponent of the token distribution
    copy_frac: float       # fraction of each session replaced by copied spans
    span_lo: int           # copied / script span length ~ U[span_lo, span_hi]
    span_hi: int
    B: int                 # request streams
    steps: int             # closed-loop steps
    K: int                 # maximum draft length
    min_match: int
    accept_p: float        # probability that a drafted token is planted as row max
    tie_frac: float        # fraction of used rows that get an exact tie at the max
    mutation: float = 0.10  # per-token mutation rate of stream scripts
    prime: int = 32        # script tokens fed to each stream before step 0
    seed: int = 0

    @property
    def separator(self) -> int:
        return self.vocab

    @property
    def n_corpus(self) -> int:
        return self.sessions * self.session_len + self.sessions - 1

    @property
    def rows(self) -> int:
        return self.B * (self.K + 1)

    @property
    def script_len(self) -> int:
        return self.prime + (self.steps + 2) * (self.K + 1)

    def scaled(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


CONFIGS: List[WorkloadConfig] = [
    WorkloadConfig("cfg0_tiny", 4, 2000, 1000, 1.1, 0.30, 8, 64,
                   B=4, steps=16, K=8, min_match=2, accept_p=0.7, tie_frac=0.01, seed=0),
    WorkloadConfig("cfg1_1M", 256, 4096, 151936, 1.1, 0.40, 16, 256,
                   B=64, steps=64, K=8, min_match=2, accept_p=0.7, tie_frac=0.0, seed=1),
    WorkloadConfig("cfg2_16M_B256_K16", 4096, 4096, 151936, 1.05, 0.50, 16, 512,
                   B=256, steps=128, K=16, min_match=3, accept_p=0.6, tie_frac=0.0, seed=2),
    WorkloadConfig("cfg3_verify_heavy", 1024, 4096, 151936, 1.1, 0.40, 16, 256,
                   B=512, steps=8, K=16, min_match=2, accept_p=0.5, tie_frac=0.01, seed=3),
    WorkloadConfig("cfg4_long_trace", 8192, 8192, 151936, 1.05, 0.70, 32, 1024,
                   B=1024, steps=64, K=32, min_match=4, accept_p=0.7, tie_frac=0.0, seed=4),
    # the shape of the paper's own evaluation (Section 6.5: batch size 4, one autoregressive + three speculative
    # tokens per step), on the 1M-token corpus: a latency case, not a bandwidth case
    WorkloadConfig("cfg5_paper_eval_shape_B4_K3", 256, 4096, 151936, 1.1, 0.40, 16, 256,
                   B=4, steps=64, K=3, min_match=2, accept_p=0.7, tie_frac=0.0, seed=5),
]


def _rng(cfg: WorkloadConfig, purpose: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([cfg.seed, purpose]))


# --------------------------------------------------------------------------- bf16 bits
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even. NaN-free input."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# --------------------------------------------------------------------------- tokens
def zipf_cdf(vocab: int, s: float) -> np.ndarray:
    """CDF of P(rank r) ~ r^-s over ranks 1..vocab; token id = rank - 1."""
    w = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    c /= c[-1]
    return c


def _draw_zipf(rng: np.random.Generator, cdf: np.ndarray, n: int) -> np.ndarray:
    ids = np.searchsorted(cdf, rng.random(n), side="right")
    return np.minimum(ids, len(cdf) - 1).astype(np.int32)


def make_corpus(cfg: WorkloadConfig) -> np.ndarray:
    """Flat int32 corpus: session_0 SEP session_1 SEP ... session_{S-1} (no trailing SEP).

    Sessions i >= 1 have about copy_frac of their tokens overwritten by spans
    copied from uniformly chosen earlier sessions (overlaps counted naively).
    """
    cdf = zipf_cdf(cfg.vocab, cfg.zipf_s)
    ln = cfg.session_len
    sess = _draw_zipf(_rng(cfg, _P_CORPUS), cdf, cfg.sessions * ln).reshape(cfg.sessions, ln)
    rng = _rng(cfg, _P_COPY)
    target = int(round(cfg.copy_frac * ln))
    hi = min(cfg.span_hi, ln)
    lo = min(cfg.span_lo, hi)
    for i in range(1, cfg.sessions):
        copied = 0
        while copied < target:
            span = int(rng.integers(lo, hi + 1))
            span = max(1, min(span, target - copied))
            j = int(rng.integers(0, i))
            so = int(rng.integers(0, ln - span + 1))
            do = int(rng.integers(0, ln - span + 1))
            sess[i, do:do + span] = sess[j, so:so + span]
            copied += span
    out = np.full(cfg.n_corpus, cfg.separator, dtype=np.int32)
    view = np.lib.stride_tricks.as_strided(
        out, shape=(cfg.sessions, ln), strides=((ln + 1) * 4, 4))
    view[:, :] = sess
    return out


def make_scripts(cfg: WorkloadConfig, corpus: np.ndarray) -> np.ndarray:
    """[B, script_len] int32: concatenated random corpus spans (never crossing a
    separator) with per-token mutation to a fresh Zipf draw."""
    rng = _rng(cfg, _P_SCRIPT)
    cdf = zipf_cdf(cfg.vocab, cfg.zipf_s)
    ln = cfg.session_len
    hi = min(cfg.span_hi, ln)
    lo = min(cfg.span_lo, hi)
    n = cfg.script_len
    scripts = np.empty((cfg.B, n), dtype=np.int32)
    for b in range(cfg.B):
        filled = 0
        while filled < n:
            span = int(rng.integers(lo, hi + 1))
            sess = int(rng.integers(0, cfg.sessions))
            off = int(rng.integers(0, ln - span + 1))
            start = sess * (ln + 1) + off
            take = min(span, n - filled)
            scripts[b, filled:filled + take] = corpus[start:start + take]
            filled += take
    mut = rng.random((cfg.B, n)) < cfg.mutation
    fresh = _draw_zipf(rng, cdf, cfg.B * n).reshape(cfg.B, n)
    scripts[mut] = fresh[mut]
    return scripts


def make_open_loop_feed(cfg: WorkloadConfig, scripts: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Open-loop feed: per step and stream, the next n ~ U[1, K+1] script tokens.

    Returns (new_tokens [steps, B, K+1] padded with -1, n_new [steps, B])."""
    rng = _rng(cfg, _P_FEED)
    ld = cfg.K + 1
    n_new = rng.integers(1, ld + 1, size=(cfg.steps, cfg.B)).astype(np.int32)
    toks = np.full((cfg.steps, cfg.B, ld), -1, dtype=np.int32)
    pos = np.zeros(cfg.B, dtype=np.int64)
    for t in range(cfg.steps):
        for b in range(cfg.B):
            k = int(n_new[t, b])
            toks[t, b, :k] = scripts[b, pos[b]:pos[b] + k]
            pos[b] += k
    return toks, n_new


# --------------------------------------------------------------------------- logits
def make_noise_logits(cfg: WorkloadConfig, rows: int | None = None) -> np.ndarray:
    """[rows, V] bf16 bit patterns (uint16) of N(0,1) noise; rows defaults to B*(K+1).
    Generated in float32 on the host and rounded to nearest even."""
    rows = cfg.rows if rows is None else rows
    rng = _rng(cfg, _P_NOISE)
    out = np.empty((rows, cfg.vocab), dtype=np.uint16)
    blk = max(1, (1 << 24) // cfg.vocab)
    for r0 in range(0, rows, blk):
        r1 = min(rows, r0 + blk)
        out[r0:r1] = f32_to_bf16_bits(
            rng.standard_normal((r1 - r0, cfg.vocab), dtype=np.float32))
    return out


def planted_value_bits(rowmax_bits: np.ndarray) -> np.ndarray:
    """bf16(float(row max of the noise) + 1): strictly above every noise entry."""
    return f32_to_bf16_bits(bf16_bits_to_f32(rowmax_bits) + np.float32(1.0))


class ClosedLoopFeeder:
    """Stand-in for the target model in the closed loop.

    Per step it decides, for every used logits row (b, j) with j <= n_draft[b],
    which token the "model" wants: the drafted token with probability accept_p
    (rows j < n_draft[b]), otherwise the stream's script token at pos_b + j.
    It returns the sparse overwrite list that makes that token the unique row
    maximum (plus, for a tie_frac share of used rows, one extra entry equal to
    the maximum at a random other column).  All random numbers are pre-drawn.

    The caller owns the logits (numpy on the host or a torch tensor on the
    device), applies the overwrite list, runs the step, restores the original
    entries and calls ``advance(n_accepted)``.
    """

    def __init__(self, cfg: WorkloadConfig, scripts: np.ndarray, rowmax_bits: np.ndarray):
        self.cfg = cfg
        self.scripts = scripts
        self.pos = np.full(cfg.B, cfg.prime, dtype=np.int64)
        self.plant_bits = planted_value_bits(rowmax_bits).reshape(cfg.B, cfg.K + 1)
        shape = (cfg.steps, cfg.B, cfg.K + 1)
        self.u_plant = _rng(cfg, _P_PLANT).random(shape, dtype=np.float32)
        tr = _rng(cfg, _P_TIE)
        self.u_tie = tr.random(shape, dtype=np.float32)
        self.tie_col = tr.integers(0, cfg.vocab, size=shape, dtype=np.int64)

    def prime_tokens(self) -> Tuple[np.ndarray, np.ndarray]:
        """Tokens fed to every stream before step 0: ([B, prime], [B])."""
        c = self.cfg
        return (np.ascontiguousarray(self.scripts[:, :c.prime]),
                np.full(c.B, c.prime, dtype=np.int32))

    def overwrites(self, step: int, drafts: np.ndarray, n_draft: np.ndarray) -> Dict[str, np.ndarray]:
        """Sparse logits overwrites for this step, in application order.

        Returns dict(row=[M] flat row index b*(K+1)+j, col=[M], bits=[M] uint16,
        target=[B, K+1] wanted token per used row, -1 elsewhere)."""
        c = self.cfg
        K1 = c.K + 1
        j = np.arange(K1)[None, :]
        nd = n_draft.astype(np.int64)[:, None]
        used = j <= nd
        is_draft_row = j < nd
        script_idx = self.pos[:, None] + j
        want = np.take_along_axis(self.scripts, script_idx, axis=1).astype(np.int64)
        dr = np.concatenate([drafts.astype(np.int64), np.full((c.B, 1), -1, np.int64)], axis=1)
        take_draft = is_draft_row & (self.u_plant[step] < c.accept_p)
        want = np.where(take_draft, dr, want)
        target = np.where(used, want, -1)
        b_idx, j_idx = np.nonzero(used)
        rows = b_idx * K1 + j_idx
        cols = target[b_idx, j_idx]
        bits = self.plant_bits[b_idx, j_idx]
        tie = self.u_tie[step][b_idx, j_idx] < c.tie_frac
        if tie.any():
            tcol = self.tie_col[step][b_idx, j_idx][tie]
            tcol = np.where(tcol == cols[tie], (tcol + 1) % c.vocab, tcol)
            rows = np.concatenate([rows, rows[tie]])
            cols = np.concatenate([cols, tcol])
            bits = np.concatenate([bits, bits[tie]])
        return dict(row=rows.astype(np.int64), col=cols.astype(np.int64),
                    bits=bits.astype(np.uint16), target=target.astype(np.int64))

    def advance(self, n_accepted: np.ndarray) -> None:
        self.pos += n_accepted.astype(np.int64)
