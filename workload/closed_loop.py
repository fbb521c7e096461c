"""Closed-loop driver shared by the oracle runs and the CUDA runs.

It only sequences calls: prime the streams, then per step {plant the wanted
tokens into the logits, run the backend's step, undo the planting, advance the
scripts}.  The backend object hides where the logits live (numpy on the host
or a torch tensor on the device) and which implementation runs the step.

Backend protocol (duck-typed):
    prime(tokens [B, P] int32, n [B] int32) -> (drafts [B,K], n_draft [B]) numpy
    poke(rows, cols, bits) -> saved bits            # logits[row, col] = bits, returns previous values
    unpoke(rows, cols, saved)                        # restore
    step(drafts, n_draft) -> dict(argmax, accepted, n_accepted, drafts, n_draft, state, matched_len) numpy
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional

import numpy as np

from .agent_memory import ClosedLoopFeeder, WorkloadConfig


def _first_write_only(rows: np.ndarray, cols: np.ndarray):
    """Indices of the first occurrence of every (row, col) pair, so that saved
    originals are taken before any overwrite of the same element."""
    key = rows.astype(np.int64) * (1 << 32) + cols.astype(np.int64)
    _, first = np.unique(key, return_index=True)
    return np.sort(first)


def run_closed_loop(cfg: WorkloadConfig, feeder: ClosedLoopFeeder, backend,
                    steps: Optional[int] = None,
                    on_step: Optional[Callable[[int, Dict[str, np.ndarray]], None]] = None
                    ) -> List[Dict[str, np.ndarray]]:
    """Runs the loop and returns the per-step outputs (numpy copies)."""
    steps = cfg.steps if steps is None else steps
    toks, n = feeder.prime_tokens()
    drafts, n_draft = backend.prime(toks, n)
    trace: List[Dict[str, np.ndarray]] = []
    for t in range(steps):
        ow = feeder.overwrites(t, drafts, n_draft)
        rows, cols, bits = ow["row"], ow["col"], ow["bits"]
        keep = _first_write_only(rows, cols)
        saved = backend.poke(rows, cols, bits, keep)
        out = backend.step(drafts, n_draft)
        backend.unpoke(rows[keep], cols[keep], saved)
        out = {k: np.array(v, copy=True) for k, v in out.items()}
        out["target"] = ow["target"]
        out["in_drafts"] = drafts
        out["in_n_draft"] = n_draft
        trace.append(out)
        if on_step is not None:
            on_step(t, out)
        feeder.advance(out["n_accepted"])
        drafts, n_draft = out["drafts"], out["n_draft"]
    return trace


class HostLogits:
    """poke/unpoke on a host uint16 [rows, V] array (bf16 bit patterns)."""

    def __init__(self, bits: np.ndarray):
        self.bits = bits

    def poke(self, rows, cols, bits, keep):
        saved = self.bits[rows[keep], cols[keep]].copy()
        self.bits[rows, cols] = bits        # (row, col) pairs are distinct by construction
        return saved

    def unpoke(self, rows, cols, saved):
        self.bits[rows, cols] = saved


def trace_stats(cfg: WorkloadConfig, trace) -> Dict[str, float]:
    """OTE = committed tokens per verification pass; SHR = accepted speculative tokens
    over proposed ones, on steps with a non-empty proposal (Section 6.5 definitions)."""
    acc = sum(int(o["n_accepted"].sum()) for o in trace)
    passes = sum(int(o["n_accepted"].shape[0]) for o in trace)
    prop = sum(int(o["in_n_draft"].sum()) for o in trace)
    hit = sum(int((o["n_accepted"] - 1).sum()) for o in trace)
    nonempty = sum(int((o["in_n_draft"] > 0).sum()) for o in trace)
    return dict(tokens=acc, stream_steps=passes, ote=acc / max(passes, 1),
                shr=hit / max(prop, 1), shr_k=hit / max(cfg.K * nonempty, 1),
                nonempty_frac=nonempty / max(passes, 1),
                mean_n_draft=prop / max(passes, 1))
