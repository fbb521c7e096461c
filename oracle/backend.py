"""Closed-loop backend that runs every step with the CPU oracle (host logits).

Test infrastructure like the rest of this package: used by the tests, the smoke check and the
benchmark's CPU legs; it sequences oracle calls and holds the per-stream state, nothing more."""
from __future__ import annotations

import numpy as np

import oracle
from workload import HostLogits


class OracleBackend(HostLogits):
    def __init__(self, cfg, corpus, noise_bits, threads=1):
        super().__init__(noise_bits)
        self.cfg = cfg
        self.sam = oracle.OracleSAM(corpus, [cfg.separator])
        self.state = np.zeros(cfg.B, np.int32)
        self.mlen = np.zeros(cfg.B, np.int32)
        self.threads = threads

    def prime(self, toks, n):
        c = self.cfg
        return self.sam.draft_batch(self.state, self.mlen, toks, n, c.K, c.min_match, self.threads)

    def step(self, drafts, n_draft):
        c = self.cfg
        out = self.sam.step(self.bits, c.B, c.K, c.vocab, drafts, n_draft,
                            self.state, self.mlen, c.min_match, self.threads)
        out["state"] = self.state.copy()
        out["matched_len"] = self.mlen.copy()
        return out
