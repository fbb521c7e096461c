"""Closed-loop backend that runs every step through the C-ABI CUDA library (device logits)."""
from __future__ import annotations

import numpy as np
import torch

import paper_2512_18337_b200 as S


def bits_to_device(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    """uint16 bf16 bit patterns (host) -> torch.bfloat16 tensor on the device, same shape."""
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


class CudaBackend:
    def __init__(self, cfg, corpus, logits_dev: torch.Tensor, index: S.SamIndex | None = None, device="cuda:0"):
        self.cfg = cfg
        self.device = device
        self.index = index if index is not None else S.SamIndex(corpus, [cfg.separator], device=device)
        B, K = cfg.B, cfg.K
        assert logits_dev.dtype == torch.bfloat16 and logits_dev.is_contiguous()
        self.logits = logits_dev.view(B * (K + 1), -1)
        self.stride = self.logits.shape[1]
        self.raw = self.logits.view(torch.int16)
        i32 = dict(dtype=torch.int32, device=device)
        self.state = torch.zeros(B, **i32)
        self.mlen = torch.zeros(B, **i32)
        self.drafts = torch.full((B, K), -7, **i32)
        self.n_draft = torch.zeros(B, **i32)
        self.argmax = torch.full((B, K + 1), -7, **i32)
        self.accepted = torch.full((B, K + 1), -7, **i32)
        self.n_accepted = torch.zeros(B, **i32)
        self.flags = 0              # SAM_STEP_* options used by launch_step
        self.chain_row_lists = False  # with SAM_STEP_SKIP_UNUSED_ROWS: let each step list the rows of the next one
        self._list_ready = False
        self.counters = None        # optional int64[SAM_N_COUNTERS] device tensor
        self.ws_bytes = S.sam_workspace_bytes(B, K)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=device)
        S.sam_workspace_init(self.ws, self.ws_bytes)

    def prime(self, toks, n):
        c = self.cfg
        t = torch.from_numpy(np.ascontiguousarray(toks)).to(self.device)
        nn = torch.from_numpy(n).to(self.device)
        S.sam_draft(self.index.handle, c.B, self.state, self.mlen, t, t.shape[1], nn, c.K, c.min_match,
                    self.drafts, self.n_draft)
        torch.cuda.synchronize()
        return self.drafts.cpu().numpy(), self.n_draft.cpu().numpy()

    def poke(self, rows, cols, bits, keep):
        r = torch.from_numpy(rows).to(self.device)
        c = torch.from_numpy(cols).to(self.device)
        v = torch.from_numpy(bits.view(np.int16)).to(self.device)
        k = torch.from_numpy(keep).to(self.device)
        saved = self.raw[r[k], c[k]].clone()
        self.raw[r, c] = v
        return saved

    def unpoke(self, rows, cols, saved):
        r = torch.from_numpy(rows).to(self.device)
        c = torch.from_numpy(cols).to(self.device)
        self.raw[r, c] = saved

    def launch_step(self):
        """Enqueue one fused step on the current stream (drafts/n_draft are updated in place)."""
        c = self.cfg
        flags = self.flags
        if self.chain_row_lists and (flags & S.SAM_STEP_SKIP_UNUSED_ROWS):
            # drafts / n_draft are fed straight back, so from the second step on the previous step's list is the one
            if self._list_ready:
                flags |= S.SAM_STEP_ROW_LIST_READY
            self._list_ready = True
        S.sam_step_ex(self.index.handle, self.logits, self.stride, c.B, c.K, c.vocab, self.drafts, self.n_draft,
                      self.argmax, self.accepted, self.n_accepted, self.state, self.mlen, c.min_match,
                      self.drafts, self.n_draft, flags, self.counters, self.ws, self.ws_bytes)

    def status(self) -> int:
        return S.sam_workspace_status(self.ws, self.cfg.B, self.cfg.K)

    def step(self, drafts, n_draft):
        # the device already holds drafts/n_draft from the previous call; the arguments are the host copies
        self.launch_step()
        torch.cuda.synchronize()
        return dict(argmax=self.argmax.cpu().numpy(), accepted=self.accepted.cpu().numpy(),
                    n_accepted=self.n_accepted.cpu().numpy(), drafts=self.drafts.cpu().numpy(),
                    n_draft=self.n_draft.cpu().numpy(), state=self.state.cpu().numpy(),
                    matched_len=self.mlen.cpu().numpy())
