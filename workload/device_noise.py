"""N(0,1) bf16 noise logits drawn on the device (input generation only).

The large workloads have up to 10 GB of logits; drawing them on the host takes minutes, so the
harness draws them once on the GPU with a seeded torch generator and, where the CPU oracle needs
the same bytes, copies them to the host.  No part of the method lives here.
"""
from __future__ import annotations

import numpy as np

from .agent_memory import WorkloadConfig


def make_noise_logits_device(cfg: WorkloadConfig, device):
    """([rows, V] torch.bfloat16 tensor on `device`, [rows] uint16 bf16 bits of every row's maximum)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(1000 + cfg.seed)
    R = cfg.rows
    logits = torch.empty((R, cfg.vocab), dtype=torch.bfloat16, device=device)
    blk = max(1, (1 << 26) // cfg.vocab)
    for r0 in range(0, R, blk):
        r1 = min(R, r0 + blk)
        logits[r0:r1] = torch.randn((r1 - r0, cfg.vocab), generator=g, device=device,
                                    dtype=torch.float32).to(torch.bfloat16)
    rowmax = logits.max(dim=1).values.view(torch.int16).cpu().numpy().view(np.uint16)
    return logits, rowmax


def device_bits_to_host(logits) -> np.ndarray:
    """uint16 host copy of a bf16 device tensor's bit patterns (copied in slabs to bound pinned staging)."""
    import torch
    raw = logits.view(torch.int16)
    out = np.empty(tuple(raw.shape), dtype=np.uint16)
    rows = raw.shape[0]
    blk = max(1, (1 << 28) // max(1, raw.shape[1]))
    for r0 in range(0, rows, blk):
        r1 = min(rows, r0 + blk)
        out[r0:r1] = raw[r0:r1].cpu().numpy().view(np.uint16)
    return out
