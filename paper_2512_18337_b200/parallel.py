"""Multi-GPU plumbing (torch.distributed only; no arithmetic of the method lives here).

Streams are independent, so data parallelism needs no communication at all: every rank owns its
streams and a replica of the index.  The one exchange this module offers is for a vocabulary that
is sharded over ranks (tensor-parallel output layer): each rank reduces its shard with
``sam_argmax_partial`` and the packed per-row words are combined by one MAX all-reduce.
"""
from __future__ import annotations


def reduce_argmax_keys(keys, rows: int, group=None):
    """In-place MAX all-reduce of the first `rows` packed words of `keys` (int64 tensor, any device
    the process group supports).  The trailing status word is left alone.  Returns `keys`."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(keys[:rows], op=dist.ReduceOp.MAX, group=group)
    return keys


def shard_bounds(V: int, rank: int, world: int, multiple: int = 8):
    """Columns [lo, hi) of rank's vocabulary shard; shard starts are multiples of `multiple` elements
    so that shard rows stay 16-byte aligned when the full rows are."""
    per = -(-V // world)
    per = -(-per // multiple) * multiple
    lo = min(V, rank * per)
    return lo, min(V, lo + per)
