"""Batch-row data parallelism: rows of a speculation step never interact (signals, controller
and verification are all per row), so N GPUs each take a contiguous share of the rows and run
the single-GPU step on it.  No collective sits on the data path; the only optional exchange is
an all-gather of the small per-row outputs when one rank wants all of them."""
from __future__ import annotations

from typing import Dict

import torch
import torch.distributed as dist


def row_range(B: int, rank: int, world: int) -> range:
    """Contiguous rows of rank `rank` when B rows are split as evenly as possible."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def gather_rows(local: Dict[str, torch.Tensor], B: int, group=None) -> Dict[str, torch.Tensor]:
    """All-gather per-row outputs (first dimension = local rows) into full-batch tensors, in row
    order.  Works on any backend (NCCL over NVLink on GPUs, gloo in CPU tests)."""
    world = dist.get_world_size(group)
    out = {}
    for k, v in local.items():
        sizes = [len(row_range(B, r, world)) for r in range(world)]
        pad = max(sizes)
        buf = v.new_zeros((pad,) + tuple(v.shape[1:]))
        buf[: v.shape[0]] = v
        parts = [torch.empty_like(buf) for _ in range(world)]
        dist.all_gather(parts, buf, group=group)
        out[k] = torch.cat([p[:n] for p, n in zip(parts, sizes)], dim=0)
    return out
