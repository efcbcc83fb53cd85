"""Host-side helpers for running the step on several GPUs.

Rollouts (batch rows) are independent for the whole denoising loop, so ranks take disjoint row ranges,
weights are replicated and there is no collective on the data path.  The only communication is the
bookkeeping below (barrier, max of the times, sum of the token counts).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_rows(n_rows: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous row range [lo, hi) of `rank`; ranges are disjoint, cover [0, n_rows) and differ by <= 1 row."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_rows, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def reduce_step_stats(ms: float, tokens: float, device="cpu", group=None) -> Tuple[float, float]:
    """(max over ranks of the elapsed time, sum over ranks of the committed tokens)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(ms), float(tokens)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    n = torch.tensor([tokens], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(n, op=dist.ReduceOp.SUM, group=group)
    return float(t.item()), float(n.item())


def gather_tokens(tokens: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of the final int32 token rows of equally sized shards (the one exchange after a generation)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return tokens
    parts = [torch.empty_like(tokens) for _ in range(dist.get_world_size(group))]
    dist.all_gather(parts, tokens.contiguous(), group=group)
    return torch.cat(parts, dim=0)
