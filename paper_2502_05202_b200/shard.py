"""Row sharding for more than one GPU.

Sequences are independent, so a batch is split into contiguous blocks of rows,
one per rank; the id map is replicated and nothing is exchanged while verifying.
Only if one rank wants every result does a gather of the two int32 outputs follow.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def row_block(B: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the rows rank ``rank`` of ``world`` verifies; blocks differ by at most one row."""
    if not (0 <= rank < world) or B < 0:
        raise ValueError("bad rank/world/B")
    base, extra = divmod(B, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def row_blocks(B: int, world: int) -> List[Tuple[int, int]]:
    return [row_block(B, r, world) for r in range(world)]


def gather_rows(local: torch.Tensor, B: int, group=None) -> torch.Tensor:
    """All ranks' row blocks of a per-row tensor, concatenated in row order (every rank gets the result)."""
    world = dist.get_world_size(group)
    blocks = row_blocks(B, world)
    width = max(e - b for b, e in blocks)
    pad = torch.zeros((width,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad, group=group)
    return torch.cat([parts[r][: e - b] for r, (b, e) in enumerate(blocks)], dim=0)
