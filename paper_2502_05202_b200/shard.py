"""Sharding over more than one GPU.

Rows: sequences are independent, so a batch is split into contiguous blocks of
rows, one per rank; the id map is replicated and nothing is exchanged while
verifying.  Only if one rank wants every result does a gather of the two int32
outputs follow.

Vocabulary (tensor-parallel LM heads): every rank holds a slice of each logit
row; ``ShardedVerifier`` strings the four local calls of the library together
with the three small exchanges between them.  The exchange is a callable, so
that the same driver runs over ``torch.distributed`` (NCCL on GPUs) and, for
tests on one GPU, over a plain stack of the shards' buffers.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Sequence, Tuple

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


def vocab_slice(V: int, rank: int, world: int) -> Tuple[int, int, int]:
    """(begin, count, width) of the ids of shard ``rank``: ``width = ceil(V / world)`` ids per shard,
    trailing shards hold what is left (possibly nothing).  The same rule as tli_shard_create()."""
    if not (0 <= rank < world) or V < 1:
        raise ValueError("bad rank/world/V")
    width = -(-V // world)
    begin = min(V, rank * width)
    return begin, min(V, (rank + 1) * width) - begin, width


def all_gather_dist(local: torch.Tensor, group=None) -> torch.Tensor:
    """[world, *local.shape]: every rank's buffer, in rank order (torch.distributed; NCCL on GPUs)."""
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous(), group=group)
    return out


class ShardedVerifier:
    """One shard of a vocabulary-sharded verification: context, scratch and exchange buffers.

    ``step1 .. step4`` are the four local calls; ``verify`` runs them with ``all_gather`` (a callable
    taking this shard's buffer and returning all shards' buffers stacked in shard order) between them
    and ``max_reduce`` (element-wise maximum over shards of an int32 tensor, in place) at the end.
    """

    def __init__(self, V_t: int, V_d: int, id_map, n_shards: int, shard: int, device: int = 0):
        from . import tli
        self.tli = tli
        self.device = torch.device("cuda", device)
        self.n_shards, self.shard = n_shards, shard
        self.ctx = tli.tli_shard_create(device, V_t, V_d, id_map, n_shards, shard)
        self.info = tli.tli_shard_info(self.ctx)

    def close(self) -> None:
        if self.ctx:
            self.tli.tli_destroy(self.ctx)
            self.ctx = 0

    def prepare(self, target_slice, drafter_slice, draft_ids, temperature, uniforms) -> Dict[str, torch.Tensor]:
        """Outputs, scratch and exchange buffers for one call; ``target_slice`` / ``drafter_slice`` are this
        shard's [B, K+1, width] / [B, K, width] slices (columns beyond the shard's id count are not read)."""
        tli, lib = self.tli, self.tli.load()
        B, K1, _ = target_slice.shape
        K = K1 - 1
        dt = tli.TLI_F32 if target_slice.dtype == torch.float32 else tli.TLI_BF16
        dev = self.device
        st = {"accepted": torch.empty(B, dtype=torch.int32, device=dev),
              "next_token": torch.empty(B, dtype=torch.int32, device=dev),
              "row_status": torch.empty(B, dtype=torch.int32, device=dev),
              "p_draft": torch.empty(B, K, dtype=torch.float32, device=dev),
              "q_draft": torch.empty(B, K, dtype=torch.float32, device=dev),
              "ws": torch.empty(lib.tli_shard_workspace_bytes(self.ctx, B, K, dt), dtype=torch.uint8, device=dev),
              "record": torch.empty(lib.tli_shard_record_bytes(self.ctx, B, K) // 8, dtype=torch.float64, device=dev),
              "rows": torch.empty(lib.tli_shard_rows_bytes(self.ctx, B, dt), dtype=torch.uint8, device=dev),
              "mass": torch.empty(B, 2, dtype=torch.float64, device=dev)}
        st["args"] = tli.make_args(target_slice, drafter_slice, draft_ids, temperature, uniforms, st["accepted"],
                                   st["next_token"], st["ws"], st["row_status"], st["p_draft"], st["q_draft"])
        st["keep"] = (target_slice, drafter_slice, draft_ids, temperature, uniforms)
        return st

    def step1(self, st) -> torch.Tensor:
        self.tli.tli_shard_stats(self.ctx, st["args"], st["record"])
        return st["record"]

    def step2(self, st, records_all: torch.Tensor) -> torch.Tensor:
        st["records_all"] = records_all.contiguous()
        self.tli.tli_shard_decide(self.ctx, st["args"], st["records_all"], st["rows"])
        return st["rows"]

    def step3(self, st, rows_all: torch.Tensor) -> torch.Tensor:
        st["rows_all"] = rows_all.contiguous()
        self.tli.tli_shard_weights(self.ctx, st["args"], st["rows_all"], st["mass"])
        return st["mass"]

    def step4(self, st, masses_all: torch.Tensor) -> torch.Tensor:
        st["masses_all"] = masses_all.contiguous()
        self.tli.tli_shard_select(self.ctx, st["args"], st["rows_all"], st["masses_all"])
        return st["next_token"]

    def verify(self, target_slice, drafter_slice, draft_ids, temperature, uniforms,
               all_gather: Callable[[torch.Tensor], torch.Tensor] = all_gather_dist,
               max_reduce: Optional[Callable[[torch.Tensor], None]] = None) -> Dict[str, torch.Tensor]:
        st = self.prepare(target_slice, drafter_slice, draft_ids, temperature, uniforms)
        self.step2(st, all_gather(self.step1(st)))
        self.step3(st, all_gather(st["rows"]))
        self.step4(st, all_gather(st["mass"]))
        if max_reduce is None:
            dist.all_reduce(st["next_token"], op=dist.ReduceOp.MAX)
        else:
            max_reduce(st["next_token"])
        return {k: st[k] for k in ("accepted", "next_token", "row_status", "p_draft", "q_draft")}


def verify_on_one_device(shards: Sequence["ShardedVerifier"], target_slices, drafter_slices, draft_ids, temperature,
                         uniforms) -> Dict[str, torch.Tensor]:
    """All shards of a sharded verification on one device, one after the other (tests, and measurements
    where only one GPU is to be had): the exchanges are plain stacks of the shards' buffers."""
    sts = [s.prepare(zt, zd, draft_ids, temperature, uniforms) for s, zt, zd in zip(shards, target_slices, drafter_slices)]
    records = torch.stack([s.step1(st) for s, st in zip(shards, sts)])
    rows = torch.stack([s.step2(st, records) for s, st in zip(shards, sts)])
    masses = torch.stack([s.step3(st, rows) for s, st in zip(shards, sts)])
    tokens = torch.stack([s.step4(st, masses) for s, st in zip(shards, sts)])
    out = {k: sts[0][k] for k in ("accepted", "row_status", "p_draft", "q_draft")}
    out["next_token"] = tokens.max(dim=0).values
    out["per_shard"] = sts
    return out
