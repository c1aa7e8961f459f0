"""Vocabulary-parallel vocab pass: the logits of a tensor-parallel LM head are split over V across ranks.  Each
rank runs the vocab pass on its shard and leaves per-row pieces (log-sum-exp parts and its K best keys); one
all-gather of 280 bytes per row and rank brings every rank's pieces into local memory; a merge kernel then gives
the full rows' candidates and log-probabilities on every rank.  The exchange is the only collective."""
from __future__ import annotations

import torch

from .binding import VOCAB_PARTIAL_BYTES


def vocab_range(V: int, rank: int, world: int, align: int = 8) -> tuple[int, int]:
    """Token ids [lo, hi) of `rank`: contiguous, in rank order, starts on multiples of `align` (16 bytes of bf16)."""
    if world < 1 or not (0 <= rank < world) or V < world:
        raise ValueError("bad shard arguments")
    per = -(-V // world)
    per = -(-per // align) * align
    if (world - 1) * per >= V:
        raise ValueError("vocabulary too small for this many aligned shards")
    lo = rank * per
    return lo, min(V, lo + per)


def gather_partials(parts: torch.Tensor, group=None) -> torch.Tensor:
    """All ranks' partials in rank order: uint8 [rows, 280] -> uint8 [world, rows, 280].  With no process group
    (single process) the result is this rank's alone."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return parts.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(parts.shape), dtype=parts.dtype, device=parts.device)
    dist.all_gather(list(out.unbind(0)), parts.contiguous(), group=group)
    return out


def vocab_pass_parallel(g, logits_shard, V: int, ids, lp, lse, row_status, group=None):
    """g: a context created with V = this rank's shard width.  Outputs are the full rows' on every rank."""
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    rows = logits_shard.shape[0] * logits_shard.shape[1]
    parts = torch.empty((rows, VOCAB_PARTIAL_BYTES), dtype=torch.uint8, device=logits_shard.device)
    g.vocab_pass_partial(logits_shard, parts)
    allp = gather_partials(parts, group)
    offsets = [vocab_range(V, r, world)[0] for r in range(world)]
    g.vocab_merge(allp, offsets, ids, lp, lse, row_status)
