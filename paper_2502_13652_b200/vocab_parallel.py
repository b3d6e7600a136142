"""Vocabulary-parallel levels over several GPUs: the exchange step.

When the draft model's output layer is sharded over the vocabulary, every rank holds the logits
of one contiguous token range of every frontier row.  A level then costs each rank one sharded
vocabulary pass, one export of per-row records (288 bytes per row), ONE all-gather of those
records, and the prune from the gathered records, which every rank runs identically, so that
all ranks hold the same tree and the same next frontier (Sec. 4.2.1, Eq. 2, Sec. 4.2.2 for the
pass; Eq. 1, Eq. 4 and Alg. 1 for the prune).  The all-gather is the only collective of the
path; it goes through `torch.distributed` (NCCL between GPUs).
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import torch
import torch.distributed as dist


def shard_ranges(vocab: int, world: int, elem_bytes: int) -> List[Tuple[int, int]]:
    """Contiguous token ranges, one per rank, in rank order; every range starts on a 16-byte boundary
    of the row (the library's alignment rule) and the last one takes the remainder."""
    step = 16 // elem_bytes
    per = -(-vocab // world)
    per = -(-per // step) * step
    out = []
    for r in range(world):
        v0 = min(vocab, r * per)
        v1 = min(vocab, (r + 1) * per)
        out.append((v0, v1))
    if any(v1 <= v0 for v0, v1 in out):
        raise ValueError(f"vocabulary of {vocab} tokens is too small for {world} shards")
    return out


def gather_row_records(local: torch.Tensor, group: Optional[dist.ProcessGroup] = None,
                       out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All-gathers one rank's records [B, F, bytes] into [world, B, F, bytes], shard-major in rank order
    (= ascending token order when the ranges come from `shard_ranges`).  `out`: a buffer of that shape to
    gather into (allocated if absent)."""
    world = dist.get_world_size(group)
    if out is None:
        out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    assert out.is_contiguous() and tuple(out.shape) == (world,) + tuple(local.shape)
    dist.all_gather_into_tensor(out.view((world * local.shape[0],) + tuple(local.shape[1:])), local.contiguous(),
                                group=group)                               # concatenated along the first dimension
    return out


class ExchangeBuffers:
    """The buffers of the exchange, allocated once per context and process group, so that a level allocates nothing."""

    def __init__(self, ctx, group: Optional[dist.ProcessGroup] = None):
        world = dist.get_world_size(group)
        self.records = ctx.new_row_records(world)                      # [world, B, F, bytes]
        self.local = ctx.new_row_records(1)[0]                         # [B, F, bytes]
        self.keys = torch.zeros((world, ctx.B, ctx.Nw), dtype=torch.int64, device=self.records.device)
        self.local_keys = torch.zeros((ctx.B, ctx.Nw), dtype=torch.int64, device=self.records.device)
        self.walk_keys = torch.zeros((world, ctx.B), dtype=torch.int64, device=self.records.device)
        self.local_walk_keys = torch.zeros((ctx.B,), dtype=torch.int64, device=self.records.device)


def vocab_parallel_level(ctx, level: int, shard_logits: torch.Tensor, vocab_begin: int,
                         group: Optional[dist.ProcessGroup] = None, stream=None,
                         buffers: Optional[ExchangeBuffers] = None) -> None:
    """One level of the tree on this rank: `shard_logits` [B, F, count] are this rank's token range
    starting at `vocab_begin`.  The collective runs on the current stream, after the export.  Pass the
    `ExchangeBuffers` of the context to keep allocations off this path."""
    buffers = buffers or ExchangeBuffers(ctx, group)
    ctx.c2t_expand_level_shard(level, shard_logits, stream)
    ctx.c2t_export_row_records(level, vocab_begin, buffers.local, stream)
    records = gather_row_records(buffers.local, group, buffers.records)
    ctx.c2t_prune_gathered(level, records, stream)


def vocab_parallel_accept(ctx, target_shard: torch.Tensor, vocab_begin: int,
                          group: Optional[dist.ProcessGroup] = None, stream=None,
                          buffers: Optional[ExchangeBuffers] = None) -> None:
    """The acceptance walk with sharded target logits: this rank's best key per final node, one all-gather of
    8 bytes per node, the walk on every rank."""
    buffers = buffers or ExchangeBuffers(ctx, group)
    ctx.c2t_argmax_shard(target_shard, vocab_begin, buffers.local_keys, stream)
    ctx.c2t_accept_gathered(gather_row_records(buffers.local_keys, group, buffers.keys), stream)



def vocab_parallel_accept_lazy(ctx, target_shard: torch.Tensor, vocab_begin: int,
                               group: Optional[dist.ProcessGroup] = None, stream=None,
                               buffers: Optional[ExchangeBuffers] = None) -> None:
    """The same walk reading only the target rows on the accepted path: D + 1 rounds of "this rank's best key of
    every walking sequence's current row, an all-gather of 8 bytes per sequence, one step of every walk"."""
    buffers = buffers or ExchangeBuffers(ctx, group)
    ctx.c2t_lazy_begin(stream)
    for r in range(1, ctx.D + 2):
        ctx.c2t_lazy_argmax_shard(target_shard, vocab_begin, buffers.local_walk_keys, stream)
        ctx.c2t_lazy_step_gathered(r, gather_row_records(buffers.local_walk_keys, group, buffers.walk_keys), stream)
