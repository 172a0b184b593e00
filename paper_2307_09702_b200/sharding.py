"""Sharding of the path over several GPUs (one process per GPU, ``torch.distributed``).

The path has no exchange step: index rows (states) are independent of one
another, and so are the batch rows of a decode step.  A rank therefore builds a
contiguous slab of states with ``fsm_index_build_rows`` from a replicated
automaton and vocabulary, or steps a contiguous slice of the batch against a
replicated index.  The only collective is the optional all-gather that gives
every rank the whole index; it works on whatever backend the process group
uses (NCCL over NVLink for CUDA tensors, gloo for CPU tensors).

This module holds partition arithmetic and the gather only.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def contiguous_shards(n: int, world: int) -> list[tuple[int, int]]:
    """Splits ``range(n)`` into ``world`` contiguous, balanced ``(begin, end)`` pieces
    (the first ``n % world`` pieces are one longer; pieces may be empty)."""
    if n < 0 or world <= 0:
        raise ValueError("n >= 0 and world > 0 required")
    base, extra = divmod(n, world)
    out, begin = [], 0
    for r in range(world):
        end = begin + base + (1 if r < extra else 0)
        out.append((begin, end))
        begin = end
    return out


def state_slab(Q: int, rank: int, world: int) -> tuple[int, int]:
    """States ``[q_begin, q_end)`` whose index rows ``rank`` builds."""
    return contiguous_shards(Q, world)[rank]


def batch_slice(B: int, rank: int, world: int) -> tuple[int, int]:
    """Batch rows ``[b_begin, b_end)`` that ``rank`` decodes."""
    return contiguous_shards(B, world)[rank]


def all_gather_rows(local: torch.Tensor, total_rows: int, group=None) -> torch.Tensor:
    """Concatenates the row slabs of all ranks (slab sizes as ``contiguous_shards``
    gives them) into one ``[total_rows, ...]`` tensor on every rank."""
    world = dist.get_world_size(group)
    shards = contiguous_shards(total_rows, world)
    rank = dist.get_rank(group)
    if local.shape[0] != shards[rank][1] - shards[rank][0]:
        raise ValueError("local slab does not have this rank's row count")
    longest = max(e - b for b, e in shards)
    padded = local.new_zeros((longest,) + tuple(local.shape[1:]))
    padded[: local.shape[0]] = local
    pieces = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(pieces, padded.contiguous(), group=group)
    return torch.cat([pieces[r][: e - b] for r, (b, e) in enumerate(shards)], dim=0)


def equal_slab(n: int, rank: int, world: int) -> tuple[int, int]:
    """Rows ``[begin, end)`` of ``rank`` when every rank gets ``ceil(n / world)`` rows and the
    last ranks take what is left (possibly nothing).  With slabs of one size the gathered
    array is contiguous: row q of the whole sits at position q."""
    per = -(-n // world)
    begin = min(n, rank * per)
    return begin, min(n, begin + per)


def all_gather_slabs_in_place(full: torch.Tensor, total_rows: int, group=None) -> torch.Tensor:
    """All-gather without staging copies.  ``full`` has ``world * ceil(total_rows / world)``
    rows on every rank; rank r has written its ``equal_slab`` at its own position, and after
    the call every rank holds all slabs (rows beyond ``total_rows`` are padding).  One
    collective on tensors the ranks own; no kernel is handed another rank's memory."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    per = -(-total_rows // world)
    if full.shape[0] != world * per:
        raise ValueError("full must have world * ceil(total_rows / world) rows")
    dist.all_gather_into_tensor(full, full[rank * per:(rank + 1) * per], group=group)
    return full[:total_rows]
