"""TP-balanced placement, second stage (Section 4.3): the TP group as one storage pool.

At Store every rank holds the packed units of its shard of a checkpoint (``U_r`` rows); the group
redistributes them so that every rank stores at most ``C = ceil(sum U_r / T)`` rows, moving only
remotely owned rows; Load applies the inverse transfer.  The split sizes come from the library
(``dasc_tp_balance``); the transfer here is the plain ``torch.distributed`` variable-split
all-to-all (NCCL on GPUs, gloo on CPU), i.e. the baseline form of the exchange: the library's
device path is one GPU and has no collective.  Both directions are exact row moves.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from .binding import dasc_tp_balance


def gather_unit_counts(local_rows: int, group=None) -> list[int]:
    """Every rank's packed row count ``U_r`` (static per plan: exchange once, reuse for every checkpoint)."""
    world = dist.get_world_size(group)
    out = [None] * world
    dist.all_gather_object(out, int(local_rows), group=group)
    return [int(x) for x in out]


def store_exchange(packed_local: torch.Tensor, units_per_rank, group=None) -> torch.Tensor:
    """Store: ``packed_local`` [U_r, row] (this rank's packed rows, in order) -> the rows this rank stores
    [<= C, row]: consecutive runs of the group-wide sequence, in rank order."""
    rank = dist.get_rank(group)
    _, send = dasc_tp_balance(units_per_rank)
    assert packed_local.shape[0] == int(units_per_rank[rank])
    in_splits = [int(x) for x in send[rank]]                  # what this rank sends to each rank (diagonal: keeps)
    out_splits = [int(x) for x in send[:, rank]]              # what it receives from each rank
    stored = packed_local.new_empty((sum(out_splits),) + tuple(packed_local.shape[1:]))
    dist.all_to_all_single(stored, packed_local.contiguous(), out_splits, in_splits, group=group)
    return stored


def load_exchange(stored: torch.Tensor, units_per_rank, group=None) -> torch.Tensor:
    """Load: the inverse transfer; returns this rank's own packed rows [U_r, row] in their original order."""
    rank = dist.get_rank(group)
    _, send = dasc_tp_balance(units_per_rank)
    in_splits = [int(x) for x in send[:, rank]]               # rows stored here, grouped by owner
    out_splits = [int(x) for x in send[rank]]                 # rows of this rank, grouped by where they were stored
    assert stored.shape[0] == sum(in_splits)
    packed = stored.new_empty((sum(out_splits),) + tuple(stored.shape[1:]))
    dist.all_to_all_single(packed, stored.contiguous(), out_splits, in_splits, group=group)
    return packed
