"""Worker-sharded rTop-k round over several processes (one per GPU).

Workers are independent until the master's average (Algorithm 1: the node loop, then
ghat = (1/n) sum_i ghat_i), so the W workers are split by rows across ranks.  Each rank sparsifies
its rows with ``worker_base`` = its first global worker id (the subsets then equal the single-process
run), the fixed-size messages are exchanged with one all-gather, and every rank aggregates all W
messages into the same dense update.

The functions take the sparsify / aggregate callables as arguments so that the identical sharding
logic runs with the CUDA library on GPUs and, in CPU tests, with any stand-in.
"""
from __future__ import annotations

from typing import Callable, Tuple

import torch
import torch.distributed as dist


def shard_rows(W_total: int, world: int, rank: int) -> Tuple[int, int]:
    """(first global worker id, number of workers) of ``rank``: contiguous, sizes differ by <= 1."""
    base, extra = divmod(W_total, world)
    rows = base + (1 if rank < extra else 0)
    begin = rank * base + min(rank, extra)
    return begin, rows


def gather_messages(idx_local: torch.Tensor, val_local: torch.Tensor, W_total: int, world: int, rank: int,
                    group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """All-gathers [rows, k] message blocks into [W_total, k], ordered by global worker id."""
    k = idx_local.shape[1]
    if world == 1:
        return idx_local, val_local
    counts = [shard_rows(W_total, world, r)[1] for r in range(world)]
    if len(set(counts)) == 1:
        idx_all = torch.empty((W_total, k), dtype=idx_local.dtype, device=idx_local.device)
        val_all = torch.empty((W_total, k), dtype=val_local.dtype, device=val_local.device)
        dist.all_gather_into_tensor(idx_all, idx_local.contiguous(), group=group)
        dist.all_gather_into_tensor(val_all, val_local.contiguous(), group=group)
        return idx_all, val_all
    # uneven shards: pad every block to the largest shard, gather, then drop the padding rows
    cmax = max(counts)

    def padded(x):
        buf = torch.zeros((cmax, k), dtype=x.dtype, device=x.device)
        buf[: x.shape[0]] = x
        return buf

    idx_pad = torch.empty((world * cmax, k), dtype=idx_local.dtype, device=idx_local.device)
    val_pad = torch.empty((world * cmax, k), dtype=val_local.dtype, device=val_local.device)
    dist.all_gather_into_tensor(idx_pad, padded(idx_local), group=group)
    dist.all_gather_into_tensor(val_pad, padded(val_local), group=group)
    keep = torch.cat([torch.arange(r * cmax, r * cmax + c, device=idx_local.device) for r, c in enumerate(counts)])
    return idx_pad.index_select(0, keep), val_pad.index_select(0, keep)


def sharded_round(sparsify: Callable, aggregate: Callable, grad_local: torch.Tensor,
                  residual_local: torch.Tensor, W_total: int, world: int, rank: int, group=None):
    """One round.  ``sparsify(grad, residual, worker_base) -> (idx [rows,k], val [rows,k])`` updates the
    residual in place; ``aggregate(idx_all [W,k], val_all [W,k]) -> out``.  Returns (idx_all, val_all, out)."""
    begin, rows = shard_rows(W_total, world, rank)
    assert grad_local.shape[0] == rows and residual_local.shape[0] == rows
    idx_l, val_l = sparsify(grad_local, residual_local, begin)
    idx_all, val_all = gather_messages(idx_l, val_l, W_total, world, rank, group)
    return idx_all, val_all, aggregate(idx_all, val_all)
