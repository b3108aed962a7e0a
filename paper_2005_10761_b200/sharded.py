"""Worker-sharded rTop-k round over several processes (one per GPU).

Workers are independent until the master's average (Algorithm 1: the node loop, then
ghat = (1/n) sum_i ghat_i), so the W workers are split by rows across ranks.  Each rank sparsifies
its rows with ``worker_base`` = its first global worker id (the subsets then equal the single-process
run) into one buffer of 8-byte (index, value) pairs, the buffers are exchanged with ONE all-gather of a
fixed size per rank, and every rank aggregates the gathered buffer in place into the same dense update.

Rows are dealt out in blocks of ceil(W / world): rank p holds workers [p * c, min(W, (p + 1) * c)).
The last ranks may hold fewer rows (or none), but the step time is that of the largest shard either
way, and with this split the gathered buffer [world * c, k] holds the W messages in global worker
order in its first W rows, whatever the shard sizes: no re-ordering, no copy, no second collective.

The functions take the sparsify / aggregate callables as arguments so that the identical sharding
logic runs with the CUDA library on GPUs and, in CPU tests, with any stand-in.  Nothing here reads
another rank's memory: the gathered messages land in this rank's own buffer before any kernel uses them.
"""
from __future__ import annotations

from typing import Callable, Tuple

import torch
import torch.distributed as dist


def shard_block(W_total: int, world: int) -> int:
    """Rows per rank of the block split: ceil(W / world)."""
    return (W_total + world - 1) // world


def shard_rows(W_total: int, world: int, rank: int) -> Tuple[int, int]:
    """(first global worker id, number of workers) of ``rank``: blocks of ceil(W / world) rows."""
    c = shard_block(W_total, world)
    begin = min(W_total, rank * c)
    return begin, min(W_total, begin + c) - begin


class Exchange:
    """The buffers of the one all-gather, allocated once: ``send`` [c, k] pairs of this rank (rows beyond
    its shard stay zero and are never read), ``recv`` [world * c, k] pairs of everybody."""

    def __init__(self, W_total: int, k: int, world: int, rank: int, device, group=None, always_collective=False):
        """``always_collective``: issue the all-gather even in a group of one rank (it then copies ``send``
        to ``recv``), so that a single process runs exactly the calls of a sharded job."""
        self.W_total, self.k, self.world, self.rank, self.group = W_total, k, world, rank, group
        self.c = shard_block(W_total, world)
        self.begin, self.rows = shard_rows(W_total, world, rank)
        self.collective = world > 1 or always_collective
        self.send = torch.zeros((self.c, k), dtype=torch.int64, device=device)
        self.recv = torch.zeros((world * self.c, k), dtype=torch.int64, device=device) if self.collective else self.send

    def local_pairs(self) -> torch.Tensor:
        """Where this rank's sparsify call writes its messages: [rows, k] pairs."""
        return self.send[: self.rows]

    def gather(self) -> torch.Tensor:
        """All ranks' messages, [W_total, k] pairs in global worker order (a view of ``recv``)."""
        if self.collective:
            dist.all_gather_into_tensor(self.recv, self.send, group=self.group)
        return self.recv[: self.W_total]


def sharded_round(sparsify_pairs: Callable, aggregate_pairs: Callable, grad_local: torch.Tensor,
                  residual_local: torch.Tensor, ex: Exchange):
    """One round.  ``sparsify_pairs(grad, residual, worker_base, pairs [rows, k])`` fills ``pairs`` and
    updates the residual in place; ``aggregate_pairs(pairs_all [W, k]) -> out``.  Returns (pairs_all, out)."""
    assert grad_local.shape[0] == ex.rows and residual_local.shape[0] == ex.rows
    if ex.rows > 0:
        sparsify_pairs(grad_local, residual_local, ex.begin, ex.local_pairs())
    pairs_all = ex.gather()
    return pairs_all, aggregate_pairs(pairs_all)


def pack_pairs(idx: torch.Tensor, val: torch.Tensor) -> torch.Tensor:
    """(index, value) arrays -> 8-byte pairs: low half the index, high half the value's bit pattern.
    (Host-side helper for tests and stand-ins; the CUDA library writes pairs itself.)"""
    lo = idx.to(torch.int64) & 0xFFFFFFFF
    hi = val.contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    return lo | (hi << 32)


def unpack_pairs(pairs: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """8-byte pairs -> (int32 index bits, float32 values)."""
    idx = (pairs & 0xFFFFFFFF).to(torch.int32)          # (indices are below 2^31)
    val = (pairs >> 32).to(torch.int32).view(torch.float32)
    return idx, val
