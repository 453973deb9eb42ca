"""Shards spread over several GPUs (Algorithm 1: process i holds W_i, every process sees the
same batch).  Plumbing only: each step is the single-table call sequence of `binding.Table`
plus the one exchange the forward needs; the backward needs none (Section 3.2).

    rank r owns the shards s with s mod world == r           (des_config_t.shard_world / shard_rank)
    forward : des_forward_partials -> des_rank_partial -> all-gather [world][B][k+4]
              -> des_aggregate_ranks (fixed rank order, then F: the same bits on every rank)
              pooled blocks / first-layer partials Z: des_aggregate locally -> all-reduce(sum)
    backward: des_backward_update on the local table with the replicated upstream gradients

The exchange is `torch.distributed` (NCCL over NVLink / NVSwitch) by default; `gather` /
`reduce` can be replaced, which is how a single-GPU test drives several ranks one after the
other.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch

from .binding import OP_DENSE1, OP_FM, OP_LR, OP_POOL, DeviceBatch, Table


def owned_shards(num_shards: int, world: int, rank: int):
    """The shards of `rank` under the s mod world rule."""
    return [s for s in range(num_shards) if s % max(world, 1) == rank]


def _dist_gather(local: torch.Tensor, world: int) -> torch.Tensor:
    import torch.distributed as dist
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous())       # rank order
    return out


def _dist_reduce(t: torch.Tensor) -> torch.Tensor:
    import torch.distributed as dist
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


class ShardedTable:
    """One rank's table plus the exchange.  `table` must have been created with the same
    shard_world / shard_rank."""

    def __init__(self, table: Table, world: int, rank: int,
                 gather: Optional[Callable[[torch.Tensor, int], torch.Tensor]] = None,
                 reduce: Optional[Callable[[torch.Tensor], torch.Tensor]] = None):
        self.t, self.world, self.rank = table, world, rank
        self.gather = gather or _dist_gather
        self.reduce = reduce or _dist_reduce

    # local half of the forward: everything up to the message this rank sends
    def forward_local(self, ops: int, db: DeviceBatch, pooled: Optional[torch.Tensor] = None,
                      Z: Optional[torch.Tensor] = None):
        t, B = self.t, db.batch
        msg = None
        part_small = None
        if ops & (OP_LR | OP_FM):
            part_small = torch.empty((t.S, B, t.k + 4), dtype=torch.float32, device="cuda")
        t.forward_partials(ops, db, part_small, pooled, None, None)
        if part_small is not None:
            msg = torch.empty((B, t.k + 4), dtype=torch.float32, device="cuda")
            t.rank_partial(B, part_small, msg)
        if ops & (OP_POOL | OP_DENSE1):
            # local pooled blocks (zero where another rank owns the keys) and, with DENSE1, this rank's
            # row-split partial Z_r = V_r W
            t.aggregate(ops & (OP_POOL | OP_DENSE1), db, None, pooled, None, None, None, pooled, Z)
        return msg

    # the exchange and what follows it
    def forward_finish(self, ops: int, B: int, msg: Optional[torch.Tensor], out_small: Optional[torch.Tensor],
                       pooled: Optional[torch.Tensor] = None, Z: Optional[torch.Tensor] = None,
                       reduce_pooled: bool = True):
        if msg is not None:
            allmsg = self.gather(msg, self.world)
            self.t.aggregate_ranks(ops, B, self.world, allmsg, out_small)
        pooled_all = None
        if (ops & OP_POOL) and reduce_pooled:
            pooled_all = self.reduce(pooled.clone())       # the local blocks stay: the backward's wgrad uses them
        if ops & OP_DENSE1:
            self.reduce(Z)
        return pooled_all

    def forward(self, ops, db, out_small=None, pooled=None, Z=None):
        msg = self.forward_local(ops, db, pooled, Z)
        return self.forward_finish(ops, db.batch, msg, out_small, pooled, Z)

    def backward_update(self, ops, db, out_small, pooled_local, Z, gL, gF, gE, gZ, gE_work):
        """No exchange: replicated gradients in, own keys updated."""
        self.t.backward_update(ops, db, out_small, pooled_local, Z, gL, gF, gE, gZ, gE_work)
