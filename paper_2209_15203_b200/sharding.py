"""Workers spread over GPUs, one process per GPU.

The only exchange of the iteration is the uplink: every worker sends its Top_K message to
the server (SEND / RECV of Algorithm 1/2).  With the workers' rows sharded over ranks and the
server replicated on every rank, that is one all-gather of the message buffer — N*K_up
entries of 8 bytes, a few MB at most — after which every rank sums in the same worker order
and so keeps bit-identical replicas of w (and of the server memory).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def row_range(N: int, rank: int, world: int) -> Tuple[int, int]:
    """(first row, number of rows) of `rank`: equal contiguous shares (N must divide evenly,
    which is what lets the all-gather run in place on the message buffer)."""
    if N % world != 0:
        raise ValueError("N = %d workers do not split evenly over %d ranks" % (N, world))
    rows = N // world
    return rank * rows, rows


def all_gather_messages(msgs: torch.Tensor, row0: int, rows: int, group=None) -> None:
    """msgs: [N][K_up] int64 message buffer whose rows row0..row0+rows-1 this rank has just
    produced; on return every rank holds all N rows."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return
    mine = msgs[row0:row0 + rows].reshape(-1).clone()
    dist.all_gather_into_tensor(msgs.view(-1), mine, group=group)


def sharded_step(ctx, w: torch.Tensor, grads_local: torch.Tensor, alpha: float, mode: int, group=None) -> None:
    """One iteration with this rank holding the gradients of its own workers only."""
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    row0, rows = row_range(ctx.N, rank, world)
    assert grads_local.numel() == rows * ctx.d
    ctx.tk_step_uplink(grads_local, row0, alpha, mode)
    all_gather_messages(ctx.tk_messages(), row0, rows, group)
    ctx.tk_step_server(w, alpha, mode)
