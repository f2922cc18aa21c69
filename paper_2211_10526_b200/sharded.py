"""Sequence-sharded forward: the token grid is cut into bands of rows, one per rank.

Per rank: sums over its own tokens (``CastlingAttn.shard_state``), ONE all-reduce of the ``B*H*(d*d+d)`` floats
of state over the ranks, the rows of V that the depthwise filters reach in the neighbouring bands (an exchange
of ``(ksize-1)/2`` grid rows with each neighbour), then the band's output rows (``CastlingAttn.shard_apply``).
The collective and the exchange go through ``torch.distributed`` (NCCL on GPUs); the arithmetic is the
library's.  The helpers that only move or index data work on CPU tensors too (gloo), which is how they are tested
without GPUs.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch


def band_rows(gridH: int, world: int, rank: int) -> Tuple[int, int]:
    """Rows [y0, y1) of the grid held by `rank`: bands as equal as possible, in rank order."""
    if not (0 <= rank < world) or gridH < world:
        raise ValueError("need 0 <= rank < world <= gridH")
    return gridH * rank // world, gridH * (rank + 1) // world


def halo_rows(gridH: int, y0: int, y1: int, ksize: int) -> Tuple[int, int]:
    """(rows needed from above, rows needed from below): the filter radius, or 0 at the edge of the grid."""
    r = (ksize - 1) // 2
    return (r if y0 > 0 else 0), (r if y1 < gridH else 0)


def exchange_halo(v_local: torch.Tensor, gridW: int, ksize: int, rank: int, world: int,
                  group=None) -> Tuple[torch.Tensor, int, int]:
    """v_local: [B, H, rows*gridW, d] of this rank's band (every band at least (ksize-1)/2 rows tall).  Sends its
    first / last (ksize-1)/2 rows to the ranks above / below and returns (v with the received rows attached,
    halo_top, halo_bottom)."""
    import torch.distributed as dist
    r = (ksize - 1) // 2
    B, H, n, d = v_local.shape
    rows = n // gridW
    if r == 0 or world == 1:
        return v_local, 0, 0
    if rows < r:
        raise ValueError("a band is shorter than the filter radius")
    up, down = rank - 1, rank + 1
    top = torch.empty(B, H, r * gridW, d, dtype=v_local.dtype, device=v_local.device) if up >= 0 else None
    bot = torch.empty(B, H, r * gridW, d, dtype=v_local.dtype, device=v_local.device) if down < world else None
    ops = []
    if up >= 0:
        ops.append(dist.P2POp(dist.isend, v_local[:, :, :r * gridW].contiguous(), up, group))
        ops.append(dist.P2POp(dist.irecv, top, up, group))
    if down < world:
        ops.append(dist.P2POp(dist.isend, v_local[:, :, n - r * gridW:].contiguous(), down, group))
        ops.append(dist.P2POp(dist.irecv, bot, down, group))
    for req in dist.batch_isend_irecv(ops):
        req.wait()
    parts = [t for t in (top, v_local, bot) if t is not None]
    return torch.cat(parts, dim=2).contiguous(), (r if top is not None else 0), (r if bot is not None else 0)


def forward_sharded(attn, q_local, k_local, v_local, dw_weight, dw_bias: Optional[torch.Tensor], gridW: int,
                    rank: int, world: int, group=None) -> torch.Tensor:
    """This rank's rows of the output.  q/k/v_local: [B, H, rows*gridW, d] of this rank's band on its GPU."""
    import torch.distributed as dist
    state = attn.shard_state(k_local, v_local)
    if world > 1:
        dist.all_reduce(state, op=dist.ReduceOp.SUM, group=group)
    v_halo, top, bottom = exchange_halo(v_local, gridW, attn.ksize, rank, world, group)
    rows = q_local.shape[2] // gridW
    return attn.shard_apply(q_local, v_halo, dw_weight, dw_bias, state, rows, gridW, top, bottom)
