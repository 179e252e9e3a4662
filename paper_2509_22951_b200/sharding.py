"""Row sharding of a compressed linear layer across ranks (one process per GPU).

A matrix is split by output rows: every rank holds the token segments of its own rows, the whole
table and the whole activation, and produces its slice of y.  The only exchange is an all-gather
of the output slices; no reduction is needed and no rank ever reads another rank's memory from
inside a kernel.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_range(rows: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [r0, r1) owned by `rank`; sizes differ by at most one row."""
    base, rem = divmod(rows, world)
    r0 = rank * base + min(rank, rem)
    return r0, r0 + base + (1 if rank < rem else 0)


def all_gather_rows(y_local: torch.Tensor, rows: int, rank: int, world: int) -> torch.Tensor:
    """y_local: [B][r1-r0] slice of this rank -> full [B][rows] on every rank."""
    B = y_local.shape[0]
    sizes = [row_range(rows, r, world)[1] - row_range(rows, r, world)[0] for r in range(world)]
    pad = max(sizes)
    send = torch.zeros((B, pad), dtype=y_local.dtype, device=y_local.device)
    send[:, : y_local.shape[1]] = y_local
    recv = [torch.empty_like(send) for _ in range(world)]
    dist.all_gather(recv, send)
    return torch.cat([recv[r][:, : sizes[r]] for r in range(world)], dim=1)
