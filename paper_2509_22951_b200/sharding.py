"""Row sharding of compressed linear layers across ranks (one process per GPU).

A matrix is split by output rows: every rank holds the tokens of its own rows, the whole table and
the whole activation, and produces its slice of y.  The only exchange is an all-gather of the
output slices; no reduction is needed and no rank ever reads another rank's memory from inside a
kernel.  Shards are cut at multiples of 16 rows, the height of a token tile, so a shard's tiles are
the tiles those rows have in the unsharded image.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_range(rows: int, rank: int, world: int, align: int = 16) -> tuple[int, int]:
    """Contiguous [r0, r1) owned by `rank`: whole blocks of `align` rows, block counts differing by at
    most one between ranks (the last block of the matrix may be short; a rank may own nothing when
    there are fewer blocks than ranks)."""
    blocks = -(-rows // align)
    b0, b1 = blocks * rank // world, blocks * (rank + 1) // world
    return min(rows, b0 * align), min(rows, b1 * align)


def all_gather_rows(y_local: torch.Tensor, rows: int, rank: int, world: int, align: int = 16) -> torch.Tensor:
    """y_local: [B][r1-r0] slice of this rank -> full [B][rows] on every rank."""
    B = y_local.shape[0]
    sizes = [row_range(rows, r, world, align)[1] - row_range(rows, r, world, align)[0] for r in range(world)]
    pad = max(sizes)
    send = torch.zeros((B, pad), dtype=y_local.dtype, device=y_local.device)
    send[:, : y_local.shape[1]] = y_local
    recv = [torch.empty_like(send) for _ in range(world)]
    dist.all_gather(recv, send)
    return torch.cat([recv[r][:, : sizes[r]] for r in range(world)], dim=1)


class ShardedOutputs:
    """Where every rank's output slices lie in one flat arena per rank, so that a whole stack of
    matrices needs ONE all-gather per step: rank r's arena holds, matrix after matrix, its
    [B][rows_r] slice (offsets rounded up to 4 floats); all arenas are padded to the longest."""

    def __init__(self, shapes, batch: int, world: int, align: int = 16):
        self.shapes, self.batch, self.world = list(shapes), batch, world
        self.ranges = [[row_range(rows, r, world, align) for (_, rows, _) in self.shapes] for r in range(world)]
        self.offsets, lengths = [], []
        for r in range(world):
            off, o = [], 0
            for (r0, r1) in self.ranges[r]:
                off.append(o)
                o += -(-batch * (r1 - r0) // 4) * 4
            self.offsets.append(off)
            lengths.append(o)
        self.arena_len = max(max(lengths), 4)

    def local_views(self, arena: torch.Tensor, rank: int):
        """The [B][rows_r] output tensors of `rank` inside its arena (what the kernels write)."""
        out = []
        for i, (r0, r1) in enumerate(self.ranges[rank]):
            o = self.offsets[rank][i]
            out.append(arena[o: o + self.batch * (r1 - r0)].view(self.batch, r1 - r0))
        return out

    def all_gather(self, arena: torch.Tensor, gathered: torch.Tensor | None = None) -> torch.Tensor:
        """One collective: every rank's arena, rank after rank, on every rank ([world * arena_len])."""
        if gathered is None:
            gathered = torch.empty(self.world * self.arena_len, dtype=arena.dtype, device=arena.device)
        dist.all_gather_into_tensor(gathered, arena)
        return gathered

    def full_output(self, gathered: torch.Tensor, i: int) -> torch.Tensor:
        """Matrix i's full [B][rows] output assembled from the gathered arenas."""
        parts = []
        for r in range(self.world):
            r0, r1 = self.ranges[r][i]
            o = r * self.arena_len + self.offsets[r][i]
            parts.append(gathered[o: o + self.batch * (r1 - r0)].view(self.batch, r1 - r0))
        return torch.cat(parts, dim=1)


def upload_row_shards(tq, ddict, levels, scales, rank: int, world: int, zeros=None, levels_signed: bool = True):
    """This rank's shard of every matrix: levels[i] CUDA int8/uint8 [rows][cols], scales[i] CUDA fp32 [rows].
    A rank that owns no row of a matrix gets None for it."""
    mats = []
    for i, (q, s) in enumerate(zip(levels, scales)):
        r0, r1 = row_range(q.shape[0], rank, world)
        z = None if zeros is None else zeros[i]
        mats.append(tq.tq_upload_device_rows(ddict, q, r0, r1, s, z, levels_signed) if r1 > r0 else None)
    return mats
