"""Splitting independent decode units (tensors, layers, tile ranges) over ranks.

Tiles and tensors are independently decodable, so a multi-GPU job needs no data-path collective:
every rank decodes its own contiguous share and only timings / byte counts are reduced.
"""
from __future__ import annotations


def shard_range(n_units: int, world: int, rank: int) -> range:
    """Contiguous, balanced share of units [0, n_units) for `rank` of `world` (sizes differ by at most one)."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad world / rank")
    lo = n_units * rank // world
    hi = n_units * (rank + 1) // world
    return range(lo, hi)


def tile_range_rows(info, tiles: range) -> tuple[int, int]:
    """Rows of the output touched by a range of tiles: [first_row, last_row_exclusive)."""
    per_row = info.C // 8
    if len(tiles) == 0:
        return 0, 0
    v0 = tiles.start * info.V
    v1 = min(tiles.stop * info.V, info.R * per_row)
    return v0 // per_row, -(-v1 // per_row)
