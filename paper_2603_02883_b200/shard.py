"""Row sharding of one activation tensor over several GPUs (one process per GPU).

Blocks, salient-token tiles and SeDA clusters are all local to a token, so the quantizer
shards by contiguous token ranges with no data-path collective: every rank quantizes its rows
with its own context (the lookup tables and the cluster-mask table are replicated) and keeps its
part of the outputs.  The only constraint is that a salient-token tile must not straddle two
ranks, so shard boundaries are multiples of the tile size.
"""
from __future__ import annotations


def row_shard(T: int, world: int, rank: int, align: int = 1) -> tuple[int, int]:
    """Rows [r0, r1) of rank `rank`: the T rows are cut into `world` contiguous ranges whose
    boundaries are multiples of `align` (the last range takes the ragged end).  Ranges differ by
    less than 2 * `align` rows; a rank may get an empty range when T is small."""
    if T < 0 or world <= 0 or not 0 <= rank < world or align <= 0:
        raise ValueError("bad shard arguments")
    units = -(-T // align)
    base, extra = divmod(units, world)
    u0 = rank * base + min(rank, extra)
    u1 = u0 + base + (1 if rank < extra else 0)
    return min(u0 * align, T), min(u1 * align, T)


def local_salient_to_global(salient_idx, r0: int):
    """Salient-token indices returned for a shard are relative to its first row."""
    return salient_idx + r0
