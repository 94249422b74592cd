"""TEST INFRASTRUCTURE — plain restatement of the paper's attention Token-Table,
decomposition and Task-Table (Sections 3.2.1 and 3.3.1), in slow pure Python.

Token-Table: one entry per stage with stageID, start position, tokenNum,
historical kvLen and tileSize.  Decomposition: a stage gives
ceil(tokenNum / tileSize) tile blocks, each block gives headNum tile units.
Reordering: load of a tile = tileSize x kvLen; sort from largest to smallest;
deal the tiles to the cores in a symmetric round-robin 1..C, C..1, 1..C, ...

Readings where the paper leaves a choice (all stated in the design notes):
  * "kvLen" of a tile is the number of keys the tile can see, i.e. the stage's
    historical kvLen plus the new tokens up to the tile's last row, because a
    causal tile never visits later keys (Section 4.2.2);
  * "tileSize" in the load is the tile's actual row count (the last block of a
    stage may be short);
  * ties keep the order (stage, head, block): the sort is stable;
  * the round-robin starts at core 0 going up.
"""
from __future__ import annotations

from typing import List, NamedTuple


class TokenEntry(NamedTuple):
    stage_id: int
    start: int  # start position = prefix sum of tokenNum
    token_num: int
    kv_len: int  # historical
    tile_size: int


class TileUnit(NamedTuple):
    stage_id: int
    head: int
    block: int
    row0: int  # first row of the block inside the stage
    rows: int
    visible: int  # keys the tile can see
    load: int


def token_table(q_len, kv_len, tile_size) -> List[TokenEntry]:
    out, start = [], 0
    for s, (n, h) in enumerate(zip(q_len, kv_len)):
        ts = tile_size[s] if hasattr(tile_size, "__len__") else tile_size
        out.append(TokenEntry(s, start, int(n), int(h), int(ts)))
        start += int(n)
    return out


def decompose(table: List[TokenEntry], head_num: int) -> List[TileUnit]:
    units = []
    for e in table:
        blocks = -(-e.token_num // e.tile_size)
        for head in range(head_num):
            for b in range(blocks):
                row0 = b * e.tile_size
                rows = min(e.tile_size, e.token_num - row0)
                visible = e.kv_len + row0 + rows
                units.append(TileUnit(e.stage_id, head, b, row0, rows, visible, rows * visible))
    return units


def reorder(units: List[TileUnit], num_cores: int) -> List[List[TileUnit]]:
    order = sorted(range(len(units)), key=lambda k: -units[k].load)  # stable
    cores: List[List[TileUnit]] = [[] for _ in range(num_cores)]
    for pos, k in enumerate(order):
        lap, idx = divmod(pos, num_cores)
        core = idx if lap % 2 == 0 else num_cores - 1 - idx
        cores[core].append(units[k])
    return cores


def core_sequence(num_units: int, num_cores: int) -> List[int]:
    """Core id that receives the k-th tile of the sorted list."""
    seq = []
    for pos in range(num_units):
        lap, idx = divmod(pos, num_cores)
        seq.append(idx if lap % 2 == 0 else num_cores - 1 - idx)
    return seq
