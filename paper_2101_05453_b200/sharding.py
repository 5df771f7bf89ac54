"""Batch sharding for multi-GPU runs: rows (utterances) never interact, so ranks take disjoint row ranges,
keep a full copy of the weights and exchange nothing on the data path."""
from __future__ import annotations

from typing import Tuple


def shard_bounds(n_rows: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [begin, end) of batch rows for `rank`; sizes differ by at most one, earlier ranks get the extra."""
    assert 0 <= rank < world and n_rows >= 0
    base, extra = divmod(n_rows, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def state_slices(layers, n_rows: int, begin: int, end: int):
    """Index arrays selecting rows [begin, end) out of the flat per-layer h (int8) and c (int16) state vectors."""
    import numpy as np
    h_idx, c_idx, ho, co = [], [], 0, 0
    for q in layers:
        h_idx.append(ho + np.arange(begin * q.n_output, end * q.n_output))
        c_idx.append(co + np.arange(begin * q.n_cell, end * q.n_cell))
        ho += n_rows * q.n_output
        co += n_rows * q.n_cell
    return np.concatenate(h_idx), np.concatenate(c_idx)
