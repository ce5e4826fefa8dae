"""Seeded choice of the token rows that the full-size GPU tests compare with the oracle one by one."""

from __future__ import annotations

import numpy as np


def sample_rows(seq_offsets, T: int, n: int, rng: np.random.Generator) -> np.ndarray:
    """Tile edges (first and last row, both sides of the last 128-row boundary), then the same number of rows from
    every sequence -- at least eight where n allows it -- then random rows up to n.  Sorted, unique."""
    offs = np.asarray(seq_offsets, dtype=np.int64)
    S = len(offs) - 1
    rows = {0, T - 1, max(0, T - 2), (T // 128) * 128 - 1 if T >= 128 else 0, min(T - 1, (T // 128) * 128)}
    per = max(1, (n - len(rows)) // S)
    for s in range(S):
        lo, hi = offs[s], offs[s + 1]
        if hi > lo:
            rows.update(int(x) for x in rng.choice(np.arange(lo, hi), size=min(per, hi - lo), replace=False))
    while len(rows) < n:
        rows.add(int(rng.integers(0, T)))
    return np.array(sorted(rows))


def rows_per_sequence(rows, seq_offsets) -> np.ndarray:
    return np.histogram(rows, bins=np.asarray(seq_offsets, dtype=np.int64))[0]
