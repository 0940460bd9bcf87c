"""Oracle for the grouped-CSR storage format of a SIMD-structured sparse weight matrix.
Test infrastructure only; shares no code with the library's packer.

Follows the paper's storage-format paragraph (Section 3.2.2, "Storage format of
SIMD-structured sparse tensor"): each group of g filters is stored as
  (i)   the number of non-zero columns of the group,
  (ii)  one column offset per non-zero column = how many columns of the original (flattened)
        kernel matrix come before it, i.e. its absolute 0-based column index,
  (iii) the non-zero values, one g-long column after another.
Which columns count as "non-zero" is decided by the pruning mask, not by testing values:
a kept block is stored even if its values happen to be zero.

Written as plain Python loops over small/medium matrices; values are moved, never computed,
so every comparison against this oracle is bit-exact.
"""
from __future__ import annotations

import numpy as np


def pack(W: np.ndarray, mask: np.ndarray, g: int):
    """Return (counts, offsets, values): per group r, counts[r] = number of kept columns,
    offsets[r] = their ascending absolute column indices, values[r] = array [counts[r], g]
    holding the group's g weights of each kept column (rows past cout read as +0)."""
    cout, cin = W.shape
    rows = (cout + g - 1) // g
    assert mask.shape == (rows, cin)
    counts, offsets, values = [], [], []
    for r in range(rows):
        offs = []
        vals = []
        for c in range(cin):
            if mask[r, c]:
                offs.append(c)                      # c columns precede column c
                col = np.zeros(g, dtype=W.dtype)
                for j in range(g):
                    co = r * g + j
                    if co < cout:
                        col[j] = W[co, c]
                vals.append(col)
        counts.append(len(offs))
        offsets.append(np.array(offs, dtype=np.int32))
        values.append(np.array(vals, dtype=W.dtype).reshape(len(offs), g))
    return counts, offsets, values


def flatten(counts, offsets, values, g: int, dtype):
    """The same content as three flat arrays: row_ptr[R+1] (prefix sums of the counts),
    col_idx[nb], vals[nb*g] (value j of kept block k at k*g + j)."""
    row_ptr = np.zeros(len(counts) + 1, dtype=np.int32)
    for r, c in enumerate(counts):
        row_ptr[r + 1] = row_ptr[r] + c
    col_idx = (np.concatenate(offsets) if len(offsets) else np.zeros(0)).astype(np.int32)
    vals = (np.concatenate([v.reshape(-1) for v in values]) if len(values)
            else np.zeros(0)).astype(dtype)
    return row_ptr, col_idx, vals


def unpack(counts, offsets, values, cout: int, cin: int, g: int, dtype):
    """Inverse of pack: dense W with dropped blocks as +0, and the block mask."""
    rows = (cout + g - 1) // g
    W = np.zeros((cout, cin), dtype=dtype)
    mask = np.zeros((rows, cin), dtype=np.uint8)
    for r in range(rows):
        for k in range(counts[r]):
            c = int(offsets[r][k])
            mask[r, c] = 1
            for j in range(g):
                co = r * g + j
                if co < cout:
                    W[co, c] = values[r][k, j]
    return W, mask
