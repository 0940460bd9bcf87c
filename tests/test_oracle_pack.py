"""Pins of the storage-format oracle: the paper's printed example, structural invariants,
round trips, and a mutation check."""
import os

import numpy as np
import pytest

from alcs_workloads import rng
from oracle import storage as opack

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "storage_format_example.txt")


def _read_golden():
    d = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(None, 1)
        d[k] = v
    g = int(d["g"])
    count = int(d["count"])
    offsets = [None if t == "?" else int(t) for t in d["offsets"].split()]
    values = [[None if t == "?" else float(t) for t in col.split()] for col in d["values"].split("|")]
    return g, count, offsets, values


def test_paper_storage_example():
    """Section 3.2.2 storage-format paragraph: a g=2 group with 3 non-zero columns, the first
    [1,3]^T at offset 1, the second [2,1]^T at offset 3.  Any matrix consistent with that prose
    must pack to count 3, offsets (1, 3, x) and values (1,3), (2,1), (., .): offsets are absolute
    0-based column indices and values are stored column by column."""
    g, count, offsets, values = _read_golden()
    cin = 6
    W = np.zeros((2, cin), np.float32)
    W[:, 1] = [1, 3]
    W[:, 3] = [2, 1]
    W[:, 5] = [4, 2]          # the third column is only in the (missing) figure: our choice
    M = (np.abs(W).sum(0) > 0).astype(np.uint8).reshape(1, cin)
    counts, offs, vals = opack.pack(W, M, g)
    assert counts == [count]
    for k, o in enumerate(offsets):
        if o is not None:
            assert offs[0][k] == o
    for k, col in enumerate(values):
        for j, v in enumerate(col):
            if v is not None:
                assert vals[0][k, j] == v
    assert offs[0][2] > 3


def _case(seed, cout, cin, g, density=0.4, dtype=np.float32):
    rows = (cout + g - 1) // g
    W = rng.normal(seed, 1, cout * cin).reshape(cout, cin).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    return W, M


@pytest.mark.parametrize("cout,cin,g", [(8, 7, 4), (10, 9, 4), (7, 5, 1), (16, 16, 16), (9, 4, 2), (5, 3, 8)])
def test_roundtrip_and_invariants(cout, cin, g):
    W, M = _case(cout * 100 + g, cout, cin, g)
    counts, offs, vals = opack.pack(W, M, g)
    # count per group = kept blocks of that group; offsets strictly ascending and in range
    assert counts == [int(x) for x in M.sum(1)]
    for r, o in enumerate(offs):
        assert np.all(np.diff(o) > 0) and np.all((o >= 0) & (o < cin))
        assert np.array_equal(o, np.nonzero(M[r])[0])
    W2, M2 = opack.unpack(counts, offs, vals, cout, cin, g, W.dtype)
    Wm = W * np.repeat(M, g, 0)[:cout].astype(W.dtype)
    assert np.array_equal(M2, M)
    assert np.array_equal(W2, Wm)
    kept = np.repeat(M, g, 0)[:cout].astype(bool)
    bits = np.uint32 if W.dtype == np.float32 else np.uint16
    assert np.array_equal(W2.view(bits)[kept], W.view(bits)[kept])     # kept values bit-exact
    assert not np.any(W2.view(bits)[~kept])                            # dropped blocks are +0
    row_ptr, col_idx, v = opack.flatten(counts, offs, vals, g, W.dtype)
    assert row_ptr[-1] == M.sum() == col_idx.size and v.size == col_idx.size * g


def test_values_are_moved_bit_exactly():
    """-0, subnormals, NaN payloads and infinities survive; dropped blocks vanish even if non-zero;
    kept blocks are stored even if zero."""
    g = 2
    W = np.array([[-0.0, 1e-45, np.inf, 5.0], [np.nan, 0.0, -np.inf, 6.0]], np.float32)
    M = np.array([[1, 1, 1, 0]], np.uint8)
    counts, offs, vals = opack.pack(W, M, g)
    assert counts == [3] and list(offs[0]) == [0, 1, 2]
    assert np.array_equal(vals[0].view(np.uint32), W[:, :3].T.copy().view(np.uint32))
    W2, M2 = opack.unpack(counts, offs, vals, 2, 4, g, np.float32)
    assert np.array_equal(W2[:, :3].view(np.uint32), W[:, :3].view(np.uint32))
    assert np.array_equal(W2[:, 3], [0, 0]) and np.array_equal(M2, M)


def test_group_uses_adjacent_channels_and_column_major_values():
    """Values of kept block k of group r are W[r*g + j, col] for j = 0..g-1, contiguous."""
    g = 4
    W = np.arange(8 * 3, dtype=np.float32).reshape(8, 3)
    M = np.array([[0, 1, 0], [1, 0, 1]], np.uint8)
    counts, offs, vals = opack.pack(W, M, g)
    assert np.array_equal(vals[0], [[1, 4, 7, 10]])
    assert np.array_equal(vals[1], [[12, 15, 18, 21], [14, 17, 20, 23]])


def test_ragged_last_group_is_zero_padded():
    W = np.ones((5, 2), np.float32)
    M = np.ones((2, 2), np.uint8)
    _, _, vals = opack.pack(W, M, 4)
    assert np.array_equal(vals[1], [[1, 0, 0, 0], [1, 0, 0, 0]])


def test_flatten_on_the_paper_example():
    """The paper's worked example (Section 3.2.2, storage-format paragraph) through flatten(): one
    group of g = 2 filters with 3 non-zero columns gives row_ptr [0, 3]; the column indices begin
    1, 3; the flat value array begins 1, 3, 2, 1 (the g values of a column are contiguous, columns in
    order).  The third column is only in the missing figure: any column after 3, any values."""
    g, count, offsets, values = _read_golden()
    known = [o for o in offsets if o is not None]
    W = np.zeros((2, 6), np.float32)
    M = np.zeros((1, 6), np.uint8)
    cols = known + [5]
    vals = [pair for pair in values if None not in pair] + [[7.0, 9.0]]
    for c, v in zip(cols, vals):
        W[:, c] = v
        M[0, c] = 1
    row_ptr, col_idx, flat = opack.flatten(*opack.pack(W, M, g), g, np.float32)
    assert list(row_ptr) == [0, count] == [0, 3]
    assert list(col_idx[:2]) == [1, 3]
    assert list(flat[:4]) == [1.0, 3.0, 2.0, 1.0]
    assert row_ptr.dtype == np.int32 and col_idx.dtype == np.int32 and flat.dtype == np.float32
    # two groups: the second group's entries follow the first's, offsets restart from the column index
    W2 = np.vstack([W, 10 * W])
    M2 = np.vstack([M, M])
    row_ptr, col_idx, flat = opack.flatten(*opack.pack(W2, M2, g), g, np.float32)
    assert list(row_ptr) == [0, 3, 6] and list(col_idx) == [1, 3, 5, 1, 3, 5]
    assert list(flat[6:10]) == [10.0, 30.0, 20.0, 10.0]
