"""Host logic of the launch schedule of the CUDA-core kernels: the library walks every (warp,
accumulator set)'s segments the way a consumer warp does and must find exactly the kept blocks of
the storage format (paper, Section 3.2.2), for uniform, skewed, empty and ragged matrices; and the
rows of a work item are spread evenly over the SM's four schedulers.  No GPU needed."""
import numpy as np
import pytest

import paper_2109_00170_b200 as A
from alcs_workloads import rng, zipf_block_mask


def _matrix(seed, cout, cin, g, density, dtype=np.float32):
    rows = (cout + g - 1) // g
    W = (rng.normal(seed, 1, cout * cin)).reshape(cout, cin).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    return W, M


@pytest.mark.parametrize("cout,cin,g,density", [(64, 48, 4, 0.3), (130, 200, 4, 0.1), (512, 512, 4, 0.25),
                                                (36, 70, 2, 0.5), (24, 33, 1, 0.4), (128, 96, 8, 0.25),
                                                (96, 64, 16, 0.5), (19, 7, 4, 1.0)])
@pytest.mark.parametrize("kc,n_rg,warps,slots", [(16, 1, 12, 2), (64, 3, 8, 3), (0, 2, 16, 1), (32, 7, 6, 2), (96, 1, 4, 4)])
def test_schedule_reproduces_the_storage_format(cout, cin, g, density, kc, n_rg, warps, slots):
    W, M = _matrix(cout + cin, cout, cin, g, density)
    p = A.alcs_pack(W, M, g)
    st = A.alcs_schedule_selfcheck(p, kc, n_rg, warps, slots)
    rows = (cout + g - 1) // g
    assert st["nb"] == int(M.sum())
    assert st["row_groups"] >= max(1, -(-rows // (warps * slots)))
    # padding: at most one block per (block row, chunk) segment
    nch = 1 if kc == 0 or kc >= cin else -(-cin // kc)
    assert 2 * st["pairs"] - st["nb"] <= rows * nch


def test_schedule_special_masks():
    g = 4
    W, M = _matrix(5, 64, 80, g, 0.3)
    for mask in (np.zeros_like(M), np.ones_like(M), zipf_block_mask(16, 80, 9)):
        p = A.alcs_pack(W, mask, g)
        A.alcs_schedule_selfcheck(p, 32, 1, 4, 4)
        A.alcs_schedule_selfcheck(p, 16, 2, 8, 1)
    Mh = M.copy()
    Mh[::2] = 0                      # every other block row empty
    A.alcs_schedule_selfcheck(A.alcs_pack(W, Mh, g), 16, 1, 8, 2)
    Wh, Mh16 = _matrix(6, 40, 50, 8, 0.4, np.float16)
    A.alcs_schedule_selfcheck(A.alcs_pack(Wh, Mh16, 8), 16, 1, 4, 2)


def test_schedule_balances_the_schedulers():
    """512 -> 512 with 128 block rows in 6 row groups on 12 warps x 2 slots: the row groups hold 20 or
    24 rows (multiples of 4), so each of the four schedulers gets the same number of rows, and its
    share of the kept blocks is within a few per cent of the others'."""
    W, M = _matrix(77, 512, 512, 4, 0.26)
    p = A.alcs_pack(W, M, 4)
    st = A.alcs_schedule_selfcheck(p, 64, 6, 12, 2)
    assert st["row_groups"] == 6
    assert (st["max_rows"], st["min_rows"]) == (6, 5)       # 24-row groups: 6 per scheduler, 20-row groups: 5
    per_rg = st["nb"] / 6 / 4
    assert st["max_sched"] <= 1.25 * per_rg      # (24-row groups carry 24/21.3 of the average)
    st1 = A.alcs_schedule_selfcheck(p, 64, 4, 16, 2)          # 32 rows per group: identical groups
    assert st1["max_sched"] <= 1.06 * st1["min_sched"]


def test_selfcheck_argument_errors():
    W, M = _matrix(1, 8, 8, 4, 0.5)
    p = A.alcs_pack(W, M, 4)
    for bad in ((16, 1, 0, 2), (16, 1, 40, 2), (16, 1, 4, 0), (16, 1, 4, 16)):
        with pytest.raises(A.AlcsError) as e:
            A.alcs_schedule_selfcheck(p, *bad)
        assert e.value.status == A.ALCS_ERR_INVALID_ARG


def test_long_rows_are_split_into_parts():
    """Zipf-distributed row lengths: with spare (warp, set) pairs the longest rows are split, every kept block
    still multiplied exactly once (the self-check walks all parts), and the most loaded scheduler carries far
    less than the longest row would alone."""
    W, _ = _matrix(3, 512, 512, 4, 0.5)
    M = zipf_block_mask(128, 512, 9)
    p = A.alcs_pack(W, M, 4)
    longest = int(M.sum(axis=1).max())
    st = A.alcs_schedule_selfcheck(p, 64, 8, 12, 2)
    assert st["secondary_units"] > 0
    assert st["max_sched"] < 1.3 * longest
    assert st["nb"] == int(M.sum())
    uniform = A.alcs_schedule_selfcheck(A.alcs_pack(*_matrix(4, 512, 512, 4, 0.25), 4), 64, 6, 12, 2)
    assert uniform["secondary_units"] == 0


def test_bfloat16_weights_pack_and_schedule():
    """bfloat16 weights travel as bit patterns: pack -> unpack and the serialised blob return them bit for
    bit, and the schedule (which widens them to fp32 exactly) passes the walk check."""
    g = 8
    W = rng.to_bf16_bits(rng.normal(8, 1, 64 * 48).astype(np.float32)).reshape(64, 48)
    M = (rng.uniform01(8, 3, 8 * 48) < 0.4).astype(np.uint8).reshape(8, 48)
    p = A.alcs_pack(W, M, g, bf16=True)
    W2, M2 = A.alcs_unpack(p)
    assert W2.dtype == np.uint16 and np.array_equal(M2, M)
    assert np.array_equal(W2, W * np.repeat(M, g, axis=0).astype(np.uint16))
    q = A.alcs_packed_deserialize(A.alcs_packed_serialize(p))
    assert np.array_equal(A.alcs_unpack(q)[0], W2)
    A.alcs_schedule_selfcheck(p, 16, 1, 4, 2)
    with pytest.raises(TypeError):
        A.alcs_pack(W.astype(np.float64), M, g)
