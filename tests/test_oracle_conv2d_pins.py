"""Pins of the general (k x k) convolution oracle against things other than itself.

The paper's Section 3.2.2 formula  O(n,h,w) = sum_c sum_r sum_s W(n,c,r,s) I(c,h+r,w+s)  fixes the
stride-1, unpadded case; stride and zero padding are the usual extension and must reduce to it.
Pins: exact rational arithmetic on tiny shapes, an independent library routine (torch float64
conv2d), the reduction to the (separately pinned) pointwise oracle at kh = kw = 1, a closed form
(a single unit weight at tap (r, s) shifts the image by (r, s)), the flattened-filter view of the
same section (W* times the stacked input patches), and the 0 % / 100 % sparsity cases.  The last test
plants mistakes in the oracle (flipped kernel, transposed taps, strided taps, wrong padding sign)
and checks that the pins reject each.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle
from alcs_workloads import rng

pytestmark = pytest.mark.filterwarnings("ignore")


def _ints(seed, shape, lo=-6, hi=6):
    n = int(np.prod(shape))
    b = rng.bits64(seed, 78, n)
    return ((b % np.uint64(hi - lo + 1)).astype(np.int64) + lo).reshape(shape)


def _case(seed, n, cin, cout, h, w, kh, kw, g, density=0.5, ints=False, dtype=np.float32):
    rows = (cout + g - 1) // g
    if ints:
        W = _ints(seed, (cout, cin, kh, kw)).astype(dtype)
        X = _ints(seed + 1, (n, cin, h, w)).astype(dtype)
        b = _ints(seed + 2, (cout,)).astype(np.float32)
    else:
        W = rng.normal(seed, 1, cout * cin * kh * kw).reshape(cout, cin, kh, kw).astype(dtype)
        X = rng.normal(seed, 2, n * cin * h * w).reshape(n, cin, h, w).astype(dtype)
        b = rng.normal(seed, 4, cout).astype(np.float32)
    M = (rng.uniform01(seed, 3, rows * cin * kh * kw) < density).astype(np.uint8).reshape(rows, cin * kh * kw)
    return W, M, X, b


def _masked(W, M, g):
    """W with dropped blocks set to zero, as float64 [cout,cin,kh,kw]."""
    cout = W.shape[0]
    full = np.repeat(M, g, axis=0)[:cout].reshape(W.shape)
    return W.astype(np.float64) * full


def _exact(W, M, X, b, relu, g, stride, pad):
    """The definition in exact rational arithmetic, loops in the order (ow, oh, co, n | s, r, c)."""
    cout, cin, kh, kw = W.shape
    n, _, h, w = X.shape
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (w + 2 * pad - kw) // stride + 1
    out = np.empty((n, cout, oh, ow), dtype=object)
    for x, y, co, i in itertools.product(range(ow), range(oh), range(cout), range(n)):
        acc = Fraction(0)
        for s, r, c in itertools.product(range(kw), range(kh), range(cin)):
            if not M[co // g, (c * kh + r) * kw + s]:
                continue
            ih, iw = y * stride - pad + r, x * stride - pad + s
            if 0 <= ih < h and 0 <= iw < w:
                acc += Fraction(float(W[co, c, r, s])) * Fraction(float(X[i, c, ih, iw]))
        if b is not None:
            acc += Fraction(float(b[co]))
        if relu and acc < 0:
            acc = Fraction(0)
        out[i, co, y, x] = acc
    return out


@pytest.mark.parametrize("kh,kw,stride,pad", [(3, 3, 1, 0), (3, 3, 1, 1), (3, 3, 2, 1), (2, 3, 1, 0),
                                               (5, 5, 2, 2), (1, 1, 1, 0), (3, 1, 2, 0)])
def test_integer_data_is_exact(kh, kw, stride, pad):
    """Small-integer data: every partial sum is representable, so the oracle must equal exact
    arithmetic bit for bit (ragged last block row included: cout = 6, g = 4)."""
    W, M, X, b = _case(100 + kh * 10 + kw + stride, 2, 3, 6, 6, 7, kh, kw, 4, ints=True)
    Y = oracle.conv2d(W, M, X, b, True, 4, stride, pad)
    E = _exact(W, M, X, b, True, 4, stride, pad)
    assert Y.shape == E.shape
    assert all(Fraction(float(Y[i])) == E[i] for i in np.ndindex(Y.shape))


@pytest.mark.parametrize("g", [1, 2, 4])
def test_bruteforce_rational_tiny(g):
    """Random real data, 3x3 pad 1: within a few ulps (of the scale A) of the exact rational value."""
    W, M, X, b = _case(7 + g, 1, 2, 4, 4, 5, 3, 3, g)
    Y, A = oracle.conv2d(W, M, X, b, False, g, 1, 1, want_scale=True)
    E = _exact(W, M, X, b, False, g, 1, 1)
    for idx in np.ndindex(Y.shape):
        assert abs(Fraction(float(Y[idx])) - E[idx]) <= Fraction(float(A[idx])) * 32 * Fraction(2) ** -53


@pytest.mark.parametrize("kh,kw,stride,pad", [(3, 3, 1, 1), (3, 3, 2, 1), (5, 3, 1, 2), (7, 7, 2, 3)])
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_against_torch_conv2d_float64(kh, kw, stride, pad, dtype):
    """Independent witness: torch's float64 conv2d (cross-correlation, zero padding) on the
    mask-applied weights."""
    torch = pytest.importorskip("torch")
    g = 4
    W, M, X, b = _case(300 + kh, 2, 5, 10, 13, 11, kh, kw, g, dtype=dtype)
    Y, A = oracle.conv2d(W, M, X, b, True, g, stride, pad, want_scale=True)
    ref = torch.nn.functional.conv2d(torch.from_numpy(X.astype(np.float64)), torch.from_numpy(_masked(W, M, g)),
                                     torch.from_numpy(b.astype(np.float64)), stride=stride, padding=pad).relu().numpy()
    assert Y.shape == ref.shape
    assert np.all(np.abs(Y - ref) <= 256 * 2.0 ** -53 * A + 1e-300)


def test_1x1_reduces_to_pointwise_oracle():
    """kh = kw = 1, stride 1, no padding: identical to the pointwise oracle (same summation order)."""
    W, M, X, b = _case(41, 2, 12, 8, 5, 6, 1, 1, 4)
    Y2, A2 = oracle.conv2d(W, M, X, b, True, 4, 1, 0, want_scale=True)
    Y1, A1 = oracle.conv1x1(W.reshape(8, 12), M, X.reshape(2, 12, 30), b, True, 4, want_scale=True)
    assert np.array_equal(Y2.reshape(Y1.shape), Y1) and np.array_equal(A2.reshape(A1.shape), A1)


@pytest.mark.parametrize("r,s", [(0, 0), (0, 2), (2, 0), (1, 2), (2, 1)])
def test_unit_tap_shifts_the_image(r, s):
    """One kept block whose only non-zero weight is W(co, c, r, s) = 1, stride 1, no padding:
    O(co, h, w) = I(c, h + r, w + s), the paper's index convention, exactly."""
    cin, cout, h, w = 3, 4, 6, 7
    W = np.zeros((cout, cin, 3, 3), np.float32)
    W[2, 1, r, s] = 1.0
    M = np.zeros((1, cin * 9), np.uint8)
    M[0, (1 * 3 + r) * 3 + s] = 1
    X = rng.normal(55, 2, cin * h * w).reshape(1, cin, h, w).astype(np.float32)
    Y = oracle.conv2d(W, M, X, None, False, 4, 1, 0)
    exp = np.zeros((1, cout, h - 2, w - 2))
    exp[0, 2] = X[0, 1, r:r + h - 2, s:s + w - 2]
    assert np.array_equal(Y, exp)


def test_flattened_filter_matrix_view():
    """Section 3.2.2: the convolution is W* (filters flattened to rows, column = (c, r, s)) times
    I* (the stacked, vectorised input patches).  Build I* explicitly (stride 2, pad 1) and
    multiply; exact on integer data."""
    kh = kw = 3
    stride, pad, g = 2, 1, 2
    W, M, X, _ = _case(61, 2, 3, 4, 7, 6, kh, kw, g, ints=True)
    n, cin, h, w = X.shape
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (w + 2 * pad - kw) // stride + 1
    Xp = np.zeros((n, cin, h + 2 * pad, w + 2 * pad))
    Xp[:, :, pad:pad + h, pad:pad + w] = X
    cols = np.empty((n, cin * kh * kw, oh * ow))
    for c, r, s in itertools.product(range(cin), range(kh), range(kw)):
        cols[:, (c * kh + r) * kw + s, :] = Xp[:, c, r:r + stride * oh:stride, s:s + stride * ow:stride].reshape(n, -1)
    Wstar = _masked(W, M, g).reshape(W.shape[0], -1)
    exp = np.einsum("ok,nkp->nop", Wstar, cols).reshape(n, W.shape[0], oh, ow)
    assert np.array_equal(oracle.conv2d(W, M, X, None, False, g, stride, pad), exp)


def test_sparsity_extremes():
    W, M, X, b = _case(71, 2, 4, 8, 6, 6, 3, 3, 4)
    Y0 = oracle.conv2d(W, np.zeros_like(M), X, b, True, 4, 1, 1)
    assert np.array_equal(Y0, np.broadcast_to(np.maximum(b.astype(np.float64), 0)[None, :, None, None], Y0.shape))
    # all kept: mask plays no role, so any g gives the same (dense) result
    Ya = oracle.conv2d(W, np.ones((2, 36), np.uint8), X, b, False, 4, 1, 1)
    Yb = oracle.conv2d(W, np.ones((8, 36), np.uint8), X, b, False, 1, 1, 1)
    assert np.array_equal(Ya, Yb)


def test_points_agree_with_full():
    W, M, X, b = _case(81, 2, 5, 8, 9, 8, 3, 3, 4)
    Y, A = oracle.conv2d(W, M, X, b, True, 4, 2, 1, want_scale=True)
    idx = rng.permutation(82, 1, Y.size)[:60]
    v, m = oracle.conv2d_points(W, M, X, idx, b, True, 4, 2, 1)
    assert np.array_equal(v, Y.reshape(-1)[idx]) and np.array_equal(m, A.reshape(-1)[idx])


def _pins_pass(mutant, build_dir):
    ok = True
    for kh, kw, stride, pad in [(3, 3, 1, 1), (3, 2, 2, 1)]:
        W, M, X, b = _case(100 + kh * 10 + kw + stride, 2, 3, 6, 6, 7, kh, kw, 4, ints=True)
        Y = oracle.conv2d(W, M, X, b, True, 4, stride, pad, mutant=mutant, build_dir=build_dir)
        E = _exact(W, M, X, b, True, 4, stride, pad)
        ok &= Y.shape == E.shape and all(Fraction(float(Y[i])) == E[i] for i in np.ndindex(E.shape))
    return ok


def test_pins_reject_planted_mistakes(tmp_path):
    assert _pins_pass(0, None)
    for mutant in (6, 7, 8, 9):
        assert not _pins_pass(mutant, str(tmp_path)), f"mutant {mutant} slipped through"
