"""Pins of the oracle's strided pointwise convolution with a residual operand (the paper's Section
3.2.2 formula at k_h = k_w = 1 sampled at stride s, then bias, residual, activation): exact
rational arithmetic, reduction to the plain oracle, a float64 library witness, closed forms, and
planted mistakes that must be caught."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from alcs_workloads import rng


def _ints(seed, shape, lo=-4, hi=4):
    n = int(np.prod(shape))
    return ((rng.bits64(seed, 77, n) % np.uint64(hi - lo + 1)).astype(np.int64) + lo).reshape(shape)


def _case(seed, n, cin, cout, h, wd, g, stride, dtype=np.float32):
    rows = -(-cout // g)
    W = _ints(seed, (cout, cin)).astype(dtype)
    X = _ints(seed + 1, (n, cin, h, wd)).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < 0.5).astype(np.uint8).reshape(rows, cin)
    b = _ints(seed + 2, (cout,)).astype(np.float32)
    oh, ow = -(-h // stride), -(-wd // stride)
    R = _ints(seed + 3, (n, cout, oh * ow)).astype(dtype)
    return W, M, X, b, R


def _brute(W, M, X, b, R, relu, g, stride):
    n, cin, h, wd = X.shape
    cout = W.shape[0]
    oh, ow = -(-h // stride), -(-wd // stride)
    Y = np.zeros((n, cout, oh * ow), dtype=object)
    for i in range(n):
        for co in range(cout):
            for y in range(oh):
                for x in range(ow):
                    s = Fraction(0)
                    for c in range(cin):
                        if M[co // g, c]:
                            s += Fraction(float(W[co, c])) * Fraction(float(X[i, c, y * stride, x * stride]))
                    s += Fraction(float(b[co])) if b is not None else 0
                    s += Fraction(float(R[i, co, y * ow + x])) if R is not None else 0
                    if relu and s < 0:
                        s = Fraction(0)
                    Y[i, co, y * ow + x] = s
    return Y


@pytest.mark.parametrize("g,stride,h,wd", [(4, 1, 3, 5), (4, 2, 5, 4), (2, 2, 6, 6), (1, 3, 7, 5), (8, 2, 3, 3)])
@pytest.mark.parametrize("relu", [False, True])
def test_exact_rational_brute_force(g, stride, h, wd, relu, f=None):
    f = f or oracle.conv1x1_ex
    W, M, X, b, R = _case(10 * g + stride, 2, 6, 10, h, wd, g, stride)
    Y = f(W, M, X, b, R, relu, g, stride)
    ref = _brute(W, M, X, b, R, relu, g, stride)
    assert Y.shape == ref.shape
    assert all(Fraction(float(a)) == r for a, r in zip(Y.reshape(-1), ref.reshape(-1)))


def test_reduces_to_the_plain_oracle(f=None):
    """Stride 1 and no residual is oracle.conv1x1 bit for bit (values and scale); a zero residual too."""
    f = f or oracle.conv1x1_ex
    n, cin, cout, h, wd, g = 2, 9, 12, 4, 5, 4
    W = rng.normal(3, 1, cout * cin).reshape(cout, cin).astype(np.float32)
    X = rng.normal(3, 2, n * cin * h * wd).reshape(n, cin, h, wd).astype(np.float32)
    M = (rng.uniform01(3, 3, (cout // g) * cin) < 0.6).astype(np.uint8).reshape(cout // g, cin)
    b = rng.normal(3, 4, cout).astype(np.float32)
    Y0, A0 = oracle.conv1x1(W, M, X.reshape(n, cin, h * wd), b, True, g, want_scale=True)
    Y1, A1 = f(W, M, X, b, None, True, g, 1, want_scale=True)
    assert np.array_equal(Y0, Y1) and np.array_equal(A0, A1)
    Y2 = f(W, M, X, b, np.zeros((n, cout, h * wd), np.float32), True, g, 1)
    assert np.array_equal(Y0, Y2)


def test_library_witness_float64(f=None):
    """torch conv2d (float64, CPU) with a 1x1 kernel and stride, plus residual and relu."""
    import torch
    f = f or oracle.conv1x1_ex
    n, cin, cout, h, wd, g, s = 2, 8, 8, 7, 6, 4, 2
    W = rng.normal(5, 1, cout * cin).reshape(cout, cin).astype(np.float32)
    X = rng.normal(5, 2, n * cin * h * wd).reshape(n, cin, h, wd).astype(np.float32)
    M = (rng.uniform01(5, 3, (cout // g) * cin) < 0.5).astype(np.uint8).reshape(cout // g, cin)
    b = rng.normal(5, 4, cout).astype(np.float32)
    oh, ow = 4, 3
    R = rng.normal(5, 6, n * cout * oh * ow).reshape(n, cout, oh * ow).astype(np.float32)
    Wm = W.astype(np.float64) * np.repeat(M, g, axis=0)[:cout]
    t = torch.nn.functional.conv2d(torch.from_numpy(X.astype(np.float64)), torch.from_numpy(Wm)[:, :, None, None],
                                   torch.from_numpy(b.astype(np.float64)), stride=s)
    ref = torch.relu(t + torch.from_numpy(R.astype(np.float64)).reshape(n, cout, oh, ow)).numpy().reshape(n, cout, oh * ow)
    Y = f(W, M, X, b, R, True, g, s)
    assert np.abs(Y - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


def test_closed_forms(f=None):
    """Empty mask: y = relu(bias + residual) exactly; identity weights at stride 2: y = the sampled
    pixels plus the residual; the residual passes through the activation, not around it."""
    f = f or oracle.conv1x1_ex
    n, c, h, wd, g = 1, 4, 4, 4, 4
    X = np.arange(n * c * h * wd, dtype=np.float32).reshape(n, c, h, wd) - 20
    b = np.array([1, -2, 3, -4], np.float32)
    R = -np.ones((n, c, 4), np.float32) * 30
    Y = f(np.ones((c, c), np.float32), np.zeros((1, c), np.uint8), X, b, R, True, g, 2)
    assert np.array_equal(Y, np.maximum(b[None, :, None] + R, 0))
    Y = f(np.eye(c, dtype=np.float32), np.ones((1, c), np.uint8), X, None, None, False, g, 2)
    assert np.array_equal(Y.reshape(n, c, 2, 2), X[:, :, ::2, ::2])
    # positive convolution result, residual negative enough to flip the sum: the activation sees the sum
    Xp = np.ones((1, 4, 2, 2), np.float32)
    Rn = -np.full((1, 4, 4), 10.0, np.float32)
    Y = f(np.ones((4, 4), np.float32), np.ones((1, 4), np.uint8), Xp, None, Rn, True, 4, 1)
    assert np.array_equal(Y, np.zeros((1, 4, 4)))


def test_half_precision_residual_is_decoded_exactly():
    W, M, X, b, R = _case(42, 1, 4, 4, 4, 4, 4, 2, np.float16)
    Y16 = oracle.conv1x1_ex(W, M, X, b, R, False, 4, 2)
    Y32 = oracle.conv1x1_ex(W.astype(np.float32), M, X.astype(np.float32), b, R.astype(np.float32), False, 4, 2)
    assert np.array_equal(Y16, Y32)


def _pins_pass(mutant, build_dir):
    f = lambda *a, **k: oracle.conv1x1_ex(*a, mutant=mutant, build_dir=build_dir, **k)
    try:
        test_exact_rational_brute_force(4, 2, 5, 4, True, f=f)
        test_exact_rational_brute_force(2, 2, 6, 6, False, f=f)
        test_closed_forms(f=f)
        test_library_witness_float64(f=f)
    except AssertionError:
        return False
    return True


def test_pins_reject_planted_mistakes(tmp_path):
    assert _pins_pass(0, None)
    for mutant in (10, 11):       # residual added after the activation; sampling grid shifted by one pixel
        assert not _pins_pass(mutant, str(tmp_path)), f"mutant {mutant} slipped through"


def test_bfloat16_decoding_and_encoding():
    """Every bfloat16 bit pattern decodes to what an independent library says it is, and the workloads'
    encoder rounds float32 to the nearest bfloat16 with ties to even (the same library as witness)."""
    import torch
    bits = np.arange(65536, dtype=np.uint16)
    ours = oracle.bf16_decode(bits)
    theirs = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours.view(np.uint32), theirs.view(np.uint32))
    x = np.concatenate([rng.normal(9, 1, 200000).astype(np.float32) * 37.0,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, np.inf, -np.inf], np.float32)])
    enc = rng.to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(enc, ref)
    assert np.isnan(oracle.bf16_decode(rng.to_bf16_bits(np.array([np.nan], np.float32)))).all()
