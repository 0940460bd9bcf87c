"""Pins of the convolution oracle against things other than itself.

Each test fixes the oracle to something the paper or the mathematics determines:
exact rational arithmetic on tiny inputs, an independent library routine, closed forms,
the 0 % and 100 % sparsity special cases, and algebraic invariants.  A final test compiles
deliberately wrong variants of the oracle and checks that these pins reject each of them.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle
from alcs_workloads import rng

pytestmark = pytest.mark.filterwarnings("ignore")


def _ints(seed, shape, lo=-8, hi=8):
    n = int(np.prod(shape))
    b = rng.bits64(seed, 77, n)
    return ((b % np.uint64(hi - lo + 1)).astype(np.int64) + lo).reshape(shape)


def _rand_case(seed, n, cin, cout, hw, g, density=0.5, dtype=np.float32):
    rows = (cout + g - 1) // g
    W = rng.normal(seed, 1, cout * cin).reshape(cout, cin).astype(dtype)
    X = rng.normal(seed, 2, n * cin * hw).reshape(n, cin, hw).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = rng.normal(seed, 4, cout).astype(np.float32)
    return W, M, X, b


def _exact(W, M, X, b, relu, g):
    """The definition in exact rational arithmetic, loop order (p, n, co, ci)."""
    cout, cin = W.shape
    n, _, hw = X.shape
    out = np.empty((n, cout, hw), dtype=object)
    for p, i, co in itertools.product(range(hw), range(n), range(cout)):
        s = Fraction(0)
        for ci in range(cin):
            if M[co // g, ci]:
                s += Fraction(float(W[co, ci])) * Fraction(float(X[i, ci, p]))
        if b is not None:
            s += Fraction(float(b[co]))
        if relu and s < 0:
            s = Fraction(0)
        out[i, co, p] = s
    return out


@pytest.mark.parametrize("g", [1, 2, 4, 8])
@pytest.mark.parametrize("relu", [False, True])
def test_bruteforce_rational_tiny(g, relu):
    """N=2, Cin=5, Cout=8, HW=3: the double-precision oracle is within n*2^-53*A of the exact
    rational value of the definition (Section 3.2.2 formula at kh=kw=1)."""
    W, M, X, b = _rand_case(10 + g, 2, 5, 8, 3, g)
    Y, A = oracle.conv1x1(W, M, X, b, relu, g, want_scale=True)
    E = _exact(W, M, X, b, relu, g)
    for idx in np.ndindex(Y.shape):
        assert abs(Fraction(float(Y[idx])) - E[idx]) <= Fraction(float(A[idx])) * 8 * Fraction(2) ** -53


@pytest.mark.parametrize("g,cout", [(4, 8), (4, 10), (3, 7), (16, 16)])
def test_integer_data_is_exact(g, cout):
    """Small-integer W, X, bias: every partial sum is exactly representable, so the oracle
    must equal exact arithmetic bit for bit, ragged last block row included."""
    rows = (cout + g - 1) // g
    W = _ints(1, (cout, 6)).astype(np.float32)
    X = _ints(2, (2, 6, 5)).astype(np.float32)
    b = _ints(3, (cout,)).astype(np.float32)
    M = (rng.uniform01(4, 3, rows * 6) < 0.6).astype(np.uint8).reshape(rows, 6)
    Y = oracle.conv1x1(W, M, X, b, True, g)
    E = _exact(W, M, X, b, True, g)
    assert all(Fraction(float(Y[i])) == E[i] for i in np.ndindex(Y.shape))


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_against_torch_conv2d_float64(dtype):
    """Independent witness: a 1x1 convolution is a matrix product (paper, Section 4.2: matrix
    multiplication is equivalent to a convolution layer with 1x1 kernels); torch's float64
    conv2d on the mask-applied weights must agree to rounding."""
    torch = pytest.importorskip("torch")
    g = 4
    W, M, X, b = _rand_case(21, 3, 24, 20, 35, g, dtype=dtype)
    Y, A = oracle.conv1x1(W, M, X, b, True, g, want_scale=True)
    Wm = torch.from_numpy(W.astype(np.float64) * np.repeat(M, g, 0)[:20].astype(np.float64))
    ref = torch.nn.functional.conv2d(
        torch.from_numpy(X.astype(np.float64)).reshape(3, 24, 5, 7), Wm.reshape(20, 24, 1, 1),
        torch.from_numpy(b.astype(np.float64))).relu().reshape(3, 20, 35).numpy()
    assert np.all(np.abs(Y - ref) <= 64 * 2.0 ** -53 * A)


def test_zero_sparsity_is_dense_conv():
    """All blocks kept: identical to the unpruned dense product W X + b."""
    W, _, X, b = _rand_case(31, 2, 16, 12, 9, 4)
    M = np.ones((3, 16), np.uint8)
    Y = oracle.conv1x1(W, M, X, b, False, 4)
    ref = np.zeros_like(Y)
    for ci in range(16):                       # same ascending-channel order in double
        ref += W[:, ci].astype(np.float64)[None, :, None] * X[:, ci, :].astype(np.float64)[:, None, :]
    ref += b.astype(np.float64)[None, :, None]
    assert np.array_equal(Y, ref)


@pytest.mark.parametrize("relu", [False, True])
def test_full_sparsity_is_bias_only(relu):
    """All blocks dropped: Y is the broadcast bias (clamped at 0 with ReLU), exactly."""
    W, _, X, b = _rand_case(32, 2, 16, 12, 9, 4)
    M = np.zeros((3, 16), np.uint8)
    Y = oracle.conv1x1(W, M, X, b, relu, 4)
    exp = np.broadcast_to(b.astype(np.float64)[None, :, None], Y.shape)
    if relu:
        exp = np.maximum(exp, 0)
    assert np.array_equal(Y, exp)
    Y0 = oracle.conv1x1(W, M, X, None, relu, 4)
    assert np.array_equal(Y0, np.zeros_like(Y0))


def test_ones_input_gives_masked_row_sums():
    """X == 1 everywhere: Y[n,co,p] = sum of the kept weights of row co + bias[co]."""
    g = 4
    W = _ints(41, (12, 10)).astype(np.float32)
    M = (rng.uniform01(42, 3, 30) < 0.5).astype(np.uint8).reshape(3, 10)
    b = _ints(43, (12,)).astype(np.float32)
    X = np.ones((2, 10, 7), np.float32)
    Y = oracle.conv1x1(W, M, X, b, False, g)
    rows = (W.astype(np.float64) * np.repeat(M, g, 0)).sum(1) + b
    assert np.array_equal(Y, np.broadcast_to(rows[None, :, None], Y.shape))


def test_identity_pattern_copies_channels():
    """Cin == Cout, g=1, only the diagonal kept with weight 1: Y is X, exactly."""
    c = 9
    W = rng.normal(51, 1, c * c).reshape(c, c).astype(np.float32)
    W[np.arange(c), np.arange(c)] = 1.0
    M = np.eye(c, dtype=np.uint8)
    X = rng.normal(52, 2, 2 * c * 6).reshape(2, c, 6).astype(np.float32)
    assert np.array_equal(oracle.conv1x1(W, M, X, None, False, 1), X.astype(np.float64))


def test_block_selects_g_adjacent_output_channels():
    """One kept block (r, c) touches exactly output channels r*g..r*g+g-1 and input channel c."""
    g, cin, cout = 4, 6, 12
    W = np.arange(1, cout * cin + 1, dtype=np.float32).reshape(cout, cin)
    X = np.zeros((1, cin, 2), np.float32)
    X[0, 4, :] = [1.0, 2.0]
    M = np.zeros((3, cin), np.uint8)
    M[1, 4] = 1
    Y = oracle.conv1x1(W, M, X, None, False, g)
    exp = np.zeros((1, cout, 2))
    for co in range(4, 8):
        exp[0, co] = W[co, 4] * np.array([1.0, 2.0])
    assert np.array_equal(Y, exp)


def test_mask_linearity_on_integer_data():
    """Disjoint masks add: Y(M1 u M2) = Y(M1) + Y(M2) without bias/ReLU, exactly on integers."""
    g = 4
    W = _ints(61, (8, 12)).astype(np.float32)
    X = _ints(62, (2, 12, 5)).astype(np.float32)
    u = rng.uniform01(63, 3, 24).reshape(2, 12)
    M1 = (u < 0.33).astype(np.uint8)
    M2 = ((u >= 0.33) & (u < 0.66)).astype(np.uint8)
    y = lambda m: oracle.conv1x1(W, m, X, None, False, g)
    assert np.array_equal(y(M1 | M2), y(M1) + y(M2))


def test_input_channel_permutation_invariance():
    """Permuting X's channels together with W's and the mask's columns leaves Y unchanged."""
    g = 2
    W = _ints(71, (6, 7)).astype(np.float32)
    X = _ints(72, (2, 7, 4)).astype(np.float32)
    M = (rng.uniform01(73, 3, 21) < 0.5).astype(np.uint8).reshape(3, 7)
    b = _ints(74, (6,)).astype(np.float32)
    perm = rng.permutation(75, 1, 7)
    Y1 = oracle.conv1x1(W, M, X, b, True, g)
    Y2 = oracle.conv1x1(W[:, perm].copy(), M[:, perm].copy(), X[:, perm, :].copy(), b, True, g)
    assert np.array_equal(Y1, Y2)


def test_fp16_inputs_are_decoded_exactly():
    """Every finite binary16 pattern, as a weight against X = 1, comes back as its value."""
    bits = np.arange(0, 1 << 16, dtype=np.uint16)
    h = bits.view(np.float16)
    fin = np.isfinite(h)
    W = h[fin].reshape(-1, 1)
    M = np.ones((W.shape[0], 1), np.uint8)
    X = np.ones((1, 1, 1), np.float16)
    Y = oracle.conv1x1(W, M, X, None, False, 1)
    assert np.array_equal(Y.reshape(-1), W.reshape(-1).astype(np.float64))


def test_points_agree_with_full():
    W, M, X, b = _rand_case(81, 3, 10, 12, 11, 4)
    Y, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
    idx = rng.permutation(82, 1, Y.size)[:50]
    v, m = oracle.conv1x1_points(W, M, X, idx, b, True, 4)
    assert np.array_equal(v, Y.reshape(-1)[idx]) and np.array_equal(m, A.reshape(-1)[idx])


def test_scale_is_sum_of_magnitudes():
    W, M, X, b = _rand_case(91, 1, 6, 4, 3, 2)
    _, A = oracle.conv1x1(W, M, X, b, True, 2, want_scale=True)
    Wm = np.abs(W.astype(np.float64)) * np.repeat(M, 2, 0)
    exp = np.einsum("oc,ncp->nop", Wm, np.abs(X.astype(np.float64))) + np.abs(b.astype(np.float64))[None, :, None]
    assert np.allclose(A, exp, rtol=1e-14, atol=0)


# ------------------------------------------------------------------------------------------
# The pins must be able to reject a wrong oracle.

def _pins_pass(mutant, build_dir):
    """Re-run the core pins against a given oracle build; True if all hold."""
    f = lambda *a, **k: oracle.conv1x1(*a, mutant=mutant, build_dir=build_dir, **k)
    ok = True
    # integer exactness, ragged blocks, bias and ReLU (square W so that a transpose is in range)
    g, c = 4, 10
    rows = (c + g - 1) // g
    W = _ints(1, (c, c)).astype(np.float32)
    X = _ints(2, (2, c, 5)).astype(np.float32)
    b = _ints(3, (c,)).astype(np.float32)
    M = (rng.uniform01(4, 3, rows * c) < 0.6).astype(np.uint8).reshape(rows, c)
    for relu in (False, True):
        Y = f(W, M, X, b, relu, g)
        E = _exact(W, M, X, b, relu, g)
        ok &= all(Fraction(float(Y[i])) == E[i] for i in np.ndindex(Y.shape))
    return ok


def test_pins_reject_planted_mistakes(tmp_path):
    assert _pins_pass(0, None)
    for mutant in (1, 2, 3, 4, 5):
        assert not _pins_pass(mutant, str(tmp_path)), f"mutant {mutant} slipped through"
