"""GPU parity of the general k x k sparse convolution (alcs_spconv2d, through the C ABI) against the
CPU oracle, element by element.  Tolerance as for the pointwise kernels:
|Y - Yref| <= 1e-5 * A with A = |bias| + sum |Wm||X|; exact equality where the arithmetic is exact
(small-integer data, empty rows, 100 % sparsity)."""
import numpy as np
import pytest

import oracle
from alcs_workloads import (make_bias2d, make_mask2d, make_weights2d, make_x2d, resnet18_3x3_stack, rng)
from alcs_workloads.conv2d import Conv2dSpec
from gpu_util import assert_parity

pytestmark = pytest.mark.gpu


def _run(alcs, W, M, X, b, relu, g, stride, pad, cfg=None):
    import torch
    dev = torch.device("cuda:0")
    cout, cin, kh, kw = W.shape
    n, _, h, wd = X.shape
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (wd + 2 * pad - kw) // stride + 1
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W.reshape(cout, cin * kh * kw), M, g), 0)
    xd = torch.from_numpy(np.ascontiguousarray(X)).to(dev)
    yd = torch.full((n, cout, oh, ow), float("nan"), device=dev)
    bd = None if b is None else torch.from_numpy(b).to(dev)
    for _ in range(2):      # second call: schedule already resident
        yd.fill_(float("nan"))
        alcs.alcs_spconv2d(p, xd, yd, n, cin, h, wd, kh, kw, stride, pad, bd, alcs.ALCS_RELU if relu else 0,
                           torch.cuda.current_stream(), cfg)
        torch.cuda.synchronize()
    return yd.cpu().numpy()


def _case(seed, n, cin, cout, h, w, kh, kw, g, density=0.4, ints=False):
    rows = (cout + g - 1) // g
    K = cin * kh * kw
    if ints:
        mk = lambda s, shape: ((rng.bits64(seed, s, int(np.prod(shape))) % np.uint64(9)).astype(np.int64) - 4
                               ).reshape(shape).astype(np.float32)
        W, X, b = mk(1, (cout, cin, kh, kw)), mk(2, (n, cin, h, w)), mk(4, (cout,))
    else:
        W = rng.normal(seed, 1, cout * K, sigma=K ** -0.5).reshape(cout, cin, kh, kw).astype(np.float32)
        X = rng.uniform01(seed, 2, n * cin * h * w).reshape(n, cin, h, w)
        b = rng.normal(seed, 4, cout, sigma=0.1).astype(np.float32)
    M = (rng.uniform01(seed, 3, rows * K) < density).astype(np.uint8).reshape(rows, K)
    return W, M, X, b


GEOMS = [  # n, cin, cout, h, w, kh, kw, stride, pad, g
    (2, 16, 32, 20, 20, 3, 3, 1, 1, 4),
    (2, 16, 32, 21, 19, 3, 3, 2, 1, 4),      # odd sizes, stride 2
    (1, 8, 16, 56, 56, 3, 3, 1, 1, 4),       # several strips and position tiles
    (3, 24, 20, 9, 11, 3, 3, 1, 0, 4),       # no padding (the paper's formula as printed)
    (2, 12, 16, 14, 14, 5, 5, 1, 2, 4),
    (2, 12, 16, 15, 15, 5, 3, 2, 2, 8),
    (2, 6, 10, 30, 30, 7, 7, 2, 3, 2),       # cout not a multiple of g
    (2, 32, 32, 7, 7, 3, 3, 1, 1, 16),
    (2, 32, 17, 7, 7, 3, 3, 1, 1, 1),        # unstructured
    (4, 20, 24, 12, 40, 1, 1, 1, 0, 4),      # 1x1 through the general path
    (3, 32, 16, 15, 14, 1, 1, 2, 0, 4),      # strided 1x1 (projection shortcuts of ResNets)
    (1, 5, 8, 33, 65, 3, 2, 1, 1, 4),        # even kernel width, wide image
    (1, 64, 64, 28, 28, 3, 3, 2, 1, 4),
]


@pytest.mark.parametrize("geom", GEOMS, ids=lambda g: "n{}c{}o{}_{}x{}_k{}x{}s{}p{}g{}".format(*g))
@pytest.mark.parametrize("relu", [False, True])
def test_conv2d_matches_oracle(alcs, geom, relu):
    n, cin, cout, h, w, kh, kw, stride, pad, g = geom
    W, M, X, b = _case(500 + cin + kh, n, cin, cout, h, w, kh, kw, g)
    Y = _run(alcs, W, M, X, b, relu, g, stride, pad)
    Yref, A = oracle.conv2d(W, M, X, b, relu, g, stride, pad, want_scale=True)
    assert_parity(Y, Yref, A, "f32")


@pytest.mark.parametrize("cfg", [dict(chunk_channels=8), dict(chunk_channels=5, positions_per_lane=4),
                                 dict(chunk_channels=16, strip_rows=3), dict(chunk_channels=1, positions_per_lane=2),
                                 dict(strip_rows=2, row_groups=2), dict(positions_per_lane=2, strip_rows=5)])
@pytest.mark.parametrize("stride", [1, 2])
def test_conv2d_forced_configurations(alcs, cfg, stride):
    """Channel chunks (one block row per warp, accumulators kept across chunks, a ragged last chunk),
    several row groups, short strips: every path of the kernel against the oracle."""
    W, M, X, b = _case(91, 2, 24, 40, 18, 19, 3, 3, 4)
    Y = _run(alcs, W, M, X, b, True, 4, stride, 1, cfg)
    Yref, A = oracle.conv2d(W, M, X, b, True, 4, stride, 1, want_scale=True)
    assert_parity(Y, Yref, A, "f32")


@pytest.mark.parametrize("stride", [1, 2])
def test_conv2d_several_images_per_item(alcs, stride):
    """Small images: 2 or 4 whole images share one position tile (odd batch: the last item is short),
    with all channels at once and with channel chunks."""
    W, M, X, b = _case(93, 7, 20, 24, 7 * stride, 7 * stride, 3, 3, 4)
    Yref, A = oracle.conv2d(W, M, X, b, True, 4, stride, 1, want_scale=True)
    for cfg in (dict(images_per_item=4), dict(images_per_item=2, positions_per_lane=4),
                dict(images_per_item=4, chunk_channels=8), dict(images_per_item=2, chunk_channels=7)):
        assert_parity(_run(alcs, W, M, X, b, True, 4, stride, 1, cfg), Yref, A, "f32")


@pytest.mark.parametrize("stride", [1, 2])
def test_conv2d_integer_data_exact(alcs, stride):
    """Small-integer data: every order of summation gives the same fp32 result, so the kernel must
    equal the oracle bit for bit."""
    W, M, X, b = _case(77, 2, 10, 12, 17, 18, 3, 3, 4, ints=True)
    Y = _run(alcs, W, M, X, b, True, 4, stride, 1)
    Yref, A = oracle.conv2d(W, M, X, b, True, 4, stride, 1, want_scale=True)
    assert_parity(Y, Yref, A, "f32", exact=True)


def test_conv2d_empty_rows_and_full_sparsity(alcs):
    W, M, X, b = _case(78, 2, 8, 16, 10, 10, 3, 3, 4)
    M[1, :] = 0                                   # one empty block row: bias only, X never read
    Y = _run(alcs, W, M, X, b, False, 4, 1, 1)
    Yref, A = oracle.conv2d(W, M, X, b, False, 4, 1, 1, want_scale=True)
    assert_parity(Y, Yref, A, "f32")
    assert np.array_equal(Y[:, 4:8], np.broadcast_to(b[4:8][None, :, None, None], Y[:, 4:8].shape))
    M[:] = 0
    Y = _run(alcs, W, M, X, b, True, 4, 1, 1)
    assert np.array_equal(Y, np.broadcast_to(np.maximum(b, 0)[None, :, None, None], Y.shape))


def test_conv2d_unit_tap_shift(alcs):
    """A single unit weight at tap (r, s) copies the input shifted by (r, s): the paper's h+r, w+s."""
    cin, cout, h, w = 4, 4, 12, 13
    X = rng.uniform01(5, 2, cin * h * w).reshape(1, cin, h, w)
    for r, s in [(0, 2), (2, 1)]:
        W = np.zeros((cout, cin, 3, 3), np.float32)
        W[1, 2, r, s] = 1.0
        M = np.zeros((1, cin * 9), np.uint8)
        M[0, (2 * 3 + r) * 3 + s] = 1
        Y = _run(alcs, W, M, X, None, False, 4, 1, 0)
        exp = np.zeros((1, cout, h - 2, w - 2), np.float32)
        exp[0, 1] = X[0, 2, r:r + h - 2, s:s + w - 2]
        assert np.array_equal(Y, exp)


def test_conv2d_resnet18_layers_sampled(alcs):
    """The benchmark's ResNet-18 3x3 layers at batch 2 (same weights and masks as at full batch):
    first image in full, sampled points of the last."""
    for s in resnet18_3x3_stack(batch=2):
        W, M, X, b = make_weights2d(s), make_mask2d(s), make_x2d(s), make_bias2d(s)
        Y = _run(alcs, W, M, X, b, True, s.g, s.stride, s.pad)
        idx = rng.permutation(s.seed, 9, Y.size)[:20000]
        v, m = oracle.conv2d_points(W, M, X, idx, b, True, s.g, s.stride, s.pad)
        d = np.abs(Y.reshape(-1)[idx].astype(np.float64) - v)
        assert np.isfinite(Y).all() and np.all(d <= 1e-5 * m + 1e-300), s.name


def test_conv2d_resnet18_layers_full_batch_sampled(alcs):
    """The same layers at the benchmark's batch (32), i.e. in the launch configurations the benchmark
    times (several images per item, channel chunks, small strips): sampled points against the oracle."""
    for s in resnet18_3x3_stack(batch=32):
        W, M, X, b = make_weights2d(s), make_mask2d(s), make_x2d(s), make_bias2d(s)
        Y = _run(alcs, W, M, X, b, True, s.g, s.stride, s.pad)
        idx = np.concatenate([rng.permutation(s.seed, 10, Y.size)[:6000], np.arange(Y.size - 200, Y.size), np.arange(200)])
        v, m = oracle.conv2d_points(W, M, X, idx, b, True, s.g, s.stride, s.pad)
        d = np.abs(Y.reshape(-1)[idx].astype(np.float64) - v)
        assert np.isfinite(Y).all() and np.all(d <= 1e-5 * m + 1e-300), s.name


def test_conv2d_errors(alcs):
    import torch
    W, M, X, b = _case(79, 1, 4, 8, 6, 6, 3, 3, 4)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W.reshape(8, 36), M, 4), 0)
    x = torch.zeros((1, 4, 6, 6), device="cuda")
    y = torch.zeros((1, 8, 6, 6), device="cuda")
    for args, code in [((1, 5, 6, 6, 3, 3, 1, 1), alcs.ALCS_ERR_SHAPE),       # cin*kh*kw mismatch
                       ((1, 4, 6, 6, 3, 3, 3, 1), alcs.ALCS_ERR_SHAPE),       # 4*3*3 ok but stride 3 ...
                       ((1, 4, 1, 1, 3, 3, 1, 0), alcs.ALCS_ERR_SHAPE)]:      # kernel larger than image
        with pytest.raises(alcs.AlcsError) as e:
            alcs.alcs_spconv2d(p, x, y, *args)
        if args[6] == 3:
            assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED
        else:
            assert e.value.status == code
    alcs.alcs_spconv2d(p, x, y, 0, 4, 6, 6, 3, 3, 1, 1)      # n == 0: no-op
    plan = alcs.alcs_spconv2d_plan(p, 1, 4, 6, 6, 3, 3, 1, 1)
    assert plan["positions_per_lane"] in (2, 4, 8) and plan["strip_rows"] >= 1
