"""GPU parity of the small-problem kernel of the pointwise convolution (math_mode = 3: no staging, the
warps of a thread block share one block row's columns) against the oracle, through the C ABI."""
import numpy as np
import pytest

import oracle
from alcs_workloads import config_layers, make_bias, make_mask, make_weights, make_x, rng
from gpu_util import assert_parity, check_layer, run_gpu

pytestmark = pytest.mark.gpu


def _case(seed, n, cin, cout, hw, g, density=0.3, ints=False):
    rows = (cout + g - 1) // g
    if ints:
        mk = lambda s, shape: ((rng.bits64(seed, s, int(np.prod(shape))) % np.uint64(9)).astype(np.int64) - 4
                               ).reshape(shape).astype(np.float32)
        W, X, b = mk(1, (cout, cin)), mk(2, (n, cin, hw)), mk(4, (cout,))
    else:
        W = rng.normal(seed, 1, cout * cin, sigma=cin ** -0.5).reshape(cout, cin).astype(np.float32)
        X = rng.uniform01(seed, 2, n * cin * hw).reshape(n, cin, hw)
        b = rng.normal(seed, 4, cout, sigma=0.1).astype(np.float32)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    return W, M, X, b


# (g, pixels per lane, warps): the partial sums, warps * g * pixels * 128 bytes, must fit 48 KB of shared memory
SHAPES = [(g, p, ks) for g, p in [(1, 8), (1, 2), (2, 8), (4, 8), (4, 4), (4, 2), (8, 4), (8, 2), (16, 2)]
          for ks in (1, 4, 16) if ks * g * p * 128 <= 48 * 1024]


@pytest.mark.parametrize("g,p,ks", SHAPES)
@pytest.mark.parametrize("hw", [49, 196, 300, 1])
def test_gather_matches_oracle(alcs, g, p, ks, hw):
    W, M, X, b = _case(700 + g + hw, 2, 70, 44, hw, g)            # cout not a multiple of 8 or 16
    M[1, :] = 0                                                   # an empty block row
    check_layer(alcs, W, M, X, b, True, g, cfg=dict(math_mode=3, pixels_per_lane=p, warps=ks))


def test_gather_integer_data_exact(alcs):
    W, M, X, b = _case(31, 3, 40, 32, 196, 4, ints=True)
    check_layer(alcs, W, M, X, b, True, 4, cfg=dict(math_mode=3, pixels_per_lane=8, warps=8), exact=True)
    check_layer(alcs, W, M, X, None, False, 4, cfg=dict(math_mode=3, pixels_per_lane=2, warps=5), exact=True)


def test_gather_is_deterministic(alcs):
    W, M, X, b = _case(32, 1, 256, 128, 196, 4)
    cfg = dict(math_mode=3, pixels_per_lane=8, warps=8)
    Y1 = run_gpu(alcs, W, M, X, b, True, 4, cfg=cfg)
    Y2 = run_gpu(alcs, W, M, X, b, True, 4, cfg=cfg)
    assert np.array_equal(Y1, Y2)


def test_gather_on_batch1_stack(alcs):
    """Every layer of the batch-1 MobileNetV1 stack through the small-problem kernel, and through
    whatever the tuner picks for it (the staged or the small-problem kernel)."""
    for s in config_layers(1):
        W, M, X, b = make_weights(s), make_mask(s), make_x(s), make_bias(s)
        Yref, A = oracle.conv1x1(W, M, X, b, s.relu, s.g, want_scale=True)
        Y = run_gpu(alcs, W, M, X, b, s.relu, s.g, cfg=dict(math_mode=3, pixels_per_lane=8, warps=8), h=s.h, wd=s.w)
        assert_parity(Y, Yref, A, "f32")
        Y = run_gpu(alcs, W, M, X, b, s.relu, s.g, h=s.h, wd=s.w, tune=True)
        assert_parity(Y, Yref, A, "f32")


def test_gather_rejects_what_it_cannot_do(alcs):
    import torch
    W, M, X, b = _case(33, 1, 16, 16, 64, 4)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W.astype(np.float16), M, 4), 0)       # fp16 weights
    x = torch.zeros((1, 16, 64), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 16, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, x, y, 1, 8, 8, None, 0, None, dict(math_mode=3, pixels_per_lane=4, warps=4))
    assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    x, y = x.float(), y.float()
    with pytest.raises(alcs.AlcsError):
        alcs.alcs_spconv1x1(p, x, y, 1, 8, 8, None, 0, None, dict(math_mode=3, pixels_per_lane=8, warps=32))
