"""GPU parity of the tensor-core kernels (fp16 weights and activations, fp32 accumulate; launch
configurations with math_mode = 2) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

import oracle
from alcs_workloads import config_layers, make_bias, make_mask, make_weights, make_x, rng
from gpu_util import assert_parity, check_layer, run_gpu

pytestmark = pytest.mark.gpu

MMA = dict(math_mode=2)


def _rand(seed, n, cin, cout, hw, g, density, xpos=True):
    rows = (cout + g - 1) // g
    W = (rng.normal(seed, 1, cout * cin) * cin ** -0.5).reshape(cout, cin).astype(np.float16)
    X = rng.normal(seed, 2, n * cin * hw).reshape(n, cin, hw)
    X = (np.abs(X) if xpos else X).astype(np.float16)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = (0.1 * rng.normal(seed, 4, cout)).astype(np.float32)
    return W, M, X, b


SHAPES = [
    # n, cin, cout, hw, g, density: ragged pixel tails, rows of X that are not 16-byte multiples,
    # output channels that are not a multiple of g, channel counts below one step and one chunk
    (2, 64, 256, 3136, 8, 0.25), (5, 200, 68, 49, 8, 0.25), (3, 130, 72, 196, 8, 0.3),
    (1, 5, 8, 3, 8, 0.6), (2, 33, 24, 50, 8, 0.4), (1, 300, 40, 1030, 8, 0.15),
    (2, 90, 50, 100, 16, 0.5), (1, 256, 64, 777, 16, 0.25), (7, 257, 44, 12, 4, 0.3),
    (2, 100, 36, 392, 4, 0.2), (1, 1, 8, 1, 8, 1.0), (3, 17, 16, 131, 8, 1.0),
]


@pytest.mark.parametrize("n,cin,cout,hw,g,density", SHAPES)
@pytest.mark.parametrize("y_f32", [False, True])
def test_shapes(alcs, n, cin, cout, hw, g, density, y_f32):
    W, M, X, b = _rand(500 + cin + hw, n, cin, cout, hw, g, density)
    check_layer(alcs, W, M, X, b, True, g, cfg=MMA, y_f32=y_f32)


@pytest.mark.parametrize("copy_mode", [1, 2])
@pytest.mark.parametrize("relu,with_bias", [(False, True), (True, False), (False, False)])
def test_epilogue_and_copy_modes(alcs, copy_mode, relu, with_bias):
    W, M, X, b = _rand(611, 3, 96, 48, 400, 8, 0.3, xpos=False)
    check_layer(alcs, W, M, X, b if with_bias else None, relu, 8, cfg=dict(math_mode=2, copy_mode=copy_mode))


@pytest.mark.parametrize("math_mode", [1, 2])
@pytest.mark.parametrize("n,cin,cout,hw", [(5, 136, 72, 196), (3, 70, 40, 12), (2, 64, 32, 400), (2, 48, 24, 49)])
@pytest.mark.parametrize("y_f32", [False, True])
def test_unpadded_rows_staged_directly(alcs, math_mode, n, cin, cout, hw, y_f32):
    """copy_mode 3: rows that are a multiple of 8 but not of 16 bytes long (hw = 196, 12) are staged as
    they are, with 8-byte copies, by the tensor-core and by the CUDA-core fp16 kernels; for the other
    row lengths the mode must behave like copy_mode 1."""
    W, M, X, b = _rand(700 + hw, n, cin, cout, hw, 8, 0.3, xpos=False)
    check_layer(alcs, W, M, X, b, True, 8, cfg=dict(math_mode=math_mode, copy_mode=3), y_f32=y_f32)


def test_dense_empty_and_ragged_rows(alcs):
    """0 % sparsity, 100 % sparsity (bias only), and rows with 0, 1, 15, 16, 17 and 33 kept blocks
    (below, at and above one 16-block step)."""
    n, cin, cout, hw, g = 2, 80, 48, 260, 8
    W, M, X, b = _rand(77, n, cin, cout, hw, g, 0.3)
    check_layer(alcs, W, np.ones_like(M), X, b, True, g, cfg=MMA)
    Y = run_gpu(alcs, W, np.zeros_like(M), X, b, False, g, cfg=MMA, y_f32=True)
    assert np.array_equal(Y, np.broadcast_to(b[None, :, None], Y.shape))
    M2 = np.zeros_like(M)
    for r, cnt in enumerate((0, 1, 15, 16, 17, 33)):
        M2[r, rng.bits64(78, r, cin).argsort()[:cnt]] = 1
    check_layer(alcs, W, M2, X, b, False, g, cfg=MMA)


def test_small_integers_exact(alcs):
    """Small integer weights and activations: every product and partial sum is exact in fp32, so
    the tensor-core path must agree with the oracle bit for bit."""
    n, cin, cout, hw, g = 2, 120, 64, 300, 8
    W = ((rng.bits64(5, 1, cout * cin) % np.uint64(9)).astype(np.int64) - 4).reshape(cout, cin).astype(np.float16)
    X = ((rng.bits64(5, 2, n * cin * hw) % np.uint64(9)).astype(np.int64) - 4).reshape(n, cin, hw).astype(np.float16)
    M = (rng.uniform01(5, 3, (cout // g) * cin) < 0.3).astype(np.uint8).reshape(cout // g, cin)
    b = np.arange(cout, dtype=np.float32) - 30
    check_layer(alcs, W, M, X, b, False, g, cfg=MMA, y_f32=True, exact=True)


def test_every_row_group_and_chunk(alcs):
    n, cin, cout, hw, g = 2, 160, 512, 300, 8
    W, M, X, b = _rand(91, n, cin, cout, hw, g, 0.25)
    Yref, A = oracle.conv1x1(W, M, X, b, True, g, want_scale=True)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    ran = 0
    for rgs in (0, 4, 7, 16, 64):
        for kc in (16, 64, 160):
            try:
                Y = run_gpu(alcs, W, M, X, b, True, g, cfg=dict(math_mode=2, row_groups=rgs, chunk_channels=kc), packed=p)
            except alcs.AlcsError as e:
                assert e.status == alcs.ALCS_ERR_UNSUPPORTED
                continue
            assert_parity(Y, Yref, A, "f16")
            ran += 1
    assert ran >= 8


def test_resnet_layers_batch2(alcs):
    """The ResNet-50 bottleneck shapes of the fp16 configuration at a batch the oracle finishes
    quickly, through the tensor-core kernels."""
    from alcs_workloads import with_batch
    for s in (with_batch(s0, 2) for s0 in config_layers(3)):
        W, M, X, b = make_weights(s), make_mask(s), make_x(s), make_bias(s)
        check_layer(alcs, W, M, X, b, s.relu, s.g, cfg=MMA, h=s.h, wd=s.w)
