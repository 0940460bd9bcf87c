"""Parity at the benchmark's full sizes, in the launch configuration the benchmark times
(the tuned one): the first and the last image in full plus a seeded sample of outputs from the
whole batch, each computed by the oracle one by one."""
import numpy as np
import pytest

import oracle
from alcs_workloads import config_layers, make_bias, make_mask, make_weights, make_x, rng, with_batch
from gpu_util import TOL, assert_parity, run_gpu

pytestmark = pytest.mark.gpu


def _check_full_size(alcs, s, n_points=20000, tune=True):
    W, M, X, b = make_weights(s), make_mask(s), make_x(s), make_bias(s)
    kind = s.dtype
    Y = run_gpu(alcs, W, M, X, b, s.relu, s.g, h=s.h, wd=s.w, tune=tune)
    assert np.isfinite(Y).all()
    for img in (0, s.n - 1):
        Yref, A = oracle.conv1x1(W, M, X[img:img + 1], b, s.relu, s.g, want_scale=True)
        assert_parity(Y[img:img + 1], Yref, A, kind)
    idx = (rng.bits64(s.seed, 4242, n_points) % np.uint64(Y.size)).astype(np.int64)
    ref, A = oracle.conv1x1_points(W, M, X, idx, b, s.relu, s.g)
    d = np.abs(Y.reshape(-1)[idx].astype(np.float64) - ref)
    assert (d <= TOL[kind] * A + 1e-300).all(), f"worst ratio {(d / np.maximum(A, 1e-300)).max():.3e}"


@pytest.mark.parametrize("li", range(13))
def test_mobilenet_batch64_layers(alcs, li):
    """The batch-64 MobileNetV1 pointwise stack with per-layer drawn sparsity."""
    _check_full_size(alcs, config_layers(2)[li])


@pytest.mark.parametrize("li", range(8))
def test_resnet50_fp16_layers(alcs, li):
    """ResNet-50 bottleneck 1x1 layers, batch 32, g=8, fp16 in / fp32 accumulate."""
    _check_full_size(alcs, config_layers(3)[li], tune=False)


@pytest.mark.parametrize("name", ["sweep_g1_s90", "sweep_g4_s50", "sweep_g4_s95", "sweep_g8_s80",
                                  "sweep_g16_s70", "sweep_g4_zipf1.2"])
def test_sweep_cases(alcs, name):
    """Corners of the 512->512 @14x14, batch 256 sweep, including the Zipf-skewed rows."""
    s = [l for l in config_layers(4) if l.name == name][0]
    _check_full_size(alcs, s, tune=False)
