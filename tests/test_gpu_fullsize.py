"""Parity at the benchmark's full sizes, in the launch configuration the benchmark times
(the tuned one): the first and the last image in full plus a seeded sample of outputs from the
whole batch, each computed by the oracle one by one."""
import json
import os

import numpy as np
import pytest

import oracle
from alcs_workloads import config_layers, make_bias, make_mask, make_weights, make_x, rng, with_batch
from gpu_util import TOL, assert_parity, run_gpu

pytestmark = pytest.mark.gpu


def _check_full_size(alcs, s, n_points=20000, tune=True, cfg=None):
    W, M, X, b = make_weights(s), make_mask(s), make_x(s), make_bias(s)
    kind = s.dtype
    packed = None
    if cfg is not None:     # what the benchmark does with a cached configuration: store it, then call plainly
        packed = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, s.g), 0)
        alcs.alcs_spconv1x1_set_cfg(packed, s.n, s.h, s.w, alcs.ALCS_RELU if s.relu else 0, cfg)
        got = alcs.alcs_spconv1x1_plan(packed, s.n, s.h, s.w, alcs.ALCS_RELU if s.relu else 0)
        assert all(got[k] == v for k, v in cfg.items() if v), (got, cfg)
    Y = run_gpu(alcs, W, M, X, b, s.relu, s.g, h=s.h, wd=s.w, tune=tune, packed=packed)
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


@pytest.mark.parametrize("name", [l.name for l in config_layers(4)])
def test_sweep_cases(alcs, name):
    """Every case of the 512->512 @14x14, batch 256 sweep (5 sparsities x 4 group sizes) and the
    Zipf-skewed rows."""
    s = [l for l in config_layers(4) if l.name == name][0]
    _check_full_size(alcs, s, tune=False)


_TUNED = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2109_00170_b200", "tuned")


def _cached_cfgs(workload):
    path = os.path.join(_TUNED, workload + ".json")
    return json.load(open(path))["layers"] if os.path.exists(path) else {}


@pytest.mark.parametrize("workload,config", [("mbv1_b64", 2), ("rn50_b32", 3)])
def test_cached_launch_configurations_at_full_size(alcs, workload, config):
    """The launch configurations the benchmark replays from its tuning cache, layer by layer at the
    full batch: what is timed is what is checked."""
    cache = _cached_cfgs(workload)
    assert cache, f"no tuning cache for {workload}"
    for s in config_layers(config):
        assert s.name in cache, f"{s.name} missing from the tuning cache"
        _check_full_size(alcs, s, n_points=5000, tune=False, cfg=cache[s.name])
