"""GPU parity of copy_mode 4: X is first copied into a tile-major layout ([pixel tile][channel][tile pixels]),
from which a work item stages a chunk of channel rows with a few large bulk copies.  The product
W_sparse * X (paper, Section 3.2.2) must not depend on how X reaches shared memory, so every case is the
plain oracle comparison with that mode forced: all element types and kernels, ragged pixel tails, images
smaller and larger than a tile, rows that need padding, stride and residual, the allocation-free entry
point and a layer stack."""
import numpy as np
import pytest

import oracle
from alcs_workloads import rng
from gpu_util import assert_parity, check_layer

pytestmark = pytest.mark.gpu


def _rand(seed, n, cin, cout, hw, g, density, dtype):
    rows = (cout + g - 1) // g
    W = (rng.normal(seed, 1, cout * cin) * cin ** -0.5).reshape(cout, cin).astype(dtype)
    X = rng.normal(seed, 2, n * cin * hw).reshape(n, cin, hw).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = (0.1 * rng.normal(seed, 4, cout)).astype(np.float32)
    return W, M, X, b


# n, cin, cout, hw, g, density
SHAPES = [(12, 96, 64, 196, 4, 0.3), (20, 70, 36, 49, 4, 0.4), (9, 33, 20, 50, 4, 0.5), (10, 40, 24, 1030, 4, 0.25),
          (16, 17, 8, 3, 4, 1.0), (9, 130, 72, 131, 4, 0.2), (40, 64, 32, 12, 4, 0.3)]


@pytest.mark.parametrize("n,cin,cout,hw,g,density", SHAPES)
@pytest.mark.parametrize("pixels_per_lane", [4, 8])
def test_fp32(alcs, n, cin, cout, hw, g, density, pixels_per_lane):
    W, M, X, b = _rand(1300 + hw, n, cin, cout, hw, g, density, np.float32)
    cfg = dict(copy_mode=4, pixels_per_lane=pixels_per_lane)
    check_layer(alcs, W, M, X, b, True, g, cfg=cfg)
    check_layer(alcs, W, M, X, None, False, g, cfg=dict(copy_mode=4, pixels_per_lane=pixels_per_lane, chunk_channels=32, stages=2))


@pytest.mark.parametrize("n,cin,cout,hw,g,density", [(12, 96, 64, 196, 8, 0.3), (20, 200, 72, 49, 8, 0.25), (9, 48, 40, 50, 8, 0.5),
                                                     (10, 64, 24, 777, 16, 0.3), (16, 17, 8, 3, 8, 1.0)])
@pytest.mark.parametrize("math_mode", [1, 2])
@pytest.mark.parametrize("y_f32", [False, True])
def test_fp16(alcs, n, cin, cout, hw, g, density, math_mode, y_f32):
    W, M, X, b = _rand(1400 + hw, n, cin, cout, hw, g, density, np.float16)
    check_layer(alcs, W, M, X, b, True, g, cfg=dict(copy_mode=4, math_mode=math_mode), y_f32=y_f32)


def test_it_is_the_mode_that_runs(alcs):
    """The plan for a forced copy_mode 4 reports that mode, and a batch of at most 8 images has no such plan."""
    W, M, X, b = _rand(1500, 12, 64, 32, 196, 4, 0.3, np.float32)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    alcs.alcs_spconv1x1_set_cfg(p, 12, 14, 14, 0, dict(copy_mode=4))
    assert alcs.alcs_spconv1x1_plan(p, 12, 14, 14, 0)["copy_mode"] == 4
    with pytest.raises(alcs.AlcsError):
        alcs.alcs_spconv1x1_set_cfg(p, 2, 14, 14, 0, dict(copy_mode=4))
    alcs.alcs_packed_free(p)


@pytest.mark.parametrize("stride", [1, 2])
def test_stride_and_residual(alcs, stride):
    import torch
    dev = torch.device("cuda:0")
    n, cin, cout, h, wd, g = 10, 72, 40, 15, 13, 4
    W, M, X, b = _rand(1600 + stride, n, cin, cout, h * wd, g, 0.35, np.float32)
    oh, ow = -(-h // stride), -(-wd // stride)
    R = rng.normal(1600, 9, n * cout * oh * ow).reshape(n, cout, oh * ow).astype(np.float32)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    xd, rd, bd = (torch.from_numpy(a).to(dev) for a in (X, R, b))
    yd = torch.full((n, cout, oh * ow), float("nan"), device=dev)
    alcs.alcs_spconv1x1_ex(p, xd, yd, n, h, wd, stride, bd, rd, alcs.ALCS_RELU, torch.cuda.current_stream(), dict(copy_mode=4))
    torch.cuda.synchronize()
    assert alcs.alcs_packed_status(p) == 0
    Yref, A = oracle.conv1x1_ex(W, M, X.reshape(n, cin, h, wd), b, R, True, g, stride, want_scale=True)
    assert_parity(yd.cpu().numpy(), Yref, A, "f32")
    alcs.alcs_packed_free(p)


def test_stack_and_allocation_free_call(alcs):
    import torch
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream()
    layers, keep = [], []
    for i, (n, cin, cout, hw) in enumerate([(12, 64, 48, 49), (12, 48, 32, 196)]):
        W, M, X, b = _rand(1700 + i, n, cin, cout, hw, 4, 0.4, np.float32)
        p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
        h = wd = int(round(hw ** 0.5))
        alcs.alcs_spconv1x1_set_cfg(p, n, h, wd, alcs.ALCS_RELU, dict(copy_mode=4))
        xd, bd = torch.from_numpy(X).to(dev), torch.from_numpy(b).to(dev)
        yd = torch.full((n, cout, hw), float("nan"), device=dev)
        layers.append(dict(w=p, x=xd, y=yd, n=n, h=h, wd=wd, bias=bd, flags=alcs.ALCS_RELU))
        Yref, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
        keep.append((yd, Yref, A))
    for graph in (0, alcs.ALCS_STACK_GRAPH):
        st = alcs.alcs_stack_create(layers, graph)
        assert [alcs.alcs_stack_layer_cfg(st, i)["copy_mode"] for i in range(2)] == [4, 4]
        for _ in range(2):
            for yd, _, _ in keep:
                yd.fill_(float("nan"))
            torch.cuda.synchronize()
            alcs.alcs_stack_run(st, stream)
            stream.synchronize()
            for yd, Yref, A in keep:
                assert_parity(yd.cpu().numpy(), Yref, A, "f32")
        alcs.alcs_stack_destroy(st)
    # the allocation-free entry point takes the same plan (its schedule is resident after the runs above)
    L = layers[0]
    keep[0][0].fill_(float("nan"))
    with torch.cuda.stream(stream):
        alcs.alcs_spconv1x1_noalloc(L["w"], L["x"], L["y"], L["n"], L["h"], L["wd"], L["bias"], L["flags"], stream)
    stream.synchronize()
    assert_parity(keep[0][0].cpu().numpy(), keep[0][1], keep[0][2], "f32")
