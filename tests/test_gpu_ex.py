"""GPU parity of alcs_spconv1x1_ex (stride and residual operand) against the oracle's definition:
y = act(sum_c W x[..., ::s, ::s] + bias + residual), the residual added before the activation and
before the single rounding of an fp16 output."""
import numpy as np
import pytest

import oracle
from alcs_workloads import rng
from gpu_util import TOL, assert_parity

pytestmark = pytest.mark.gpu


def _case(seed, n, cin, cout, h, wd, g, density, stride, dtype=np.float32, res_dtype=None):
    rows = (cout + g - 1) // g
    W = (rng.normal(seed, 1, cout * cin) * cin ** -0.5).reshape(cout, cin).astype(dtype)
    X = rng.normal(seed, 2, n * cin * h * wd).reshape(n, cin, h, wd).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = (0.1 * rng.normal(seed, 4, cout)).astype(np.float32)
    oh, ow = -(-h // stride), -(-wd // stride)
    R = rng.normal(seed, 5, n * cout * oh * ow).reshape(n, cout, oh * ow).astype(res_dtype or dtype)
    return W, M, X, b, R


def _run(alcs, W, M, X, b, R, relu, g, stride, y_f32=False, cfg=None, packed=None):
    import torch
    dev = torch.device("cuda:0")
    n, cin, h, wd = X.shape
    cout = W.shape[0]
    oh, ow = -(-h // stride), -(-wd // stride)
    p = packed or alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    xd = torch.from_numpy(np.ascontiguousarray(X)).to(dev)
    ydt = torch.float32 if (W.dtype == np.float32 or y_f32) else torch.float16
    yd = torch.full((n, cout, oh * ow), float("nan"), dtype=ydt, device=dev)
    rd = None if R is None else torch.from_numpy(R).to(dev)
    bd = None if b is None else torch.from_numpy(b).to(dev)
    flags = (alcs.ALCS_RELU if relu else 0) | (alcs.ALCS_Y_F32 if y_f32 else 0)
    alcs.alcs_spconv1x1_ex(p, xd, yd, n, h, wd, stride, bd, rd, flags, torch.cuda.current_stream(), cfg)
    torch.cuda.synchronize()
    return yd.cpu().numpy()


def _check(alcs, W, M, X, b, R, relu, g, stride, kind, **kw):
    Y = _run(alcs, W, M, X, b, R, relu, g, stride, **kw)
    Yref, A = oracle.conv1x1_ex(W, M, X, b, R, relu, g, stride, want_scale=True)
    return assert_parity(Y, Yref, A, kind)


# n, cin, cout, h, wd, g, stride
SHAPES = [(3, 96, 64, 14, 14, 4, 1), (5, 70, 36, 7, 7, 4, 1), (2, 40, 24, 10, 5, 4, 1), (1, 64, 32, 28, 28, 4, 1),
          (3, 96, 64, 14, 14, 4, 2), (4, 80, 40, 7, 7, 4, 2), (2, 33, 20, 15, 9, 2, 2), (2, 48, 16, 12, 12, 1, 3),
          (1, 128, 64, 56, 56, 4, 2), (9, 100, 48, 8, 8, 8, 2), (2, 60, 64, 6, 11, 16, 2)]


@pytest.mark.parametrize("n,cin,cout,h,wd,g,stride", SHAPES)
def test_fp32_stride_and_residual(alcs, n, cin, cout, h, wd, g, stride):
    W, M, X, b, R = _case(n + cin + h, n, cin, cout, h, wd, g, 0.35, stride)
    _check(alcs, W, M, X, b, R, True, g, stride, "f32")
    _check(alcs, W, M, X, None, R, False, g, stride, "f32")
    if stride > 1:
        _check(alcs, W, M, X, b, None, True, g, stride, "f32")


@pytest.mark.parametrize("n,cin,cout,h,wd,g,stride", [(3, 96, 64, 14, 14, 8, 1), (5, 80, 40, 7, 7, 8, 1), (2, 64, 64, 28, 28, 8, 2),
                                                     (4, 100, 48, 7, 7, 16, 2), (2, 72, 32, 9, 13, 8, 2), (3, 64, 32, 14, 14, 4, 2)])
@pytest.mark.parametrize("math_mode", [1, 2])
def test_fp16_stride_and_residual(alcs, n, cin, cout, h, wd, g, stride, math_mode):
    W, M, X, b, R = _case(7 * n + cin + h, n, cin, cout, h, wd, g, 0.3, stride, np.float16)
    cfg = dict(math_mode=math_mode)
    _check(alcs, W, M, X, b, R, True, g, stride, "f16", cfg=cfg)
    _check(alcs, W, M, X, b, R, False, g, stride, "f16", cfg=cfg)
    R32 = R.astype(np.float32)
    _check(alcs, W, M, X, b, R32, True, g, stride, "f16", cfg=cfg, y_f32=True)
    # rows staged without the repacking pass where they allow it (14x14 at stride 1), else as before
    direct = dict(math_mode=math_mode, copy_mode=3)
    _check(alcs, W, M, X, b, R, True, g, stride, "f16", cfg=direct)
    _check(alcs, W, M, X, b, R32, False, g, stride, "f16", cfg=direct, y_f32=True)


def test_residual_is_added_before_the_activation_exactly(alcs):
    """Small integers: every sum is exact, so the result must equal the oracle bit for bit, and a large
    negative residual must clamp outputs whose convolution part is positive."""
    n, cin, cout, h, wd, g = 2, 32, 16, 8, 8, 4
    W = (rng.bits64(1, 7, cout * cin) % np.uint64(5)).astype(np.float32).reshape(cout, cin)
    X = (rng.bits64(2, 7, n * cin * h * wd) % np.uint64(4)).astype(np.float32).reshape(n, cin, h, wd)
    M = np.ones((cout // g, cin), np.uint8)
    R = -np.full((n, cout, 16), 1000.0, np.float32)
    R[:, ::2] = 3.0
    Y = _run(alcs, W, M, X, None, R, True, g, 2)
    Yref = oracle.conv1x1_ex(W, M, X, None, R, True, g, 2)
    assert np.array_equal(Y.astype(np.float64), Yref)
    assert (Y[:, 1::2] == 0).all() and (Y[:, ::2] >= 3).all()


def test_stack_layers_with_stride_and_residual(alcs):
    import torch
    dev = torch.device("cuda:0")
    specs = [(2, 48, 32, 14, 14, 4, 2), (2, 64, 32, 7, 7, 4, 1), (2, 40, 24, 9, 9, 4, 1)]
    layers, keep = [], []
    for i, (n, cin, cout, h, wd, g, s) in enumerate(specs):
        W, M, X, b, R = _case(900 + i, n, cin, cout, h, wd, g, 0.4, s)
        if i == 2:
            R = None
        p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
        oh, ow = -(-h // s), -(-wd // s)
        xd = torch.from_numpy(X).to(dev)
        yd = torch.full((n, cout, oh * ow), float("nan"), device=dev)
        rd = None if R is None else torch.from_numpy(R).to(dev)
        bd = torch.from_numpy(b).to(dev)
        layers.append(dict(w=p, x=xd, y=yd, n=n, h=h, wd=wd, bias=bd, flags=alcs.ALCS_RELU, residual=rd, stride=s))
        keep.append((W, M, X, b, R, g, s, yd))
    for graph in (0, alcs.ALCS_STACK_GRAPH):
        st = alcs.alcs_stack_create(layers, graph)
        stream = torch.cuda.Stream()
        for _ in range(2):
            for k in keep:
                k[7].fill_(float("nan"))
            torch.cuda.synchronize()
            alcs.alcs_stack_run(st, stream)
            stream.synchronize()
            for W, M, X, b, R, g, s, yd in keep:
                Yref, A = oracle.conv1x1_ex(W, M, X, b, R, True, g, s, want_scale=True)
                assert_parity(yd.cpu().numpy(), Yref, A, "f32")
        alcs.alcs_stack_destroy(st)


@pytest.mark.parametrize("graph", [False, True])
def test_stack_tuned_in_context_stays_correct(alcs, graph):
    """alcs_stack_tune swaps launch configurations (and, at batch 1, kernels) while timing the whole stack:
    afterwards every layer must still match the oracle, the reported configurations must be the ones a
    fresh stack resolves to, and the times must be positive."""
    import torch
    dev = torch.device("cuda:0")
    specs = [(1, 64, 64, 14, 14, 4, 1, False), (1, 64, 96, 14, 14, 4, 1, True), (1, 96, 48, 14, 14, 4, 2, False), (1, 48, 40, 7, 7, 4, 1, False)]
    layers, keep = [], []
    stream = torch.cuda.Stream()
    for i, (n, cin, cout, h, wd, g, s, with_res) in enumerate(specs):
        W, M, X, b, R = _case(1200 + i, n, cin, cout, h, wd, g, 0.4, s)
        if not with_res:
            R = None
        p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
        oh, ow = -(-h // s), -(-wd // s)
        xd = torch.from_numpy(X).to(dev)
        yd = torch.full((n, cout, oh * ow), float("nan"), device=dev)
        rd = None if R is None else torch.from_numpy(R).to(dev)
        bd = torch.from_numpy(b).to(dev)
        if i == 0:      # one layer with finalists of its own tuning run, the others from the cost model
            with torch.cuda.stream(stream):
                alcs.alcs_spconv1x1_tune(p, xd, yd, n, h, wd, bd, alcs.ALCS_RELU, stream)
        layers.append(dict(w=p, x=xd, y=yd, n=n, h=h, wd=wd, bias=bd, flags=alcs.ALCS_RELU, residual=rd, stride=s))
        keep.append((W, M, X, b, R, g, s, yd))
    st = alcs.alcs_stack_create(layers, alcs.ALCS_STACK_GRAPH if graph else 0)
    with torch.cuda.stream(stream):
        before, after = alcs.alcs_stack_tune(st, 2, stream)
    assert before > 0 and after > 0
    cfgs = [alcs.alcs_stack_layer_cfg(st, i) for i in range(len(layers))]
    assert all(c["pixels_per_lane"] > 0 for c in cfgs)
    assert all(c["math_mode"] != 3 for c, sp in zip(cfgs, specs) if sp[6] > 1 or sp[7])   # (that kernel takes neither)
    for k in keep:
        k[7].fill_(float("nan"))
    torch.cuda.synchronize()
    alcs.alcs_stack_run(st, stream)
    stream.synchronize()
    for W, M, X, b, R, g, s, yd in keep:
        Yref, A = oracle.conv1x1_ex(W, M, X, b, R, True, g, s, want_scale=True)
        assert_parity(yd.cpu().numpy(), Yref, A, "f32")
    alcs.alcs_stack_destroy(st)
    st2 = alcs.alcs_stack_create(layers, 0)     # the packed matrices remember what the tuning chose
    assert [alcs.alcs_stack_layer_cfg(st2, i) for i in range(len(layers))] == cfgs
    alcs.alcs_stack_destroy(st2)
    empty = alcs.alcs_stack_create([], 0)
    with pytest.raises(alcs.AlcsError):
        alcs.alcs_stack_layer_cfg(empty, 0)
    assert alcs.alcs_stack_tune(empty, 1, stream)[1] >= 0
    alcs.alcs_stack_destroy(empty)


def test_argument_errors(alcs):
    import torch
    dev = torch.device("cuda:0")
    W, M, X, b, R = _case(5, 1, 8, 8, 4, 4, 4, 0.5, 2)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    xd = torch.from_numpy(X).to(dev)
    yd = torch.empty((1, 8, 4), device=dev)
    st = torch.cuda.current_stream()
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1_ex(p, xd, yd, 1, 4, 4, 0, None, None, 0, st)
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1_ex(p, xd, yd, 1, 4, 4, 2, None, yd, 0, st)          # residual overlaps y
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1_ex(p, xd, yd, 1, 4, 4, 2, None, None, 0, st, dict(math_mode=3))   # the small-problem kernel takes neither
    assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED
