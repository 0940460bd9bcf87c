"""Helpers of the GPU parity tests: run the CUDA path through the C ABI and compare with the
oracle.  Tolerances (stated here once):

  fp32:                 |Y - Yref| <= 1e-5 * A     element-wise
  fp16 in / fp32 acc:   |Y - Yref| <= 2e-3 * A     element-wise
  and normwise          max|Y - Yref| <= tol * max|Yref|

where A = |bias| + sum_c |Wm||X| is the oracle's condition scale (the forward-error scale of a dot
product; ReLU is 1-Lipschitz so the bound survives it).  The plain relative error on outputs that
are not cancelled to nearly zero is reported by the benchmark, not asserted.
"""
from __future__ import annotations

import numpy as np

import oracle

TOL = {"f32": 1e-5, "f16": 2e-3}


def torch_dev():
    import torch
    return torch, torch.device("cuda:0")


def run_gpu(alcs, W, M, X, bias, relu, g, cfg=None, y_f32=False, h=None, wd=None, packed=None,
            tune=False):
    """One alcs_spconv1x1 call on cuda:0; returns Y as a numpy array [n, cout, hw]."""
    torch, dev = torch_dev()
    n, cin, hw = X.shape
    cout = W.shape[0]
    if h is None:
        h, wd = hw, 1
    assert h * wd == hw
    p = packed or alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    xd = torch.from_numpy(np.ascontiguousarray(X)).to(dev)
    ydt = torch.float32 if (W.dtype == np.float32 or y_f32) else torch.float16
    yd = torch.full((n, cout, hw), float("nan"), dtype=ydt, device=dev)
    bd = None if bias is None else torch.from_numpy(bias).to(dev)
    flags = (alcs.ALCS_RELU if relu else 0) | (alcs.ALCS_Y_F32 if y_f32 else 0)
    if tune:
        alcs.alcs_spconv1x1_tune(p, xd, yd, n, h, wd, bd, flags, torch.cuda.current_stream())
        yd.fill_(float("nan"))
    alcs.alcs_spconv1x1(p, xd, yd, n, h, wd, bd, flags, torch.cuda.current_stream(), cfg)
    torch.cuda.synchronize()
    return yd.cpu().numpy()


def assert_parity(Y, Yref, A, kind, exact=False):
    assert Y.shape == Yref.shape
    assert np.isfinite(Y).all(), "non-finite or unwritten output"
    d = np.abs(Y.astype(np.float64) - Yref)
    if exact:
        assert d.max() == 0.0, f"expected exact equality, max diff {d.max()}"
        return 0.0
    tol = TOL[kind]
    bad = d > tol * A + 1e-300
    assert not bad.any(), (f"{int(bad.sum())} of {bad.size} outputs beyond {tol}*A; worst ratio "
                           f"{(d / np.maximum(A, 1e-300)).max():.3e}")
    if np.abs(Yref).max() > 0:
        assert d.max() <= tol * np.abs(Yref).max()
    return float((d / np.maximum(A, 1e-300)).max())


def check_layer(alcs, W, M, X, bias, relu, g, cfg=None, y_f32=False, exact=False, **kw):
    kind = "f32" if W.dtype == np.float32 else "f16"
    Y = run_gpu(alcs, W, M, X, bias, relu, g, cfg=cfg, y_f32=y_f32, **kw)
    Yref, A = oracle.conv1x1(W, M, X, bias, relu, g, want_scale=True)
    return assert_parity(Y, Yref, A, kind, exact=exact)
