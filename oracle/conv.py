"""ctypes front end of the C oracle (oracle/alcs_oracle.c).  Test infrastructure only.

The convolution definition it evaluates is the paper's Section 3.2.2 formula over
mask-applied weights, in double precision, plus bias and ReLU: conv1x1 at k_h = k_w = 1,
conv2d for a general kernel with stride and zero padding.
"""
from __future__ import annotations

import ctypes as C
import functools

import numpy as np

from . import build as _build


@functools.lru_cache(maxsize=None)
def _lib(mutant: int = 0, build_dir: str | None = None):
    lib = C.CDLL(_build.build(mutant, build_dir))
    lib.oracle_conv1x1.restype = C.c_int
    lib.oracle_conv1x1.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                   C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_long,
                                   C.c_void_p, C.c_void_p]
    lib.oracle_conv1x1_points.restype = C.c_int
    lib.oracle_conv1x1_points.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                          C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_long,
                                          C.c_void_p, C.c_long, C.c_void_p, C.c_void_p]
    lib.oracle_conv1x1_ex.restype = C.c_int
    lib.oracle_conv1x1_ex.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p] + \
                                     [C.c_int] * 9 + [C.c_void_p, C.c_void_p]
    lib.oracle_conv2d.restype = C.c_int
    lib.oracle_conv2d.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                  C.c_int, C.c_int] + [C.c_int] * 9 + [C.c_void_p, C.c_void_p]
    lib.oracle_conv2d_points.restype = C.c_int
    lib.oracle_conv2d_points.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                         C.c_int, C.c_int] + [C.c_int] * 9 + [
                                             C.c_void_p, C.c_long, C.c_void_p, C.c_void_p]
    lib.oracle_conv2d_out_size.restype = C.c_int
    lib.oracle_conv2d_out_size.argtypes = [C.c_int] * 4
    lib.oracle_num_threads.restype = C.c_int
    lib.oracle_mutant.restype = C.c_int
    assert lib.oracle_mutant() == mutant
    return lib


def bf16_decode(bits):
    """bfloat16 bit patterns (uint16) -> the float32 values they denote, exactly: a bfloat16 number is the
    float32 number whose upper 16 bits are its bits and whose lower 16 bits are zero.  The oracle takes
    bfloat16 operands as these float32 arrays (it works in double precision either way)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def num_threads() -> int:
    """Threads the oracle's OpenMP loops will use."""
    return int(_lib().oracle_num_threads())


def _prep(W, mask, X, bias, g):
    if W.dtype not in (np.float32, np.float16) or X.dtype != W.dtype:
        raise TypeError("W and X must both be float32 or both float16")
    W = np.ascontiguousarray(W)
    X = np.ascontiguousarray(X)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    cout, cin = W.shape
    n, cin2, hw = X.shape
    rows = (cout + g - 1) // g
    if cin2 != cin or mask.shape != (rows, cin):
        raise ValueError("shape mismatch")
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        if bias.shape != (cout,):
            raise ValueError("bias shape")
    return W, mask, X, bias, n, cin, cout, hw


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def conv1x1(W, mask, X, bias=None, relu=False, g=4, want_scale=False, mutant=0, build_dir=None):
    """Y[n,cout,hw] (float64) = relu?(Wm X + bias), Wm = W with dropped blocks set to zero.

    With want_scale also returns A = |bias| + sum |Wm||X| (float64, same shape).
    """
    W, mask, X, bias, n, cin, cout, hw = _prep(W, mask, X, bias, g)
    Y = np.empty((n, cout, hw), dtype=np.float64)
    A = np.empty((n, cout, hw), dtype=np.float64) if want_scale else None
    rc = _lib(mutant, build_dir).oracle_conv1x1(
        _ptr(W), _ptr(mask), g, _ptr(X), _ptr(bias), int(bool(relu)),
        int(W.dtype == np.float16), n, cin, cout, hw, _ptr(Y), _ptr(A))
    if rc != 0:
        raise RuntimeError(f"oracle_conv1x1 failed: {rc}")
    return (Y, A) if want_scale else Y


def conv1x1_ex(W, mask, X, bias=None, residual=None, relu=False, g=4, stride=1, want_scale=False, mutant=0,
               build_dir=None):
    """Strided pointwise convolution with a residual: X [n,cin,h,wd], residual [n,cout,oh*ow] (float32 or
    float16) or None; Y[n,cout,oh*ow] (float64) = relu?(Wm X[:, :, ::s, ::s] + bias + residual).
    With want_scale also returns A = |bias| + |residual| + sum |Wm||X|."""
    if X.ndim != 4:
        raise ValueError("X must be [n, cin, h, wd]")
    n, cin, h, wd = X.shape
    W, mask, _, bias, n, cin, cout, _ = _prep(W, mask, X.reshape(n, cin, h * wd), bias, g)
    X = np.ascontiguousarray(X)
    oh, ow = -(-h // stride), -(-wd // stride)
    if residual is not None:
        if residual.dtype not in (np.float32, np.float16) or residual.shape != (n, cout, oh * ow):
            raise ValueError("residual must be float32/float16 [n, cout, oh*ow]")
        residual = np.ascontiguousarray(residual)
    Y = np.empty((n, cout, oh * ow), dtype=np.float64)
    A = np.empty((n, cout, oh * ow), dtype=np.float64) if want_scale else None
    rc = _lib(mutant, build_dir).oracle_conv1x1_ex(
        _ptr(W), _ptr(mask), g, _ptr(X), _ptr(bias), _ptr(residual),
        int(residual is not None and residual.dtype == np.float16), int(bool(relu)),
        int(W.dtype == np.float16), n, cin, cout, h, wd, stride, _ptr(Y), _ptr(A))
    if rc != 0:
        raise RuntimeError(f"oracle_conv1x1_ex failed: {rc}")
    return (Y, A) if want_scale else Y


def conv1x1_points(W, mask, X, flat_idx, bias=None, relu=False, g=4):
    """The same quantities at selected flat indices of Y[n,cout,hw]; returns (values, scale)."""
    W, mask, X, bias, n, cin, cout, hw = _prep(W, mask, X, bias, g)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    out = np.empty(idx.shape, dtype=np.float64)
    mag = np.empty(idx.shape, dtype=np.float64)
    rc = _lib().oracle_conv1x1_points(
        _ptr(W), _ptr(mask), g, _ptr(X), _ptr(bias), int(bool(relu)),
        int(W.dtype == np.float16), n, cin, cout, hw, _ptr(idx), idx.size, _ptr(out), _ptr(mag))
    if rc != 0:
        raise RuntimeError(f"oracle_conv1x1_points failed: {rc}")
    return out, mag


def _prep2d(W, mask, X, bias, g, stride, pad):
    if W.dtype not in (np.float32, np.float16) or X.dtype != W.dtype:
        raise TypeError("W and X must both be float32 or both float16")
    W = np.ascontiguousarray(W)
    X = np.ascontiguousarray(X)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    cout, cin, kh, kw = W.shape
    n, cin2, h, wd = X.shape
    rows = (cout + g - 1) // g
    if cin2 != cin or mask.shape != (rows, cin * kh * kw):
        raise ValueError("shape mismatch")
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        if bias.shape != (cout,):
            raise ValueError("bias shape")
    oh = (h + 2 * pad - kh) // stride + 1
    ow = (wd + 2 * pad - kw) // stride + 1
    if stride < 1 or pad < 0 or h + 2 * pad < kh or wd + 2 * pad < kw:
        raise ValueError("geometry")
    return W, mask, X, bias, (n, cin, cout, h, wd, kh, kw, stride, pad), (oh, ow)


def conv2d(W, mask, X, bias=None, relu=False, g=4, stride=1, pad=0, want_scale=False, mutant=0,
           build_dir=None):
    """Y[n,cout,oh,ow] (float64) of the general kernel: W [cout,cin,kh,kw], block mask
    [ceil(cout/g), cin*kh*kw] over the flattened-filter columns (c*kh + r)*kw + s,
    X [n,cin,h,w], zero padding `pad`, stride `stride`.

    With want_scale also returns A = |bias| + sum |Wm||X| (float64, same shape).
    """
    W, mask, X, bias, geo, (oh, ow) = _prep2d(W, mask, X, bias, g, stride, pad)
    n, cout = geo[0], geo[2]
    Y = np.empty((n, cout, oh, ow), dtype=np.float64)
    A = np.empty((n, cout, oh, ow), dtype=np.float64) if want_scale else None
    rc = _lib(mutant, build_dir).oracle_conv2d(
        _ptr(W), _ptr(mask), g, _ptr(X), _ptr(bias), int(bool(relu)),
        int(W.dtype == np.float16), *geo, _ptr(Y), _ptr(A))
    if rc != 0:
        raise RuntimeError(f"oracle_conv2d failed: {rc}")
    return (Y, A) if want_scale else Y


def conv2d_points(W, mask, X, flat_idx, bias=None, relu=False, g=4, stride=1, pad=0):
    """The same quantities at selected flat indices of Y[n,cout,oh,ow]; returns (values, scale)."""
    W, mask, X, bias, geo, _ = _prep2d(W, mask, X, bias, g, stride, pad)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    out = np.empty(idx.shape, dtype=np.float64)
    mag = np.empty(idx.shape, dtype=np.float64)
    rc = _lib().oracle_conv2d_points(
        _ptr(W), _ptr(mask), g, _ptr(X), _ptr(bias), int(bool(relu)),
        int(W.dtype == np.float16), *geo, _ptr(idx), idx.size, _ptr(out), _ptr(mag))
    if rc != 0:
        raise RuntimeError(f"oracle_conv2d_points failed: {rc}")
    return out, mag
