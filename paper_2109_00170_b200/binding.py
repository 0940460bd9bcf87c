"""Thin ctypes binding of libalcs.so: argument marshalling only, same names as the C ABI
(include/alcs.h).  Every step of the convolution runs in the library's CUDA kernels; there is no
Python or CPU fallback, and loading fails loudly if the shared object has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libalcs.so")

ALCS_OK = 0
ALCS_ERR_INVALID_ARG, ALCS_ERR_SHAPE, ALCS_ERR_UNSUPPORTED, ALCS_ERR_ALLOC = -1, -2, -3, -4
ALCS_ERR_CUDA, ALCS_ERR_CORRUPT, ALCS_ERR_STATE, ALCS_ERR_TOO_LARGE = -5, -6, -7, -8
ALCS_NOALLOC_SCRATCH_BYTES = 16 << 20
ALCS_F32, ALCS_F16, ALCS_BF16 = 0, 1, 2
ALCS_RELU, ALCS_Y_F32 = 1, 2
ALCS_STACK_GRAPH = 1

# every symbol include/alcs.h declares
EXPORTS = ["alcs_strerror", "alcs_last_cuda_error", "alcs_version", "alcs_pack", "alcs_unpack",
           "alcs_packed_view", "alcs_packed_serialize", "alcs_packed_deserialize",
           "alcs_packed_upload", "alcs_packed_status", "alcs_packed_free", "alcs_schedule_selfcheck",
           "alcs_variant_count", "alcs_variant_get",
           "alcs_spconv1x1", "alcs_spconv1x1_cfg", "alcs_spconv1x1_ex",
           "alcs_spconv1x1_plan", "alcs_spconv1x1_tune", "alcs_spconv1x1_set_cfg", "alcs_spconv1x1_host_workspace",
           "alcs_spconv1x1_host", "alcs_spconv1x1_noalloc", "alcs_spconv2d", "alcs_spconv2d_cfg", "alcs_spconv2d_plan", "alcs_layer_latency", "alcs_network_latency",
           "alcs_project_bisection", "alcs_probe_fma_peak", "alcs_probe_lds", "alcs_probe_segment_loop",
           "alcs_stack_create", "alcs_stack_run", "alcs_stack_destroy", "alcs_stack_tune", "alcs_stack_layer_cfg"]


class AlcsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().alcs_strerror(status).decode()
        if status == ALCS_ERR_CUDA:
            msg += " [" + lib().alcs_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {msg}")


class LaunchCfg(C.Structure):
    _fields_ = [(k, C.c_int) for k in ("pixels_per_lane", "rows_per_warp", "warps",
                                       "chunk_channels", "stages", "row_groups", "min_blocks", "copy_mode",
                                       "producer_warps", "math_mode", "consumer_groups", "split_rows")]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class Conv2dCfg(C.Structure):
    _fields_ = [(k, C.c_int) for k in ("positions_per_lane", "strip_rows", "row_groups", "position_tiles",
                                       "warps_per_tile", "smem_bytes", "chunk_channels", "images_per_item")]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class LatencyTable(C.Structure):
    _fields_ = [("n_knots", C.c_int), ("k", C.POINTER(C.c_int64)), ("t", C.POINTER(C.c_double))]


class ProjectionResult(C.Structure):
    _fields_ = [("n_keep", C.c_int64), ("n0", C.c_int64), ("n1", C.c_int64), ("n_groups", C.c_int64),
                ("iters", C.c_int), ("latency", C.c_double)]


class ProbeResult(C.Structure):
    _fields_ = [("ms", C.c_double), ("tflops", C.c_double), ("frac_of_fp32_peak", C.c_double),
                ("registers", C.c_int), ("spill_bytes", C.c_int)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class Layer(C.Structure):
    _fields_ = [("w", C.c_void_p), ("x", C.c_void_p), ("y", C.c_void_p), ("n", C.c_int),
                ("h", C.c_int), ("wd", C.c_int), ("bias", C.c_void_p), ("flags", C.c_uint),
                ("residual", C.c_void_p), ("stride", C.c_int)]


_lib = None


def lib():
    """Load libalcs.so once.  Raises if it is missing: there is nothing to fall back to."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2109_00170_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, ip, u, i, sz = C.c_void_p, C.POINTER(C.c_int), C.c_uint, C.c_int, C.c_size_t
    L.alcs_strerror.restype = C.c_char_p
    L.alcs_strerror.argtypes = [i]
    L.alcs_last_cuda_error.restype = C.c_char_p
    L.alcs_version.restype = i
    L.alcs_pack.argtypes = [vp, vp, i, i, i, i, C.POINTER(vp)]
    L.alcs_unpack.argtypes = [vp, vp, vp]
    L.alcs_packed_view.argtypes = [vp, ip, ip, ip, ip, ip, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]
    L.alcs_packed_serialize.argtypes = [vp, vp, C.POINTER(sz)]
    L.alcs_packed_deserialize.argtypes = [vp, sz, C.POINTER(vp)]
    L.alcs_packed_upload.argtypes = [vp, i, vp]
    L.alcs_packed_status.argtypes = [vp, ip]
    L.alcs_packed_free.argtypes = [vp]
    L.alcs_packed_free.restype = None
    L.alcs_schedule_selfcheck.argtypes = [vp, i, i, i, i, C.POINTER(C.c_int64)]
    L.alcs_variant_count.restype = i
    L.alcs_variant_get.argtypes = [i, ip, ip, C.POINTER(LaunchCfg)]
    L.alcs_spconv1x1.argtypes = [vp, vp, vp, i, i, i, vp, u, vp]
    L.alcs_spconv1x1_cfg.argtypes = [vp, vp, vp, i, i, i, vp, u, C.POINTER(LaunchCfg), vp]
    L.alcs_spconv1x1_ex.argtypes = [vp, vp, vp, i, i, i, i, vp, vp, u, C.POINTER(LaunchCfg), vp]
    L.alcs_spconv1x1_plan.argtypes = [vp, i, i, i, u, C.POINTER(LaunchCfg)]
    L.alcs_spconv1x1_tune.argtypes = [vp, vp, vp, i, i, i, vp, u, vp, C.POINTER(LaunchCfg)]
    L.alcs_spconv1x1_set_cfg.argtypes = [vp, i, i, i, u, C.POINTER(LaunchCfg)]
    L.alcs_spconv1x1_host_workspace.argtypes = [vp, i, i, i, u]
    L.alcs_spconv1x1_host_workspace.restype = sz
    L.alcs_spconv1x1_host.argtypes = [vp, vp, vp, i, i, i, vp, u, vp, sz, vp]
    L.alcs_spconv1x1_noalloc.argtypes = [vp, vp, vp, i, i, i, vp, u, vp]
    L.alcs_spconv2d.argtypes = [vp, vp, vp] + [i] * 8 + [vp, u, vp]
    L.alcs_spconv2d_cfg.argtypes = [vp, vp, vp] + [i] * 8 + [vp, u, C.POINTER(Conv2dCfg), vp]
    L.alcs_spconv2d_plan.argtypes = [vp] + [i] * 8 + [C.POINTER(Conv2dCfg)]
    L.alcs_layer_latency.argtypes = [C.POINTER(LatencyTable), C.c_int64, C.POINTER(C.c_double)]
    L.alcs_network_latency.argtypes = [C.c_double, C.POINTER(LatencyTable), i, C.POINTER(C.c_int64), C.POINTER(C.c_double)]
    L.alcs_project_bisection.argtypes = [C.POINTER(vp), ip, ip, i, i, C.POINTER(LatencyTable), C.c_double, C.c_double,
                                         C.c_double, vp, C.POINTER(vp), C.POINTER(C.c_int64),
                                         C.POINTER(ProjectionResult), vp]
    L.alcs_probe_fma_peak.argtypes = [i, C.POINTER(ProbeResult), vp]
    L.alcs_probe_lds.argtypes = [i, i, C.POINTER(C.c_double), vp]
    L.alcs_probe_segment_loop.argtypes = [i, i, i, i, i, i, C.POINTER(ProbeResult), vp]
    L.alcs_stack_create.argtypes = [C.POINTER(Layer), i, u, C.POINTER(vp)]
    L.alcs_stack_run.argtypes = [vp, vp]
    L.alcs_stack_destroy.argtypes = [vp]
    L.alcs_stack_tune.argtypes = [vp, i, vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.alcs_stack_layer_cfg.argtypes = [vp, i, C.POINTER(LaunchCfg)]
    for name in EXPORTS:
        f = getattr(L, name)
        if f.restype is C.c_int and name not in ("alcs_version",):
            f.restype = i
    _lib = L
    return L


def _check(status: int, where: str):
    if status != ALCS_OK:
        raise AlcsError(status, where)


def _addr(t) -> Optional[int]:
    """Address of a torch tensor, a numpy array, an int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    raise TypeError(type(t))


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None     # torch.cuda.Stream


def _cfg(cfg) -> Optional[LaunchCfg]:
    if cfg is None or isinstance(cfg, LaunchCfg):
        return cfg
    return LaunchCfg(**cfg)


class Packed:
    """Owner of one alcs_packed object."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    @property
    def handle(self):
        if not self._h:
            raise AlcsError(ALCS_ERR_STATE, "Packed (freed)")
        return self._h

    def free(self):
        if self._h:
            lib().alcs_packed_free(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def alcs_pack(w: np.ndarray, block_mask: np.ndarray, g: int, bf16: bool = False) -> Packed:
    """w: [cout, cin] float32 or float16 (host), or, with bf16=True, uint16 holding bfloat16 bit patterns;
    block_mask: [ceil(cout/g), cin] uint8."""
    if bf16:
        if w.dtype != np.uint16:
            raise TypeError("bfloat16 weights are passed as uint16 bit patterns")
        dt = ALCS_BF16
    elif w.dtype == np.float32:
        dt = ALCS_F32
    elif w.dtype == np.float16:
        dt = ALCS_F16
    else:
        raise TypeError("weights must be float32 or float16")
    w = np.ascontiguousarray(w)
    block_mask = np.ascontiguousarray(block_mask, dtype=np.uint8)
    cout, cin = w.shape
    if block_mask.shape != ((cout + max(g, 1) - 1) // max(g, 1), cin):
        raise ValueError("block_mask shape")
    out = C.c_void_p()
    _check(lib().alcs_pack(w.ctypes.data, block_mask.ctypes.data, cout, cin, g, dt, C.byref(out)), "alcs_pack")
    return Packed(out.value)


def alcs_packed_view(p: Packed):
    """Copies of the packed arrays: dict(cout, cin, g, dtype, nb, row_ptr, col_idx, vals)."""
    cout, cin, g, dt, nb = (C.c_int() for _ in range(5))
    rp, ci, va = C.c_void_p(), C.c_void_p(), C.c_void_p()
    _check(lib().alcs_packed_view(p.handle, cout, cin, g, dt, nb, C.byref(rp), C.byref(ci), C.byref(va)),
           "alcs_packed_view")
    rows = (cout.value + g.value - 1) // g.value
    npdt = {ALCS_F32: np.float32, ALCS_F16: np.float16, ALCS_BF16: np.uint16}[dt.value]     # bfloat16: bit patterns

    def arr(ptr, n, t):
        if n == 0:
            return np.zeros(0, dtype=t)
        return np.ctypeslib.as_array(C.cast(ptr, C.POINTER(C.c_uint8)), shape=(n * np.dtype(t).itemsize,)).view(t).copy()

    return dict(cout=cout.value, cin=cin.value, g=g.value, dtype=dt.value, nb=nb.value,
                row_ptr=arr(rp, rows + 1, np.int32), col_idx=arr(ci, nb.value, np.int32),
                vals=arr(va, nb.value * g.value, npdt))


def alcs_unpack(p: Packed):
    v = alcs_packed_view(p)
    npdt = {ALCS_F32: np.float32, ALCS_F16: np.float16, ALCS_BF16: np.uint16}[v["dtype"]]
    rows = (v["cout"] + v["g"] - 1) // v["g"]
    w = np.empty((v["cout"], v["cin"]), dtype=npdt)
    m = np.empty((rows, v["cin"]), dtype=np.uint8)
    _check(lib().alcs_unpack(p.handle, w.ctypes.data, m.ctypes.data), "alcs_unpack")
    return w, m


def alcs_packed_serialize(p: Packed) -> bytes:
    n = C.c_size_t(0)
    _check(lib().alcs_packed_serialize(p.handle, None, C.byref(n)), "alcs_packed_serialize")
    buf = (C.c_uint8 * n.value)()
    _check(lib().alcs_packed_serialize(p.handle, buf, C.byref(n)), "alcs_packed_serialize")
    return bytes(buf)


def alcs_packed_deserialize(blob: bytes) -> Packed:
    out = C.c_void_p()
    buf = (C.c_uint8 * len(blob)).from_buffer_copy(blob) if len(blob) else (C.c_uint8 * 1)()
    _check(lib().alcs_packed_deserialize(buf, len(blob), C.byref(out)), "alcs_packed_deserialize")
    return Packed(out.value)


def alcs_packed_upload(p: Packed, device: int = 0, stream=None) -> Packed:
    _check(lib().alcs_packed_upload(p.handle, device, _stream(stream)), "alcs_packed_upload")
    return p


def alcs_packed_status(p: Packed) -> int:
    """Device error word of p: 0 unless a kernel gave up a bounded wait."""
    code = C.c_int(0)
    _check(lib().alcs_packed_status(p.handle, code), "alcs_packed_status")
    return code.value


def alcs_packed_free(p: Packed):
    p.free()


def alcs_schedule_selfcheck(p: Packed, chunk_channels: int, row_groups: int, warps: int, slots: int) -> dict:
    """Host-only check of the balanced launch schedule against the storage format."""
    st = (C.c_int64 * 8)()
    _check(lib().alcs_schedule_selfcheck(p.handle, chunk_channels, row_groups, warps, slots, st), "alcs_schedule_selfcheck")
    return dict(row_groups=st[0], max_sched=st[1], min_sched=st[2], pairs=st[3], nb=st[4], max_rows=st[5], min_rows=st[6], secondary_units=st[7])


def alcs_variant_count() -> int:
    return int(lib().alcs_variant_count())


def alcs_variant_get(index: int) -> dict:
    """dict(dtype, g, pixels_per_lane, rows_per_warp, warps, min_blocks, ...) of one variant."""
    dt, g, c = C.c_int(), C.c_int(), LaunchCfg()
    _check(lib().alcs_variant_get(index, dt, g, C.byref(c)), "alcs_variant_get")
    return dict(dtype=dt.value, g=g.value, **c.as_dict())


def alcs_spconv1x1(w: Packed, x, y, n: int, h: int, wd: int, bias=None, flags: int = 0, stream=None,
                   cfg=None):
    """x, y, bias: device tensors (anything with data_ptr()) or raw device addresses."""
    c = _cfg(cfg)
    if c is None:
        st = lib().alcs_spconv1x1(w.handle, _addr(x), _addr(y), n, h, wd, _addr(bias), flags, _stream(stream))
    else:
        st = lib().alcs_spconv1x1_cfg(w.handle, _addr(x), _addr(y), n, h, wd, _addr(bias), flags,
                                      C.byref(c), _stream(stream))
    _check(st, "alcs_spconv1x1")


def alcs_spconv1x1_ex(w: Packed, x, y, n: int, h: int, wd: int, stride: int = 1, bias=None, residual=None,
                      flags: int = 0, stream=None, cfg=None):
    """Strided pointwise convolution with a residual operand added before the activation."""
    c = _cfg(cfg)
    _check(lib().alcs_spconv1x1_ex(w.handle, _addr(x), _addr(y), n, h, wd, stride, _addr(bias), _addr(residual), flags,
                                   C.byref(c) if c is not None else None, _stream(stream)), "alcs_spconv1x1_ex")


def alcs_spconv1x1_plan(w: Packed, n: int, h: int, wd: int, flags: int = 0) -> dict:
    c = LaunchCfg()
    _check(lib().alcs_spconv1x1_plan(w.handle, n, h, wd, flags, C.byref(c)), "alcs_spconv1x1_plan")
    return c.as_dict()


def alcs_spconv1x1_tune(w: Packed, x, y, n: int, h: int, wd: int, bias=None, flags: int = 0,
                        stream=None) -> dict:
    c = LaunchCfg()
    _check(lib().alcs_spconv1x1_tune(w.handle, _addr(x), _addr(y), n, h, wd, _addr(bias), flags,
                                     _stream(stream), C.byref(c)), "alcs_spconv1x1_tune")
    return c.as_dict()


def alcs_spconv1x1_set_cfg(w: Packed, n: int, h: int, wd: int, flags: int, cfg) -> None:
    """Use `cfg` (a dict or LaunchCfg, e.g. from a tuning cache) for later calls with this shape."""
    c = _cfg(cfg)
    _check(lib().alcs_spconv1x1_set_cfg(w.handle, n, h, wd, flags, C.byref(c)), "alcs_spconv1x1_set_cfg")


def alcs_spconv1x1_host_workspace(w: Packed, n: int, h: int, wd: int, flags: int = 0) -> int:
    return int(lib().alcs_spconv1x1_host_workspace(w.handle, n, h, wd, flags))


def alcs_spconv1x1_host(w: Packed, x_host, y_host, n: int, h: int, wd: int, bias_host=None,
                        flags: int = 0, workspace=None, workspace_bytes: int = 0, stream=None):
    """x_host / y_host / bias_host: host arrays (numpy, or pinned torch CPU tensors)."""
    _check(lib().alcs_spconv1x1_host(w.handle, _addr(x_host), _addr(y_host), n, h, wd, _addr(bias_host),
                                     flags, _addr(workspace), workspace_bytes, _stream(stream)),
           "alcs_spconv1x1_host")


def alcs_spconv1x1_noalloc(w: Packed, x, y, n: int, h: int, wd: int, bias=None, flags: int = 0, stream=None):
    """alcs_spconv1x1 for callers that must not allocate device memory: the shape must have been run
    once through alcs_spconv1x1 / tune / a stack before, and the repacked input (only needed when
    h*wd rows are not 16-byte multiples) has to fit ALCS_NOALLOC_SCRATCH_BYTES."""
    _check(lib().alcs_spconv1x1_noalloc(w.handle, _addr(x), _addr(y), n, h, wd, _addr(bias), flags, _stream(stream)),
           "alcs_spconv1x1_noalloc")


def alcs_spconv2d(w: Packed, x, y, n: int, cin: int, h: int, wd: int, kh: int, kw: int, stride: int = 1,
                  pad: int = 0, bias=None, flags: int = 0, stream=None, cfg=None):
    """General k x k convolution: x [n,cin,h,wd], y [n,cout,oh,ow] fp32 device tensors; w packed from
    the flattened filters [cout, cin*kh*kw].  cfg: optional dict of alcs_conv2d_cfg fields to fix."""
    if cfg is None:
        _check(lib().alcs_spconv2d(w.handle, _addr(x), _addr(y), n, cin, h, wd, kh, kw, stride, pad, _addr(bias),
                                   flags, _stream(stream)), "alcs_spconv2d")
    else:
        c = Conv2dCfg(**{k: int(v) for k, v in cfg.items()})
        _check(lib().alcs_spconv2d_cfg(w.handle, _addr(x), _addr(y), n, cin, h, wd, kh, kw, stride, pad, _addr(bias),
                                       flags, C.byref(c), _stream(stream)), "alcs_spconv2d_cfg")


def alcs_spconv2d_plan(w: Packed, n: int, cin: int, h: int, wd: int, kh: int, kw: int, stride: int = 1,
                       pad: int = 0) -> dict:
    out = Conv2dCfg()
    _check(lib().alcs_spconv2d_plan(w.handle, n, cin, h, wd, kh, kw, stride, pad, C.byref(out)),
           "alcs_spconv2d_plan")
    return out.as_dict()


def _tables(tables):
    """[(k, t), ...] -> (ctypes array of LatencyTable, keep-alive list)."""
    arr = (LatencyTable * len(tables))()
    keep = []
    for j, (k, t) in enumerate(tables):
        ka = np.ascontiguousarray(k, dtype=np.int64)
        ta = np.ascontiguousarray(t, dtype=np.float64)
        if ka.shape != ta.shape or ka.ndim != 1:
            raise ValueError("latency table: k and t must be 1-D of equal length")
        keep += [ka, ta]
        arr[j].n_knots = ka.size
        arr[j].k = ka.ctypes.data_as(C.POINTER(C.c_int64))
        arr[j].t = ta.ctypes.data_as(C.POINTER(C.c_double))
    return arr, keep


def alcs_layer_latency(k, t, s: int) -> float:
    arr, keep = _tables([(k, t)])
    out = C.c_double()
    _check(lib().alcs_layer_latency(arr, int(s), C.byref(out)), "alcs_layer_latency")
    return out.value


def alcs_network_latency(tau: float, tables, s) -> float:
    arr, keep = _tables(tables)
    sa = np.ascontiguousarray(s, dtype=np.int64)
    out = C.c_double()
    _check(lib().alcs_network_latency(float(tau), arr, len(tables), sa.ctypes.data_as(C.POINTER(C.c_int64)),
                                      C.byref(out)), "alcs_network_latency")
    return out.value


def alcs_project_bisection(u_tilde, g: int, tables, tau: float, t_budget: float, eps: float, mask_out,
                           u_out=None, stream=None) -> dict:
    """u_tilde: list of fp32 device tensors [cout_l, cols_l]; mask_out: uint8 device tensor with one
    byte per group, layer after layer; u_out: optional list of output tensors (entries may be None)."""
    n = len(u_tilde)
    ptrs = (C.c_void_p * n)(*[_addr(t) for t in u_tilde])
    cout = (C.c_int * n)(*[int(t.shape[0]) for t in u_tilde])
    cols = (C.c_int * n)(*[int(t.shape[1]) for t in u_tilde])
    arr, keep = _tables(tables)
    outs = None
    if u_out is not None:
        outs = (C.c_void_p * n)(*[_addr(t) for t in u_out])
    kept = (C.c_int64 * n)()
    res = ProjectionResult()
    _check(lib().alcs_project_bisection(ptrs, cout, cols, n, g, arr, float(tau), float(t_budget), float(eps),
                                        _addr(mask_out), outs, kept, C.byref(res), _stream(stream)),
           "alcs_project_bisection")
    return {"n_keep": res.n_keep, "n0": res.n0, "n1": res.n1, "n_groups": res.n_groups, "iters": res.iters,
            "latency": res.latency, "kept_per_layer": list(kept)}


def alcs_probe_fma_peak(packed: bool = True, stream=None) -> dict:
    """Measured fp32 FMA rate of the current device from register operands."""
    r = ProbeResult()
    _check(lib().alcs_probe_fma_peak(1 if packed else 0, C.byref(r), _stream(stream)), "alcs_probe_fma_peak")
    return r.as_dict()


def alcs_probe_lds(bytes_per_lane: int, uniform: bool, stream=None) -> float:
    """Load/store-pipe cycles per warp-wide shared-memory load instruction."""
    v = C.c_double()
    _check(lib().alcs_probe_lds(bytes_per_lane, 1 if uniform else 0, C.byref(v), _stream(stream)), "alcs_probe_lds")
    return v.value


def alcs_probe_segment_loop(g: int, pixels_per_lane: int, rows_per_warp: int, warps: int, deep: bool,
                            pairs_per_segment: int, stream=None) -> dict:
    """The kernel's segment loop on shared-memory-resident synthetic segments."""
    r = ProbeResult()
    _check(lib().alcs_probe_segment_loop(g, pixels_per_lane, rows_per_warp, warps, 1 if deep else 0,
                                         pairs_per_segment, C.byref(r), _stream(stream)), "alcs_probe_segment_loop")
    return r.as_dict()


class Stack:
    """Owner of one alcs_stack object."""

    def __init__(self, handle, keep):
        self._h = C.c_void_p(handle)
        self._keep = keep      # keeps the Packed objects and tensors alive

    @property
    def handle(self):
        if not self._h:
            raise AlcsError(ALCS_ERR_STATE, "Stack (destroyed)")
        return self._h

    def destroy(self):
        if self._h:
            lib().alcs_stack_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def alcs_stack_create(layers: Sequence[dict], stack_flags: int = 0) -> Stack:
    """layers: dicts with keys w (Packed), x, y, n, h, wd, bias (optional), flags (optional)."""
    arr = (Layer * max(1, len(layers)))()
    for k, L in enumerate(layers):
        arr[k] = Layer(L["w"].handle, _addr(L["x"]), _addr(L["y"]), L["n"], L["h"], L["wd"],
                       _addr(L.get("bias")), L.get("flags", 0), _addr(L.get("residual")), L.get("stride", 1))
    out = C.c_void_p()
    _check(lib().alcs_stack_create(arr, len(layers), stack_flags, C.byref(out)), "alcs_stack_create")
    return Stack(out.value, list(layers))


def alcs_stack_run(s: Stack, stream=None):
    _check(lib().alcs_stack_run(s.handle, _stream(stream)), "alcs_stack_run")


def alcs_stack_tune(s: Stack, passes: int = 0, stream=None):
    """Choose the layers' launch configurations in the context of the whole stack; returns
    (microseconds per pass before, after)."""
    before, after = C.c_double(0.0), C.c_double(0.0)
    _check(lib().alcs_stack_tune(s.handle, passes, _stream(stream), C.byref(before), C.byref(after)), "alcs_stack_tune")
    return before.value, after.value


def alcs_stack_layer_cfg(s: Stack, layer: int) -> dict:
    c = LaunchCfg()
    _check(lib().alcs_stack_layer_cfg(s.handle, layer, C.byref(c)), "alcs_stack_layer_cfg")
    return c.as_dict()


def alcs_stack_destroy(s: Stack):
    s.destroy()
