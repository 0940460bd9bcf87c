"""Host-side library tests (no GPU): the packer against the storage-format oracle, bit for bit;
serialisation; error codes; and that libalcs.so exports every symbol include/alcs.h declares."""
import os
import re

import numpy as np
import pytest

from alcs_workloads import LayerSpec, config_layers, make_mask, make_weights, rng
from oracle import storage

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bits(a):
    return a.view(np.uint32 if a.dtype == np.float32 else np.uint16)


def _case(seed, cout, cin, g, density, dtype):
    rows = (cout + g - 1) // g
    W = rng.normal(seed, 1, cout * cin).reshape(cout, cin).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    return W, M


def test_library_exports_every_declared_symbol(alcs):
    hdr = open(os.path.join(ROOT, "include", "alcs.h")).read()
    declared = sorted(set(re.findall(r"ALCS_API [\w \*]+?\b(alcs_\w+)\(", hdr)))
    assert declared and sorted(alcs.EXPORTS) == declared
    L = alcs.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert L.alcs_version() == 2


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
@pytest.mark.parametrize("cout,cin,g,density", [
    (8, 7, 4, 0.5), (10, 9, 4, 0.3), (7, 5, 1, 0.5), (16, 16, 16, 0.7), (9, 4, 2, 0.5),
    (5, 3, 8, 0.9), (128, 64, 4, 0.3), (64, 32, 8, 0.0), (64, 32, 4, 1.0), (33, 65, 3, 0.4)])
def test_pack_matches_oracle_bit_exact(alcs, dtype, cout, cin, g, density):
    W, M = _case(cout * 131 + cin * 7 + g, cout, cin, g, density, dtype)
    p = alcs.alcs_pack(W, M, g)
    v = alcs.alcs_packed_view(p)
    counts, offs, vals = storage.pack(W, M, g)
    row_ptr, col_idx, flat = storage.flatten(counts, offs, vals, g, dtype)
    assert (v["cout"], v["cin"], v["g"], v["nb"]) == (cout, cin, g, int(M.sum()))
    assert np.array_equal(v["row_ptr"], row_ptr)
    assert np.array_equal(v["col_idx"], col_idx)
    assert np.array_equal(_bits(v["vals"]), _bits(flat))
    W2, M2 = alcs.alcs_unpack(p)
    Wo, Mo = storage.unpack(counts, offs, vals, cout, cin, g, dtype)
    assert np.array_equal(M2, M) and np.array_equal(Mo, M)
    assert np.array_equal(_bits(W2), _bits(Wo))
    p.free()


def test_pack_first_benchmark_layer(alcs):
    s = config_layers(0)[0]
    W, M = make_weights(s), make_mask(s)
    v = alcs.alcs_packed_view(alcs.alcs_pack(W, M, s.g))
    counts, offs, vals = storage.pack(W, M, s.g)
    row_ptr, col_idx, flat = storage.flatten(counts, offs, vals, s.g, np.float32)
    assert v["nb"] == 614
    assert np.array_equal(v["row_ptr"], row_ptr) and np.array_equal(v["col_idx"], col_idx)
    assert np.array_equal(_bits(v["vals"]), _bits(flat))


def test_paper_example_through_library(alcs):
    """Section 3.2.2 storage-format example (g = 2): count 3, offsets start 1, 3; values start
    (1,3), (2,1)."""
    W = np.zeros((2, 6), np.float32)
    W[:, 1], W[:, 3], W[:, 5] = [1, 3], [2, 1], [4, 2]
    M = np.array([[0, 1, 0, 1, 0, 1]], np.uint8)
    v = alcs.alcs_packed_view(alcs.alcs_pack(W, M, 2))
    assert list(v["row_ptr"]) == [0, 3]
    assert list(v["col_idx"][:2]) == [1, 3]
    assert list(v["vals"][:4]) == [1, 3, 2, 1]


def test_special_values_survive(alcs):
    W = np.array([[-0.0, 1e-45, np.inf, 5.0], [np.nan, 0.0, -np.inf, 6.0]], np.float32)
    M = np.array([[1, 1, 1, 0]], np.uint8)
    p = alcs.alcs_pack(W, M, 2)
    v = alcs.alcs_packed_view(p)
    assert np.array_equal(_bits(v["vals"]), _bits(W[:, :3].T.copy().reshape(-1)))
    W2, _ = alcs.alcs_unpack(p)
    assert np.array_equal(_bits(W2[:, :3]), _bits(W[:, :3])) and not _bits(W2[:, 3]).any()


@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_serialize_roundtrip_and_corruption(alcs, dtype):
    W, M = _case(5, 20, 13, 4, 0.4, dtype)
    p = alcs.alcs_pack(W, M, 4)
    blob = alcs.alcs_packed_serialize(p)
    q = alcs.alcs_packed_deserialize(blob)
    a, b = alcs.alcs_packed_view(p), alcs.alcs_packed_view(q)
    for k in ("row_ptr", "col_idx"):
        assert np.array_equal(a[k], b[k])
    assert np.array_equal(_bits(a["vals"]), _bits(b["vals"]))
    assert alcs.alcs_packed_serialize(q) == blob
    hdr = 32
    bad = []
    bad.append(blob[:-1])                                    # truncated
    bad.append(b"XXXX" + blob[4:])                           # magic
    bad.append(blob[:4] + (9).to_bytes(4, "little") + blob[8:])      # version
    rp = bytearray(blob); rp[hdr + 4:hdr + 8] = (10 ** 6).to_bytes(4, "little"); bad.append(bytes(rp))
    nrows = (20 + 3) // 4
    ci = bytearray(blob); off = hdr + (nrows + 1) * 4; ci[off:off + 4] = (13).to_bytes(4, "little"); bad.append(bytes(ci))
    if a["row_ptr"][1] >= 2:                                 # break the ascending order in row 0
        sw = bytearray(blob); sw[off:off + 4], sw[off + 4:off + 8] = blob[off + 4:off + 8], blob[off:off + 4]
        bad.append(bytes(sw))
    bad.append(b"")
    for x in bad:
        with pytest.raises(alcs.AlcsError) as e:
            alcs.alcs_packed_deserialize(x)
        assert e.value.status in (alcs.ALCS_ERR_CORRUPT, alcs.ALCS_ERR_INVALID_ARG)


def test_pack_error_codes(alcs):
    import ctypes as C
    L = alcs.lib()
    W = np.zeros((4, 4), np.float32)
    M = np.ones((1, 4), np.uint8)
    out = C.c_void_p()
    assert L.alcs_pack(None, M.ctypes.data, 4, 4, 4, 0, C.byref(out)) == alcs.ALCS_ERR_INVALID_ARG
    assert L.alcs_pack(W.ctypes.data, None, 4, 4, 4, 0, C.byref(out)) == alcs.ALCS_ERR_INVALID_ARG
    assert L.alcs_pack(W.ctypes.data, M.ctypes.data, 4, 4, 0, 0, C.byref(out)) == alcs.ALCS_ERR_INVALID_ARG
    assert L.alcs_pack(W.ctypes.data, M.ctypes.data, 4, 4, 65, 0, C.byref(out)) == alcs.ALCS_ERR_INVALID_ARG
    assert L.alcs_pack(W.ctypes.data, M.ctypes.data, 0, 4, 4, 0, C.byref(out)) == alcs.ALCS_ERR_SHAPE
    assert L.alcs_pack(W.ctypes.data, M.ctypes.data, 4, 4, 4, 7, C.byref(out)) == alcs.ALCS_ERR_UNSUPPORTED
    assert L.alcs_unpack(None, None, None) == alcs.ALCS_ERR_INVALID_ARG
    assert b"ALCS_ERR_SHAPE" in L.alcs_strerror(alcs.ALCS_ERR_SHAPE)
    L.alcs_packed_free(None)


def test_device_entry_points_fail_loudly_without_upload(alcs):
    """No CPU fallback: a convolution on weights that were never uploaded is an error."""
    W, M = _case(6, 8, 8, 4, 0.5, np.float32)
    p = alcs.alcs_pack(W, M, 4)
    x = np.zeros((1, 8, 4), np.float32)
    y = np.zeros((1, 8, 4), np.float32)
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, x.ctypes.data, y.ctypes.data, 1, 2, 2)
    assert e.value.status in (alcs.ALCS_ERR_STATE, alcs.ALCS_ERR_CUDA)


def test_mask_generators_match_their_recipe():
    s = config_layers(0)[0]
    assert int(make_mask(s).sum()) == 2048 - round(0.7 * 2048)
    z = make_mask(config_layers(4)[-1])
    cnt = z.sum(1)
    assert cnt.min() >= 1 and cnt.max() <= 512 and 0.15 < (cnt == 1).mean() < 0.35
    sp = [l.sparsity for l in config_layers(2)]
    assert all(0.6 <= x <= 0.9 for x in sp) and len(set(sp)) == 13
