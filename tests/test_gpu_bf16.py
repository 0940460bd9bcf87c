"""bfloat16 weights and activations with fp32 accumulation (the paper's rule g = register bits /
element bits, Section 3.2.1, gives g = 8 for any 16-bit type).  Operands are bfloat16 bit patterns;
the oracle takes the float32 values they denote.  Tolerance: a bfloat16 output is one rounding of the
fp32 result, half an ulp = 2^-9 = 1.95e-3 relative, on top of the fp32 accumulation error (1e-5): 4e-3
of the condition scale A; an fp32 output (ALCS_Y_F32) is held to the fp32 tolerance."""
import numpy as np
import pytest

import oracle
from alcs_workloads import rng

pytestmark = pytest.mark.gpu

TOL_BF16 = 4e-3
TOL_F32 = 1e-5


def _case(seed, n, cin, cout, h, wd, g, density, stride=1):
    rows = (cout + g - 1) // g
    Wb = rng.to_bf16_bits((rng.normal(seed, 1, cout * cin) * cin ** -0.5).astype(np.float32)).reshape(cout, cin)
    Xb = rng.to_bf16_bits(rng.normal(seed, 2, n * cin * h * wd).astype(np.float32)).reshape(n, cin, h, wd)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = (0.1 * rng.normal(seed, 4, cout)).astype(np.float32)
    oh, ow = -(-h // stride), -(-wd // stride)
    Rb = rng.to_bf16_bits(rng.normal(seed, 5, n * cout * oh * ow).astype(np.float32)).reshape(n, cout, oh * ow)
    return Wb, Xb, M, b, Rb


def _run(alcs, Wb, M, Xb, b, Rb, relu, g, stride, y_f32, cfg=None):
    import torch
    dev = torch.device("cuda:0")
    n, cin, h, wd = Xb.shape
    cout = Wb.shape[0]
    oh, ow = -(-h // stride), -(-wd // stride)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(Wb, M, g, bf16=True), 0)
    xd = torch.from_numpy(Xb.view(np.int16)).to(dev).view(torch.bfloat16)
    ydt = torch.float32 if y_f32 else torch.bfloat16
    yd = torch.full((n, cout, oh * ow), float("nan"), dtype=ydt, device=dev)
    rd = None
    if Rb is not None:
        rd = torch.from_numpy(Rb.view(np.int16)).to(dev).view(torch.bfloat16)
        if y_f32:
            rd = rd.to(torch.float32)
    bd = None if b is None else torch.from_numpy(b).to(dev)
    flags = (alcs.ALCS_RELU if relu else 0) | (alcs.ALCS_Y_F32 if y_f32 else 0)
    alcs.alcs_spconv1x1_ex(p, xd, yd, n, h, wd, stride, bd, rd, flags, torch.cuda.current_stream(), cfg)
    torch.cuda.synchronize()
    assert alcs.alcs_packed_status(p) == 0
    return yd.to(torch.float32).cpu().numpy()


def _check(alcs, Wb, M, Xb, b, Rb, relu, g, stride, y_f32, cfg=None):
    Y = _run(alcs, Wb, M, Xb, b, Rb, relu, g, stride, y_f32, cfg)
    W, X = oracle.bf16_decode(Wb), oracle.bf16_decode(Xb)
    R = None if Rb is None else oracle.bf16_decode(Rb)
    Yref, A = oracle.conv1x1_ex(W, M, X, b, R, relu, g, stride, want_scale=True)
    assert np.isfinite(Y).all()
    d = np.abs(Y.astype(np.float64) - Yref)
    tol = TOL_F32 if y_f32 else TOL_BF16
    assert (d <= tol * A + 1e-300).all(), f"worst ratio {(d / np.maximum(A, 1e-300)).max():.3e}"


@pytest.mark.parametrize("n,cin,cout,h,wd,g,stride", [(3, 96, 64, 14, 14, 8, 1), (5, 80, 40, 7, 7, 8, 1), (2, 64, 64, 28, 28, 8, 2),
                                                     (2, 100, 48, 9, 13, 16, 1), (4, 72, 24, 10, 10, 4, 1), (1, 256, 128, 14, 14, 8, 1),
                                                     (3, 33, 20, 5, 7, 2, 2), (2, 40, 12, 6, 6, 1, 1)])
def test_bfloat16_against_the_oracle(alcs, n, cin, cout, h, wd, g, stride):
    Wb, Xb, M, b, Rb = _case(n + cin + h, n, cin, cout, h, wd, g, 0.3, stride)
    _check(alcs, Wb, M, Xb, b, None if stride > 1 else Rb, True, g, stride, False)
    _check(alcs, Wb, M, Xb, b, Rb, True, g, stride, True)
    _check(alcs, Wb, M, Xb, None, None, False, g, stride, False)


def test_every_bfloat16_variant(alcs):
    n, cin, cout, hw = 3, 200, 128, 420
    for g in (1, 2, 4, 8, 16):
        Wb, Xb, M, b, _ = _case(50 + g, n, cin, cout if g >= 4 else 96, hw, 1, g, 0.3)
        ran = 0
        for vi in range(alcs.alcs_variant_count()):
            v = alcs.alcs_variant_get(vi)
            if v["g"] != g or v["dtype"] != alcs.ALCS_BF16:
                continue
            for kc, stages in ((64, 2), (200, 2), (32, 4)):
                cfg = dict(pixels_per_lane=v["pixels_per_lane"], rows_per_warp=v["rows_per_warp"], warps=v["warps"],
                           min_blocks=v["min_blocks"], producer_warps=v["producer_warps"], math_mode=1, chunk_channels=kc, stages=stages)
                try:
                    _check(alcs, Wb, M, Xb, b, None, True, g, 1, False, cfg)
                except alcs.AlcsError as e:
                    assert e.status == alcs.ALCS_ERR_UNSUPPORTED
                    continue
                ran += 1
        assert ran >= 2, g


def test_integer_data_is_exact_and_roundtrip(alcs):
    """Small integers are exact in bfloat16 and in every partial sum: the fp32 output must equal the oracle
    bit for bit; pack -> unpack returns the bit patterns."""
    n, cin, cout, h, wd, g = 2, 64, 32, 8, 8, 8
    Wi = ((rng.bits64(1, 7, cout * cin) % np.uint64(9)).astype(np.float32) - 4).reshape(cout, cin)
    Xi = ((rng.bits64(2, 7, n * cin * h * wd) % np.uint64(9)).astype(np.float32) - 4).reshape(n, cin, h, wd)
    Wb, Xb = rng.to_bf16_bits(Wi), rng.to_bf16_bits(Xi)
    M = (rng.uniform01(3, 3, (cout // g) * cin) < 0.4).astype(np.uint8).reshape(cout // g, cin)
    Y = _run(alcs, Wb, M, Xb, None, None, False, g, 1, True)
    assert np.array_equal(Y.astype(np.float64), oracle.conv1x1_ex(Wi, M, Xi, None, None, False, g, 1))
    W2, M2 = alcs.alcs_unpack(alcs.alcs_pack(Wb, M, g, bf16=True))
    assert np.array_equal(M2, M) and np.array_equal(W2, Wb * np.repeat(M, g, axis=0).astype(np.uint16))
