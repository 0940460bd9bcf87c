"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by
element on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from alcs_workloads import (LayerSpec, config_layers, make_bias, make_mask, make_weights, make_x, rng,
                            with_batch)
from gpu_util import TOL, assert_parity, check_layer, run_gpu

pytestmark = pytest.mark.gpu


def _layer_arrays(s):
    return make_weights(s), make_mask(s), make_x(s), make_bias(s)


def _rand(seed, n, cin, cout, hw, g, density, dtype=np.float32, xpos=True):
    rows = (cout + g - 1) // g
    W = (rng.normal(seed, 1, cout * cin) * cin ** -0.5).reshape(cout, cin).astype(dtype)
    X = rng.normal(seed, 2, n * cin * hw).reshape(n, cin, hw)
    X = (np.abs(X) if xpos else X).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = (0.1 * rng.normal(seed, 4, cout)).astype(np.float32)
    return W, M, X, b


def _ints(seed, shape, lo=-4, hi=4):
    n = int(np.prod(shape))
    return ((rng.bits64(seed, 77, n) % np.uint64(hi - lo + 1)).astype(np.int64) + lo).reshape(shape)


def test_config1_single_layer(alcs):
    """64->128 @ 56x56, batch 1, g=4, 70 % sparse, bias + ReLU: full output against the oracle."""
    s = config_layers(0)[0]
    W, M, X, b = _layer_arrays(s)
    check_layer(alcs, W, M, X, b, True, s.g, h=s.h, wd=s.w)


@pytest.mark.parametrize("li", range(13))
def test_config2_mobilenet_batch1(alcs, li):
    s = config_layers(1)[li]
    W, M, X, b = _layer_arrays(s)
    check_layer(alcs, W, M, X, b, True, s.g, h=s.h, wd=s.w)


# ragged shapes: pixel counts that are not multiples of the vector width or the tile, output
# channels that are not a multiple of g, channel counts that are not a multiple of the chunk
RAGGED = [
    # n, cin, cout, hw, g, density
    (1, 5, 8, 3, 4, 0.5), (2, 7, 10, 49, 4, 0.5), (3, 33, 18, 50, 4, 0.4), (1, 64, 64, 257, 4, 0.3),
    (2, 100, 36, 196, 4, 0.2), (5, 70, 130, 49, 2, 0.3), (2, 40, 19, 131, 1, 0.3),
    (3, 130, 72, 36, 8, 0.25), (2, 90, 50, 100, 16, 0.5), (1, 300, 24, 1030, 4, 0.15),
    (7, 257, 44, 12, 4, 0.3), (1, 1, 4, 1, 4, 1.0), (2, 3, 2, 5, 1, 0.6),
]


@pytest.mark.parametrize("n,cin,cout,hw,g,density", RAGGED)
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_ragged_shapes(alcs, n, cin, cout, hw, g, density, dtype):
    W, M, X, b = _rand(n * 1000 + cin + hw, n, cin, cout, hw, g, density, dtype)
    check_layer(alcs, W, M, X, b, True, g)
    check_layer(alcs, W, M, X, None, False, g)


@pytest.mark.parametrize("g", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("dtype", [np.float32, np.float16])
def test_zero_and_full_sparsity_exact(alcs, g, dtype):
    """100 % sparsity: Y is exactly the bias (clamped); empty rows never read X.  0 % sparsity on
    small-integer data: exactly the dense product."""
    n, cin, cout, hw = 2, 48, 32, 200
    W, _, X, b = _rand(g, n, cin, cout, hw, g, 1.0, dtype)
    rows = cout // g
    M0 = np.zeros((rows, cin), np.uint8)
    for relu in (False, True):
        Y = run_gpu(alcs, W, M0, X, b, relu, g, y_f32=(dtype == np.float16))
        exp = np.broadcast_to(b[None, :, None], Y.shape)
        exp = np.maximum(exp, 0) if relu else exp
        assert np.array_equal(Y, exp)
    Wi = _ints(g + 10, (cout, cin)).astype(dtype)
    Xi = _ints(g + 20, (n, cin, hw)).astype(dtype)
    bi = _ints(g + 30, (cout,)).astype(np.float32)
    M1 = np.ones((rows, cin), np.uint8)
    check_layer(alcs, Wi, M1, Xi, bi, False, g, exact=True, y_f32=(dtype == np.float16))


@pytest.mark.parametrize("g", [1, 4, 8])
def test_integer_data_is_bit_exact_in_any_order(alcs, g):
    """Small integers: all partial sums are exact in fp32, so the GPU must equal the oracle bit
    for bit whatever its summation order."""
    n, cin, cout, hw = 3, 200, 64, 333
    rows = cout // g
    W = _ints(1, (cout, cin)).astype(np.float32)
    X = _ints(2, (n, cin, hw)).astype(np.float32)
    b = _ints(3, (cout,)).astype(np.float32)
    M = (rng.uniform01(4, 3, rows * cin) < 0.3).astype(np.uint8).reshape(rows, cin)
    check_layer(alcs, W, M, X, b, True, g, exact=True)


def test_empty_and_full_rows_and_skew(alcs):
    """Rows with no kept block, rows with every block kept, and Zipf-skewed row lengths."""
    from alcs_workloads import zipf_block_mask
    n, cin, cout, hw, g = 2, 160, 96, 300, 4
    W, M, X, b = _rand(9, n, cin, cout, hw, g, 0.3)
    M[0] = 0; M[5] = 0; M[-1] = 0; M[3] = 1; M[7] = 1
    check_layer(alcs, W, M, X, b, True, g)
    Mz = zipf_block_mask(cout // g, cin, 123)
    check_layer(alcs, W, Mz, X, b, True, g)


def test_signed_inputs_and_cancellation(alcs):
    W, M, X, b = _rand(11, 2, 256, 64, 500, 4, 0.5, xpos=False)
    check_layer(alcs, W, M, X, b, False, 4)


def test_fp16_output_modes(alcs):
    W, M, X, b = _rand(12, 2, 128, 64, 392, 8, 0.25, np.float16)
    check_layer(alcs, W, M, X, b, True, 8)
    check_layer(alcs, W, M, X, b, True, 8, y_f32=True)


def test_run_to_run_determinism(alcs):
    W, M, X, b = _rand(13, 4, 256, 128, 196, 4, 0.2)
    Y1 = run_gpu(alcs, W, M, X, b, True, 4)
    Y2 = run_gpu(alcs, W, M, X, b, True, 4)
    assert np.array_equal(Y1, Y2)


def test_misaligned_buffers_take_the_elementwise_path(alcs):
    """x / y offset by one element from a 16-byte boundary: same results."""
    import torch
    W, M, X, b = _rand(14, 2, 40, 24, 100, 4, 0.4)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    dev = torch.device("cuda:0")
    xbuf = torch.zeros(X.size + 1, device=dev)
    ybuf = torch.full((2 * 24 * 100 + 1,), float("nan"), device=dev)
    xbuf[1:].copy_(torch.from_numpy(X.reshape(-1)))
    alcs.alcs_spconv1x1(p, xbuf.data_ptr() + 4, ybuf.data_ptr() + 4, 2, 10, 10, torch.from_numpy(b).to(dev),
                        alcs.ALCS_RELU, torch.cuda.current_stream())
    torch.cuda.synchronize()
    Y = ybuf[1:].cpu().numpy().reshape(2, 24, 100)
    Yref, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
    assert_parity(Y, Yref, A, "f32")
    assert np.isnan(ybuf[0].item())


def test_guard_bands_untouched(alcs):
    """Canaries before and after Y survive (no out-of-range store on ragged tiles)."""
    import torch
    W, M, X, b = _rand(15, 3, 37, 22, 61, 2, 0.5)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 2), 0)
    dev = torch.device("cuda:0")
    pad = 1024
    ybuf = torch.full((pad + 3 * 22 * 61 + pad,), 12345.0, device=dev)
    xd = torch.from_numpy(X).to(dev)
    alcs.alcs_spconv1x1(p, xd, ybuf.data_ptr() + 4 * pad, 3, 61, 1, None, 0, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert (ybuf[:pad] == 12345.0).all() and (ybuf[-pad:] == 12345.0).all()
    Yref, A = oracle.conv1x1(W, M, X, None, False, 2, want_scale=True)
    assert_parity(ybuf[pad:-pad].cpu().numpy().reshape(3, 22, 61), Yref, A, "f32")


@pytest.mark.parametrize("g,dtype", [(4, np.float32), (1, np.float32), (2, np.float32), (8, np.float32),
                                     (16, np.float32), (4, np.float16), (8, np.float16), (16, np.float16),
                                     (1, np.float16), (2, np.float16)])
def test_every_kernel_variant(alcs, g, dtype):
    """Each compiled variant x chunk size x pipeline depth, forced through alcs_spconv1x1_cfg, on
    a shape with a ragged pixel tail and several channel chunks."""
    n, cin, cout, hw = 3, 200, 16 * g if g >= 4 else 96, 420
    W, M, X, b = _rand(100 + g, n, cin, cout, hw, g, 0.3, dtype)
    Yref, A = oracle.conv1x1(W, M, X, b, True, g, want_scale=True)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    want_dt = alcs.ALCS_F32 if dtype == np.float32 else alcs.ALCS_F16
    ran = variants = 0
    for vi in range(alcs.alcs_variant_count()):
        v = alcs.alcs_variant_get(vi)
        if v["g"] != g or v["dtype"] != want_dt or v["split_rows"] == 1:    # (split flavours: the test below)
            continue
        variants += 1
        for kc in (32, 64, 128, 200):
            for stages in (2, 3, 4):
                cfg = dict(pixels_per_lane=v["pixels_per_lane"], rows_per_warp=v["rows_per_warp"],
                           warps=v["warps"], min_blocks=v["min_blocks"], producer_warps=v["producer_warps"],
                           math_mode=v["math_mode"], consumer_groups=v["consumer_groups"], split_rows=v["split_rows"],
                           chunk_channels=kc,
                           stages=stages, row_groups=0)
                try:
                    Y = run_gpu(alcs, W, M, X, b, True, g, cfg=cfg, packed=p)
                except alcs.AlcsError as e:     # e.g. the tile does not fit shared memory
                    assert e.status == alcs.ALCS_ERR_UNSUPPORTED
                    continue
                assert_parity(Y, Yref, A, "f32" if dtype == np.float32 else "f16")
                ran += 1
    assert variants >= 1 and ran >= 4 * variants


def test_split_row_variants_on_skewed_rows(alcs):
    """Every kernel flavour that splits long block rows into parts, on Zipf-distributed row lengths with a
    few full rows: the parts' partial sums must add up to the oracle's result, run after run."""
    from alcs_workloads import zipf_block_mask
    n, cin, cout, hw, g = 3, 256, 192, 300, 4
    W, M, X, b = _rand(31, n, cin, cout, hw, g, 0.3)
    M = zipf_block_mask(cout // g, cin, 77)
    M[3] = 1; M[17] = 1
    Yref, A = oracle.conv1x1(W, M, X, b, True, g, want_scale=True)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    ran = 0
    for vi in range(alcs.alcs_variant_count()):
        v = alcs.alcs_variant_get(vi)
        if v["g"] != g or v["dtype"] != alcs.ALCS_F32 or v["split_rows"] != 1:
            continue
        for kc, stages, rg in ((32, 3, 0), (64, 2, 3), (256, 2, 5)):
            cfg = dict(pixels_per_lane=v["pixels_per_lane"], rows_per_warp=v["rows_per_warp"], warps=v["warps"],
                       min_blocks=v["min_blocks"], producer_warps=v["producer_warps"], math_mode=1, split_rows=1,
                       chunk_channels=kc, stages=stages, row_groups=rg)
            try:
                Y1 = run_gpu(alcs, W, M, X, b, True, g, cfg=cfg, packed=p)
            except alcs.AlcsError as e:
                assert e.status == alcs.ALCS_ERR_UNSUPPORTED
                continue
            assert_parity(Y1, Yref, A, "f32")
            assert np.array_equal(Y1, run_gpu(alcs, W, M, X, b, True, g, cfg=cfg, packed=p))     # deterministic
            ran += 1
    assert ran >= 8
    # integer data: bit-exact whatever the split
    Wi = _ints(41, (cout, cin)).astype(np.float32)
    Xi = _ints(42, (n, cin, hw)).astype(np.float32)
    check_layer(alcs, Wi, M, Xi, None, False, g, cfg=dict(split_rows=1, math_mode=1), exact=True)


def test_row_group_counts(alcs):
    """Splitting the block rows of one pixel tile over 1..many thread blocks."""
    n, cin, cout, hw, g = 2, 96, 256, 300, 4
    W, M, X, b = _rand(21, n, cin, cout, hw, g, 0.3)
    Yref, A = oracle.conv1x1(W, M, X, b, True, g, want_scale=True)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    for rg in (3, 4, 5, 7, 8, 16, 64):
        cfg = dict(pixels_per_lane=8, rows_per_warp=4, warps=7, min_blocks=0, chunk_channels=32,
                   stages=3, row_groups=rg)
        assert_parity(run_gpu(alcs, W, M, X, b, True, g, cfg=cfg, packed=p), Yref, A, "f32")


def test_tuned_configuration_is_used_and_correct(alcs):
    W, M, X, b = _rand(22, 8, 256, 256, 196, 4, 0.2)
    Yref, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
    Y = run_gpu(alcs, W, M, X, b, True, 4, h=14, wd=14, tune=True)
    assert_parity(Y, Yref, A, "f32")


def test_set_cfg_is_used_by_later_calls(alcs):
    """A configuration applied with alcs_spconv1x1_set_cfg (e.g. from a tuning cache) becomes the
    plan of later automatic calls for that shape, and the result is still right."""
    W, M, X, b = _rand(26, 4, 128, 128, 196, 4, 0.25)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    cfg = dict(pixels_per_lane=4, rows_per_warp=2, warps=7, chunk_channels=32, stages=3, row_groups=0,
               min_blocks=0, copy_mode=1)
    alcs.alcs_spconv1x1_set_cfg(p, 4, 14, 14, alcs.ALCS_RELU, cfg)
    plan = alcs.alcs_spconv1x1_plan(p, 4, 14, 14, alcs.ALCS_RELU)
    for k in ("pixels_per_lane", "rows_per_warp", "warps", "chunk_channels", "stages", "copy_mode"):
        assert plan[k] == cfg[k]
    Yref, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
    assert_parity(run_gpu(alcs, W, M, X, b, True, 4, h=14, wd=14, packed=p), Yref, A, "f32")
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1_set_cfg(p, 4, 14, 14, 0, dict(pixels_per_lane=5))
    assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED


def test_host_buffer_entry_point(alcs):
    import torch
    W, M, X, b = _rand(23, 4, 64, 128, 196, 4, 0.3)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    nbytes = alcs.alcs_spconv1x1_host_workspace(p, 4, 14, 14, alcs.ALCS_RELU)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda:0")
    xh = torch.from_numpy(X).pin_memory()
    yh = torch.empty((4, 128, 196), dtype=torch.float32).pin_memory()
    bh = torch.from_numpy(b).pin_memory()
    alcs.alcs_spconv1x1_host(p, xh, yh, 4, 14, 14, bh, alcs.ALCS_RELU, ws, nbytes, torch.cuda.current_stream())
    torch.cuda.synchronize()
    Yref, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
    assert_parity(yh.numpy(), Yref, A, "f32")


@pytest.mark.parametrize("graph", [False, True])
def test_stack_runner(alcs, graph):
    """A small stack run twice (second run replays the CUDA graph) against the oracle per layer."""
    import torch
    dev = torch.device("cuda:0")
    specs = [with_batch(s, 2) for s in config_layers(1)[3:8]]
    layers, keep = [], []
    for s in specs:
        W, M, X, b = _layer_arrays(s)
        p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, s.g), 0)
        xd = torch.from_numpy(X).to(dev)
        yd = torch.full((s.n, s.cout, s.hw), float("nan"), device=dev)
        bd = torch.from_numpy(b).to(dev)
        layers.append(dict(w=p, x=xd, y=yd, n=s.n, h=s.h, wd=s.w, bias=bd, flags=alcs.ALCS_RELU))
        keep.append((W, M, X, b, yd, s))
    st = alcs.alcs_stack_create(layers, alcs.ALCS_STACK_GRAPH if graph else 0)
    stream = torch.cuda.Stream()
    for it in range(2):
        for k in keep:
            k[4].fill_(float("nan"))
        torch.cuda.synchronize()
        alcs.alcs_stack_run(st, stream)
        stream.synchronize()
        for W, M, X, b, yd, s in keep:
            Yref, A = oracle.conv1x1(W, M, X, b, True, s.g, want_scale=True)
            assert_parity(yd.cpu().numpy(), Yref, A, "f32")
    alcs.alcs_stack_destroy(st)


def test_graph_stack_survives_a_larger_call_on_the_same_weights(alcs):
    """A captured stack whose layer needs repacked input rows (7x7 images: 196-byte rows) keeps its
    own repack scratch: a later plain call with the same packed matrix and a larger batch, which
    makes the matrix grow ITS scratch, must not disturb replays of the graph."""
    import torch
    dev = torch.device("cuda:0")
    W, M, X, b = _rand(71, 2, 40, 24, 49, 4, 0.5)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    xd = torch.from_numpy(X).to(dev)
    yd = torch.full((2, 24, 49), float("nan"), device=dev)
    bd = torch.from_numpy(b).to(dev)
    # a kernel that stages x (the small-problem kernel the planner may pick at batch 2 repacks nothing)
    alcs.alcs_spconv1x1_set_cfg(p, 2, 7, 7, alcs.ALCS_RELU, dict(math_mode=1))
    st = alcs.alcs_stack_create([dict(w=p, x=xd, y=yd, n=2, h=7, wd=7, bias=bd, flags=alcs.ALCS_RELU)],
                                alcs.ALCS_STACK_GRAPH)
    stream = torch.cuda.Stream()
    Yref, A = oracle.conv1x1(W, M, X, b, True, 4, want_scale=True)
    alcs.alcs_stack_run(st, stream)
    stream.synchronize()
    assert_parity(yd.cpu().numpy(), Yref, A, "f32")
    # the same weights at a larger batch, twice (grow, then reuse), on another stream
    Xb = np.concatenate([X] * 8, axis=0)
    Wb, Mb = W, M
    big = run_gpu(alcs, Wb, Mb, Xb, b, True, 4, h=7, wd=7, packed=p)
    Yb, Ab = oracle.conv1x1(W, M, Xb, b, True, 4, want_scale=True)
    assert_parity(big, Yb, Ab, "f32")
    junk = torch.full((64 << 20,), 3.0, device=dev)     # reuse whatever memory was just released
    for _ in range(2):
        yd.fill_(float("nan"))
        torch.cuda.synchronize()
        alcs.alcs_stack_run(st, stream)
        stream.synchronize()
        assert_parity(yd.cpu().numpy(), Yref, A, "f32")
    del junk
    alcs.alcs_stack_destroy(st)


def test_device_error_paths(alcs):
    import torch
    W, M, X, b = _rand(24, 1, 8, 8, 16, 4, 0.5)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, 4), 0)
    dev = torch.device("cuda:0")
    xd = torch.from_numpy(X).to(dev)
    yd = torch.empty((1, 8, 16), device=dev)
    st = torch.cuda.current_stream()
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_packed_upload(p, 0)
    assert e.value.status == alcs.ALCS_ERR_STATE
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, xd, xd, 1, 4, 4, None, 0, st)                    # aliasing
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, None, yd, 1, 4, 4, None, 0, st)
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, xd, yd, -1, 4, 4, None, 0, st)
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, xd, yd, 1, 4, 4, None, alcs.ALCS_Y_F32, st)       # Y_F32 needs fp16 weights
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p, xd, yd, 1, 4, 4, None, 0, st, cfg=dict(pixels_per_lane=5, rows_per_warp=0, warps=0,
                                                                          chunk_channels=0, stages=0, row_groups=0, min_blocks=0))
    assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED
    W3, M3, _, _ = _rand(25, 1, 8, 9, 16, 3, 0.5)
    p3 = alcs.alcs_packed_upload(alcs.alcs_pack(W3, M3, 3), 0)
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1(p3, xd, yd, 1, 4, 4, None, 0, st)                   # g = 3 has no kernel
    assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED
    alcs.alcs_spconv1x1(p, xd, yd, 0, 4, 4, None, 0, st)                        # empty batch: no-op
    alcs.alcs_spconv1x1(p, xd, yd, 1, 0, 4, None, 0, st)
    torch.cuda.synchronize()
