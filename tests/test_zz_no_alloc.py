"""alcs_spconv1x1_noalloc: the entry point for callers that are not allowed to allocate device
memory (a serving loop that must not touch the allocator, a process that has already handed all
free device memory to someone else, a plugin host that forbids allocation after start-up).

It must give what alcs_spconv1x1 gives.  The interesting inputs are those whose rows are not a
multiple of 16 bytes (7x7 images): there alcs_spconv1x1 repacks x into scratch it allocates, while
this entry point uses the fixed array built into the library.  Two calls in a row, with different
inputs, check that nothing left in that shared array by the first call leaks into the second.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test; it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

import oracle
from alcs_workloads import rng
from gpu_util import TOL, assert_parity

pytestmark = pytest.mark.gpu


def _case(seed, n, cin, cout, hw, g, density, dtype=np.float32):
    rows = (cout + g - 1) // g
    W = (rng.normal(seed, 1, cout * cin) * cin ** -0.5).reshape(cout, cin).astype(dtype)
    X = np.abs(rng.normal(seed, 2, n * cin * hw)).reshape(n, cin, hw).astype(dtype)
    M = (rng.uniform01(seed, 3, rows * cin) < density).astype(np.uint8).reshape(rows, cin)
    b = (0.1 * rng.normal(seed, 4, cout)).astype(np.float32)
    return W, M, X, b


@pytest.mark.parametrize("h,wd,dtype,g", [(7, 7, np.float32, 4), (14, 14, np.float32, 4), (7, 7, np.float16, 8)])
def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row(alcs, h, wd, dtype, g):
    import torch
    dev = torch.device("cuda:0")
    n, cin, cout = 8, 96, 64
    hw = h * wd
    kind = "f32" if dtype == np.float32 else "f16"
    W, M, X1, b = _case(700 + hw, n, cin, cout, hw, g, 0.3, dtype)
    X2 = (np.abs(rng.normal(900 + hw, 2, n * cin * hw)).reshape(n, cin, hw) * 3.0).astype(dtype)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    bd = torch.from_numpy(b).to(dev)
    st = torch.cuda.current_stream()
    flags = alcs.ALCS_RELU
    # Pin a kernel that stages x through shared memory (math_mode 1 = CUDA cores, 2 = tensor cores):
    # at this batch size the planner may otherwise pick the small-problem kernel, which reads x in
    # place, needs no scratch and would leave the fixed array untested.
    alcs.alcs_spconv1x1_set_cfg(p, n, h, wd, flags, dict(math_mode=1 if dtype == np.float32 else 2))
    assert alcs.alcs_spconv1x1_plan(p, n, h, wd, flags)["math_mode"] in (1, 2)
    ydt = torch.float32 if dtype == np.float32 else torch.float16
    for X in (X1, X2):
        xd = torch.from_numpy(X).to(dev)
        y_ref = torch.full((n, cout, hw), float("nan"), device=dev, dtype=ydt)
        y_new = torch.full((n, cout, hw), float("nan"), device=dev, dtype=ydt)
        # the ordinary entry point: also what makes the launch schedule resident for this shape
        alcs.alcs_spconv1x1(p, xd, y_ref, n, h, wd, bd, flags, st)
        alcs.alcs_spconv1x1_noalloc(p, xd, y_new, n, h, wd, bd, flags, st)
        torch.cuda.synchronize()
        Yref, A = oracle.conv1x1(W, M, X, b, True, g, want_scale=True)
        a, r = y_new.cpu().numpy(), y_ref.cpu().numpy()
        assert np.isfinite(a).all()
        assert (np.abs(a.astype(np.float64) - r.astype(np.float64)) <= TOL[kind] * A).all()
        assert_parity(a, Yref, A, kind)
    assert alcs.alcs_packed_status(p) == 0


def test_noalloc_refuses_what_it_cannot_do_without_allocating(alcs):
    """No resident schedule for the shape -> ALCS_ERR_STATE; a repacked input larger than the
    fixed array -> ALCS_ERR_TOO_LARGE.  Neither launches anything."""
    import torch
    dev = torch.device("cuda:0")
    g = 4
    W, M, X, b = _case(71, 2, 16, 8, 49, g, 0.5)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(W, M, g), 0)
    xd = torch.from_numpy(X).to(dev)
    yd = torch.empty((2, 8, 49), device=dev)
    st = torch.cuda.current_stream()
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1_noalloc(p, xd, yd, 2, 7, 7, None, 0, st)       # shape never run before
    assert e.value.status == alcs.ALCS_ERR_STATE
    # a shape whose padded input would need more than the fixed scratch: cin*n*52*4 bytes
    n_big = alcs.ALCS_NOALLOC_SCRATCH_BYTES // (16 * 52 * 4) + 1
    xb = torch.zeros((n_big, 16, 49), device=dev)
    yb = torch.empty((n_big, 8, 49), device=dev)
    alcs.alcs_spconv1x1(p, xb, yb, n_big, 7, 7, None, 0, st)              # fine for the allocating call
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_spconv1x1_noalloc(p, xb, yb, n_big, 7, 7, None, 0, st)
    assert e.value.status == alcs.ALCS_ERR_TOO_LARGE
    torch.cuda.synchronize()
