"""GPU parity of alcs_project_bisection (Algorithm 1) against the oracle: the ranking keys are
computed in the same precision on both sides, so masks, bracket and kept counts must agree bit for
bit; the projected tensors must equal the masked inputs exactly."""
import numpy as np
import pytest

from alcs_workloads import rng
from oracle import latency as L

pytestmark = pytest.mark.gpu


def _tables(seed, sizes):
    out = []
    for l, n in enumerate(sizes):
        k = [int(round(n * i / 10)) for i in range(11)]
        t = np.concatenate([[0.5 + l], 0.5 + l + np.cumsum(rng.uniform01_f64(seed, 10 + l, 10) * 3.0 + 0.05)])
        out.append((k, [float(x) for x in t]))
    return out


def _run(alcs, layers, g, tabs, tau, budget, eps, want_u=True):
    import torch
    dev = torch.device("cuda:0")
    ud = [torch.from_numpy(u).to(dev) for u in layers]
    total = sum(((u.shape[0] + g - 1) // g) * u.shape[1] for u in layers)
    mask = torch.full((total,), 7, dtype=torch.uint8, device=dev)
    outs = [torch.full_like(u, float("nan")) for u in ud] if want_u else None
    r = alcs.alcs_project_bisection(ud, g, tabs, tau, budget, eps, mask, outs, torch.cuda.current_stream())
    return r, mask.cpu().numpy(), [o.cpu().numpy() for o in outs] if want_u else None


@pytest.mark.parametrize("g", [1, 4, 8])
@pytest.mark.parametrize("frac,eps_frac", [(0.3, 0.0), (0.62, 0.01), (0.9, 0.0)])
def test_projection_matches_oracle(alcs, g, frac, eps_frac):
    shapes = [(64, 32), (130, 64 * 9), (256, 100), (30, 7)]          # ragged last groups included
    layers = [rng.normal(100 + g, 20 + i, co * k).reshape(co, k).astype(np.float32) for i, (co, k) in enumerate(shapes)]
    tabs = _tables(5, [co * k for co, k in shapes])
    tau = 0.4
    lo = L.network_latency(tau, tabs, [0] * 4)
    hi = L.network_latency(tau, tabs, [((co + g - 1) // g) * k * g for co, k in shapes])
    budget, eps = lo + frac * (hi - lo), eps_frac * (hi - lo)
    ref = L.project_bisection(layers, g, tabs, tau, budget, eps)
    r, mask, outs = _run(alcs, layers, g, tabs, tau, budget, eps)
    assert (r["n_keep"], r["n0"], r["n1"], r["iters"]) == (ref["n_keep"], ref["n0"], ref["n1"], ref["iters"])
    assert r["latency"] == ref["latency"]
    assert np.array_equal(mask, np.concatenate([m.reshape(-1) for m in ref["masks"]]))
    assert r["kept_per_layer"] == [int(m.sum()) for m in ref["masks"]]
    for o, e in zip(outs, L.apply_masks(layers, ref["masks"], g)):
        assert np.array_equal(o, e)


def test_projection_with_ties(alcs):
    """Many equal keys (small-integer weights): equal groups keep (layer, row, column) order."""
    layers = [((rng.bits64(9, i, co * k) % np.uint64(3)).astype(np.float32) - 1).reshape(co, k)
              for i, (co, k) in enumerate([(16, 40), (8, 64)])]
    tabs = _tables(6, [16 * 40, 8 * 64])
    budget = 0.5 * (L.network_latency(0, tabs, [0, 0]) + L.network_latency(0, tabs, [640, 512]))
    ref = L.project_bisection(layers, 4, tabs, 0.0, budget, 0.0)
    r, mask, _ = _run(alcs, layers, 4, tabs, 0.0, budget, 0.0, want_u=False)
    assert r["n_keep"] == ref["n_keep"]
    assert np.array_equal(mask, np.concatenate([m.reshape(-1) for m in ref["masks"]]))


def test_projection_feeds_the_packer(alcs):
    """The mask layout is the block_mask layout of alcs_pack: pack the projected layer and run it."""
    import torch
    import oracle
    g, cout, cin, hw = 4, 64, 48, 100
    U = rng.normal(77, 1, cout * cin, sigma=cin ** -0.5).reshape(cout, cin).astype(np.float32)
    tabs = _tables(8, [cout * cin])
    budget = L.network_latency(0, tabs, [cout * cin * 3 // 10])
    r, mask, outs = _run(alcs, [U], g, tabs, 0.0, budget, 0.0)
    M = mask.reshape(cout // g, cin)
    assert abs(int(M.sum()) * g - cout * cin * 3 // 10) <= g
    X = rng.uniform01(78, 2, 2 * cin * hw).reshape(2, cin, hw)
    p = alcs.alcs_packed_upload(alcs.alcs_pack(U, M, g), 0)
    xd = torch.from_numpy(X).cuda()
    yd = torch.empty((2, cout, hw), device="cuda")
    alcs.alcs_spconv1x1(p, xd, yd, 2, 10, 10, None, 0, torch.cuda.current_stream())
    torch.cuda.synchronize()
    Yref, A = oracle.conv1x1(outs[0], np.ones_like(M), X, None, False, g, want_scale=True)   # dense conv of the projected U
    assert np.all(np.abs(yd.cpu().numpy() - Yref) <= 1e-5 * A + 1e-300)
