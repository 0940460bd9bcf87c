"""Pins of the latency-model oracle (Section 3.3) and of the projection oracle (Algorithm 1) against
things other than themselves: hand-computed values, the library interpolation routine, closed
forms, a brute-force greedy selection, and planted mistakes that the pins must reject."""
from fractions import Fraction

import numpy as np
import pytest

from alcs_workloads import rng
from oracle import latency as L


def _tables(seed, sizes, monotone=True):
    """11 knots 0, 0.1N, ..., N per layer (Section 3.3) with seeded, increasing run times."""
    out = []
    for l, n in enumerate(sizes):
        k = [int(round(n * i / 10)) for i in range(11)]
        inc = rng.uniform01_f64(seed, 10 + l, 10) * 3.0 + (0.05 if monotone else -1.0)
        t = np.concatenate([[0.5 + l], 0.5 + l + np.cumsum(inc)])
        out.append((k, list(map(float, t))))
    return out


def test_interpolation_hand_example():
    k, t = [0, 10, 20], [1.0, 2.0, 5.0]
    assert L.layer_latency(k, t, 0) == 1.0
    assert L.layer_latency(k, t, 10) == 2.0
    assert L.layer_latency(k, t, 20) == 5.0
    assert abs(L.layer_latency(k, t, 15) - 3.5) < 1e-12       # 1 + 0.1*10 + 0.3*5
    assert abs(L.layer_latency(k, t, 4) - 1.4) < 1e-12


def test_interpolation_hits_the_measured_points_and_matches_numpy_interp():
    (k, t), = _tables(3, [5000], monotone=False)
    for ki, ti in zip(k, t):
        assert abs(L.layer_latency(k, t, ki) - ti) < 1e-9
    for s in [1, 17, 499, 500, 501, 2500, 4999]:
        assert abs(L.layer_latency(k, t, s) - float(np.interp(s, k, t))) < 1e-9


def test_interpolation_exact_rational():
    k, t = [0, 3, 7, 12], [0.25, 1.5, 1.0, 4.0]
    for s in range(13):
        i = max(j for j in range(3) if k[j] <= s) if s < 12 else 2
        exact = Fraction(t[i]) + (Fraction(t[i + 1]) - Fraction(t[i])) * Fraction(s - k[i], k[i + 1] - k[i])
        assert abs(Fraction(L.layer_latency(k, t, s)) - exact) < Fraction(1, 10 ** 12)


def test_network_latency_is_tau_plus_layer_sum():
    tabs = _tables(5, [100, 2000, 30])
    s = [40, 1234, 30]
    exp = 0.75 + sum(float(np.interp(si, k, t)) for (k, t), si in zip(tabs, s))
    assert abs(L.network_latency(0.75, tabs, s) - exp) < 1e-9
    assert L.network_latency(0.75, tabs, [0, 0, 0]) == 0.75 + sum(t[0] for _, t in tabs)


def test_group_keys_small_integers_exact():
    U = np.array([[1, -2], [3, 0], [0, 4], [2, 2], [5, 1]], dtype=np.float32)       # cout = 5, g = 2: ragged
    assert np.array_equal(L.group_keys(U, 2), np.array([[10, 4], [4, 20], [25, 1]], dtype=np.float32))


def test_group_keys_rank_like_the_true_norm():
    """Algorithm 1 ranks groups by L2 norm; the oracle ranks by the squared norm accumulated in fp32.
    On real-valued data the two rankings must agree for every pair of groups except pairs whose
    true (float64) squared norms are closer than the rounding of the fp32 key: g products and g sums,
    each within 2^-24 relative, i.e. |key - norm^2| <= 2 g 2^-24 norm^2."""
    g = 4
    U = rng.normal(77, 3, 64 * 96).reshape(64, 96).astype(np.float32)
    keys = L.group_keys(U, g).astype(np.float64).reshape(-1)
    U64 = U.astype(np.float64)
    true_sq = (U64.reshape(64 // g, g, 96) ** 2).sum(axis=1).reshape(-1)      # exact to 2^-53
    bound = 2 * g * 2.0 ** -24 * true_sq
    assert (np.abs(keys - true_sq) <= bound).all()
    # the square root is monotone: ranking by the norm is ranking by its square
    assert np.array_equal(np.argsort(np.sqrt(true_sq), kind="stable"), np.argsort(true_sq, kind="stable"))
    by_key = np.argsort(-keys, kind="stable")
    rank_key = np.empty_like(by_key)
    rank_key[by_key] = np.arange(by_key.size)
    i, j = np.triu_indices(keys.size, 1)
    disagree = (true_sq[i] > true_sq[j]) != (rank_key[i] < rank_key[j])
    near = np.abs(true_sq[i] - true_sq[j]) <= bound[i] + bound[j]
    assert not (disagree & ~near).any()
    assert disagree.sum() <= near.sum()
    # a key computed from the wrong filters (a shifted group) would not pass
    wrong = L.group_keys(np.roll(U, 1, axis=0), g).astype(np.float64).reshape(-1)
    assert (np.abs(wrong - true_sq) > bound).any()


def _layers(seed, shapes):
    return [rng.normal(seed, 20 + i, co * k).reshape(co, k).astype(np.float32) for i, (co, k) in enumerate(shapes)]


def _greedy(layers, g, tables, tau, budget):
    """The direct method of Section 3.4: rank the groups, add them one by one while the latency
    stays below the budget."""
    keys = np.concatenate([L.group_keys(U, g).reshape(-1).astype(np.float64) for U in layers])
    lay = np.concatenate([np.full(((U.shape[0] + g - 1) // g) * U.shape[1], l) for l, U in enumerate(layers)])
    order = sorted(range(keys.size), key=lambda i: (-keys[i], i))
    kept = [0] * len(layers)
    n = 0
    for i in order:
        kept[lay[i]] += 1
        if L.network_latency(tau, tables, [c * g for c in kept]) >= budget:
            break
        n += 1
    return n, order


@pytest.mark.parametrize("g", [1, 2, 4])
def test_projection_with_zero_tolerance_equals_greedy(g):
    shapes = [(8, 6), (12, 10), (4, 9)]
    layers = _layers(7 + g, shapes)
    tabs = _tables(9, [co * k for co, k in shapes])
    tau = 0.3
    lo = L.network_latency(tau, tabs, [0, 0, 0])
    hi = L.network_latency(tau, tabs, [co * k for co, k in shapes])
    for frac in (0.2, 0.5, 0.83):
        budget = lo + frac * (hi - lo)
        r = L.project_bisection(layers, g, tabs, tau, budget, 0.0)
        n_greedy, order = _greedy(layers, g, tabs, tau, budget)
        assert r["n1"] - r["n0"] == 1 and r["n0"] == n_greedy == r["n_keep"]
        assert list(r["order"]) == order
        assert r["latency"] < budget
        assert sum(int(m.sum()) for m in r["masks"]) == r["n_keep"]


def test_projection_invariants_with_tolerance():
    shapes = [(16, 20), (8, 33)]
    layers = _layers(21, shapes)
    tabs = _tables(22, [co * k for co, k in shapes])
    lo = L.network_latency(0.0, tabs, [0, 0])
    hi = L.network_latency(0.0, tabs, [co * k for co, k in shapes])
    budget, eps = lo + 0.4 * (hi - lo), 0.02 * (hi - lo)
    r = L.project_bisection(layers, 4, tabs, 0.0, budget, eps)
    kept_keys = np.concatenate([L.group_keys(U, 4)[m == 1] for U, m in zip(layers, r["masks"])])
    drop_keys = np.concatenate([L.group_keys(U, 4)[m == 0] for U, m in zip(layers, r["masks"])])
    assert kept_keys.min() >= drop_keys.max()                      # the top-N groups, nothing else
    assert r["n0"] <= r["n_keep"] <= r["n1"]
    assert abs(r["latency"] - budget) <= eps + 1e-12               # inside the tolerance band
    U = L.apply_masks(layers, r["masks"], 4)
    for u, ut, m in zip(U, layers, r["masks"]):
        full = np.repeat(m, 4, 0)[: ut.shape[0]]
        assert np.array_equal(u[full == 1], ut[full == 1]) and not u[full == 0].any()


def test_projection_extremes():
    layers = _layers(31, [(8, 5)])
    tabs = _tables(32, [40])
    all_t = L.network_latency(0.0, tabs, [40])
    r = L.project_bisection(layers, 4, tabs, 0.0, all_t + 1.0, 0.0)     # budget above the dense model
    assert r["n_keep"] >= 9                                             # bracket ends at [N-1, N]
    r = L.project_bisection(layers, 4, tabs, 0.0, -1.0, 0.0)            # nothing fits
    assert r["n_keep"] == 0 and not r["masks"][0].any()


def test_pins_reject_planted_mistakes(monkeypatch):
    """Wrong variants of the oracle's steps must fail the pins above."""
    k, t = [0, 10, 20], [1.0, 2.0, 5.0]

    def wrong_alpha(k, t, s):       # slope taken from the previous interval
        total = float(t[0])
        for i in range(len(k) - 1):
            j = max(i - 1, 0)
            a = (t[j + 1] - t[j]) / (k[j + 1] - k[j])
            total += (1.0 if s >= k[i] else 0.0) * a * min(k[i + 1] - k[i], s - k[i])
        return total

    def no_delta(k, t, s):          # the indicator dropped: intervals beyond s subtract
        return float(t[0]) + sum((t[i + 1] - t[i]) / (k[i + 1] - k[i]) * min(k[i + 1] - k[i], s - k[i])
                                 for i in range(len(k) - 1))

    assert abs(wrong_alpha(k, t, 15) - 3.5) > 1e-6
    assert abs(no_delta(k, t, 4) - 1.4) > 1e-6
    # ascending instead of descending ranking must break the greedy equality
    shapes = [(8, 6), (12, 10)]
    layers = _layers(41, shapes)
    tabs = _tables(42, [co * kk for co, kk in shapes])
    budget = 0.5 * (L.network_latency(0, tabs, [0, 0]) + L.network_latency(0, tabs, [48, 120]))
    good = L.project_bisection(layers, 4, tabs, 0.0, budget, 0.0)
    monkeypatch.setattr(L, "group_keys", lambda U, g, f=L.group_keys: -f(U, g))
    bad = L.project_bisection(layers, 4, tabs, 0.0, budget, 0.0)
    assert any(not np.array_equal(a, b) for a, b in zip(good["masks"], bad["masks"]))
