"""CPU oracle of the paper's latency model (Section 3.3) and of its projection with bisection
(Section 3.4, Algorithm 1).  TEST INFRASTRUCTURE ONLY: nothing in the product package imports this.

Written step by step in the paper's notation, plain Python / numpy, no shortcuts:

  * layer_latency(k, t, s): the linear interpolation  T^(s) = t_1 + sum_i delta_i alpha_i
    min(k_{i+1} - k_i, s - k_i)  with  delta_i = [s >= k_i]  and  alpha_i = (t_{i+1} - t_i) /
    (k_{i+1} - k_i)   (the three unnumbered equations after the one for T^(l)(W^(l))).
  * network_latency(tau, tables, s): T(W) = tau + sum_l T^(l)(||W^(l)||_0).
  * group_keys(U, g): the ranking key of every group of g adjacent filters at one location
    (Section 3.2.1): its squared L2 norm, accumulated in fp32 in ascending filter order, one rounded
    multiply and one rounded add per element.  (Sorting by the squared norm orders the groups as
    the norm does; the key is kept in the precision the CUDA path ranks in, so that both sides take
    the same decision.)
  * project_bisection(...): Algorithm 1.  Groups of all layers are ranked together, largest key
    first, ties by (layer, group index) ascending; N halves the bracket [N0, N1] until the
    latencies of its ends are within eps.  ||W^(l)||_0 is read as g times the number of kept groups
    of layer l (the mask decides what counts as non-zero, as in the storage format).  The paper's
    loop has no exit for a bracket that cannot shrink (N1 - N0 <= 1 while t1 - t0 > eps); the oracle
    stops there as well.
"""
from __future__ import annotations

import numpy as np


def layer_latency(k, t, s):
    """Interpolated run time of one layer with s non-zero parameters; k[0] = 0 < ... < k[n-1] = N."""
    n = len(k)
    total = float(t[0])
    for i in range(n - 1):
        delta = 1.0 if s >= k[i] else 0.0
        alpha = (float(t[i + 1]) - float(t[i])) / (float(k[i + 1]) - float(k[i]))
        total += delta * alpha * min(float(k[i + 1]) - float(k[i]), float(s) - float(k[i]))
    return total


def network_latency(tau, tables, s):
    """tables[l] = (k, t) of layer l; s[l] = its number of non-zero parameters."""
    total = float(tau)
    for (k, t), sl in zip(tables, s):
        total += layer_latency(k, t, sl)
    return total


def group_keys(U, g):
    """U: float32 [cout, K].  Returns float32 [ceil(cout/g), K]: sum over the g filters of a group of
    the squared element, in fp32 (a missing filter of a ragged last group counts as zero)."""
    U = np.asarray(U, dtype=np.float32)
    cout, K = U.shape
    rows = (cout + g - 1) // g
    keys = np.zeros((rows, K), dtype=np.float32)
    for j in range(g):
        idx = np.arange(rows) * g + j
        ok = idx < cout
        sq = np.zeros((rows, K), dtype=np.float32)
        sq[ok] = U[idx[ok]] * U[idx[ok]]            # one rounded fp32 multiply
        keys = (keys + sq).astype(np.float32)       # one rounded fp32 add
    return keys


def project_bisection(layers, g, tables, tau, t_budget, eps):
    """Algorithm 1.  layers: list of float32 [cout_l, K_l] (the variable U~ to project).

    Returns dict(masks=[uint8 [rows_l, K_l]], n_keep=N, latency=T(U), n0, n1, iters, order)
    where `order` is the global ranking (indices into the concatenation of the layers' groups).
    """
    keys, layer_of, counts_total = [], [], []
    for l, U in enumerate(layers):
        kk = group_keys(U, g).reshape(-1)
        keys.append(kk)
        layer_of.append(np.full(kk.size, l, dtype=np.int64))
        counts_total.append(kk.size)
    keys = np.concatenate(keys)
    layer_of = np.concatenate(layer_of)
    total = keys.size
    # step 2: sort the groups by norm, largest first; equal keys keep their original order
    order = np.argsort(-keys.astype(np.float64), kind="stable")
    ranked_layer = layer_of[order]

    def latency_of_top(n):
        kept = np.bincount(ranked_layer[:n], minlength=len(layers))
        return network_latency(tau, tables, [int(c) * g for c in kept])

    n0, n1 = 0, total                              # step 3
    t0, t1 = latency_of_top(0), latency_of_top(total)   # step 4
    iters = 0
    while t1 - t0 > eps and n1 - n0 > 1:           # step 5 (second test: see the module docstring)
        n = (n0 + n1) // 2
        t = latency_of_top(n)
        if t < t_budget:
            t0, n0 = t, n
        else:
            t1, n1 = t, n
        iters += 1
    n = (n0 + n1) // 2                             # step 15
    keep = np.zeros(total, dtype=np.uint8)
    keep[order[:n]] = 1
    masks, off = [], 0
    for U, cnt in zip(layers, counts_total):
        rows = (U.shape[0] + g - 1) // g
        masks.append(keep[off:off + cnt].reshape(rows, U.shape[1]))
        off += cnt
    return {"masks": masks, "n_keep": int(n), "latency": latency_of_top(n), "n0": int(n0), "n1": int(n1),
            "iters": iters, "order": order}


def apply_masks(layers, masks, g):
    """U = the kept groups of U~, everything else zero."""
    out = []
    for U, M in zip(layers, masks):
        full = np.repeat(M, g, axis=0)[: U.shape[0]]
        out.append(np.where(full != 0, U, np.float32(0)).astype(np.float32))
    return out
