"""Host side of the latency model (alcs_layer_latency, alcs_network_latency: Section 3.3) against
the oracle, through the C ABI.  No GPU involved."""
import numpy as np
import pytest

from alcs_workloads import rng
from oracle import latency as L


def _table(seed, n):
    k = [int(round(n * i / 10)) for i in range(11)]
    t = np.concatenate([[0.7], 0.7 + np.cumsum(rng.uniform01_f64(seed, 1, 10) * 2 - 0.3)])
    return k, [float(x) for x in t]


def test_layer_latency_matches_oracle(alcs):
    k, t = _table(1, 12345)
    for s in [0, 1, 1234, 1235, 6000, 12344, 12345]:
        assert alcs.alcs_layer_latency(k, t, s) == L.layer_latency(k, t, s)


def test_network_latency_matches_oracle(alcs):
    tabs = [_table(2 + i, n) for i, n in enumerate([100, 5000, 77])]
    s = [33, 4999, 0]
    assert alcs.alcs_network_latency(0.25, tabs, s) == L.network_latency(0.25, tabs, s)


def test_latency_errors(alcs):
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_layer_latency([0, 5, 5], [1.0, 2.0, 3.0], 2)       # knots not strictly ascending
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
    with pytest.raises(alcs.AlcsError):
        alcs.alcs_layer_latency([0], [1.0], 0)
