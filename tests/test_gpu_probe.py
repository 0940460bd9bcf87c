"""The measurement probes: they must run, and their numbers must be physically sensible (an FMA
rate between half of and just above the unit-count peak, shared-memory load costs of at least one
pipe cycle and at most a few per 128 bytes, a segment loop that is slower than pure FMAs)."""
import pytest

pytestmark = pytest.mark.gpu


def test_fma_peak_is_close_to_the_unit_count_peak(alcs):
    for packed in (False, True):
        r = alcs.alcs_probe_fma_peak(packed)
        assert 0.5 < r["frac_of_fp32_peak"] < 1.05, r
        assert r["spill_bytes"] == 0


def test_shared_load_costs(alcs):
    distinct = alcs.alcs_probe_lds(16, False)
    uniform = alcs.alcs_probe_lds(16, True)
    assert 3.5 < distinct < 6.0          # 512 bytes per instruction over a 128-byte-per-cycle pipe
    assert 0.9 < uniform < distinct
    assert 0.9 < alcs.alcs_probe_lds(4, False) < 2.0


def test_segment_loop_probe(alcs):
    peak = alcs.alcs_probe_fma_peak(True)["frac_of_fp32_peak"]
    long = alcs.alcs_probe_segment_loop(4, 8, 2, 16, False, 32)
    short = alcs.alcs_probe_segment_loop(4, 8, 2, 16, False, 1)
    assert 0.3 < short["frac_of_fp32_peak"] <= long["frac_of_fp32_peak"] * 1.02 < peak
    assert long["spill_bytes"] == 0
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_probe_segment_loop(4, 8, 5, 16, False, 4)
    assert e.value.status == alcs.ALCS_ERR_UNSUPPORTED
    with pytest.raises(alcs.AlcsError) as e:
        alcs.alcs_probe_segment_loop(4, 8, 2, 16, False, 0)
    assert e.value.status == alcs.ALCS_ERR_INVALID_ARG
