"""The issue-rate probes run and give numbers of the expected kind (a B200 is assumed, not particular values)."""
import pytest

pytestmark = pytest.mark.gpu


def test_issue_rates_are_plausible():
    from paper_1505_04956_b200 import peaks
    r = dict(zip(peaks.NAMES, peaks.issue_rates()))
    assert len(r) == 13
    for name, v in r.items():
        assert 0.4 < v < 40.0, (name, v)
    # a scalar FMA issues about every cycle; the half-rate kinds take about two
    assert r["FFMA (two immediates)"] < 1.5
    assert r["LOP3"] > 1.5 * r["FFMA (two immediates)"]


def test_mma_rates_are_plausible():
    from paper_1505_04956_b200 import peaks
    r = dict(zip(peaks.MMA_NAMES, peaks.mma_rates()))
    assert len(r) == 12
    for name, v in r.items():
        assert 16.0 < v < 2000.0, (name, v)
    # a commit in the stream holds the issuing thread; a second issuing thread fills the gap
    assert r["tcgen05.mma 128x256x16, walking, commit every 4"] > 1.3 * r["tcgen05.mma 128x256x16, walking four chunks"]
    assert r["N=256 two issuing threads, commit every 4"] < r["tcgen05.mma 128x256x16, walking, commit every 4"]
