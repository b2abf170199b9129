"""Host-side latency metrics against hand-computed values (paper Section V-A, Section VI)."""
import os

import pytest

from paper_2402_04466_b200.stats import latency_summary, percentile, trim_warmup

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "latency_1_to_100.txt")


def test_summary_matches_hand_computed_golden():
    want = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        want[k] = float(v)
    got = latency_summary(range(100, 0, -1))       # order must not matter
    for k, v in want.items():
        assert got[k] == pytest.approx(v, rel=1e-12, abs=1e-12), k
    assert got["n"] == 100


def test_percentile_edges():
    assert percentile([3.0], 0) == 3.0 and percentile([3.0], 100) == 3.0
    assert percentile([1.0, 2.0], 50) == 1.5
    with pytest.raises(ValueError):
        percentile([], 50)
    with pytest.raises(ValueError):
        percentile([1.0], 101)


def test_trim_drops_first_and_last_ten():
    v = list(range(1000))
    t = trim_warmup(v)
    assert t[0] == 10 and t[-1] == 989 and len(t) == 980
    assert trim_warmup(list(range(20))) == []
    assert latency_summary([5.0, 5.0, 5.0])["flatness_p90_p10_ms"] == 0.0
