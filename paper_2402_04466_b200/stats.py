"""End-to-end latency determinism metrics (host-side measurement logic).

Definitions follow the paper's Section V-A "End-to-end Latency Determinism Metrics":
mean, maximum, standard deviation, distribution tail = P100 - P95 and distribution
flatness = P90 - P10 of the observed per-frame latencies, and its Section VI protocol of
discarding the first and last 10 messages of every run.  The benchmark's own p50/p99 and
p99 - p50 spread are reported beside them.  Percentiles use linear interpolation between
order statistics (the paper does not name an estimator).
"""
from __future__ import annotations

import math
from typing import Dict, Iterable, List, Sequence


def percentile(sorted_vals: Sequence[float], q: float) -> float:
    """q in [0, 100]; linear interpolation at rank q/100*(n-1) of an ascending sequence."""
    n = len(sorted_vals)
    if n == 0:
        raise ValueError("percentile of an empty sequence")
    if not 0.0 <= q <= 100.0:
        raise ValueError("q must lie in [0, 100]")
    pos = (q / 100.0) * (n - 1)
    lo = int(math.floor(pos))
    hi = min(lo + 1, n - 1)
    frac = pos - lo
    return float(sorted_vals[lo]) + frac * (float(sorted_vals[hi]) - float(sorted_vals[lo]))


def trim_warmup(vals: Sequence[float], head: int = 10, tail: int = 10) -> List[float]:
    """Drop the first `head` and last `tail` samples (warm-up and cool-down messages)."""
    vals = list(vals)
    if len(vals) <= head + tail:
        return []
    return vals[head:len(vals) - tail]


def latency_summary(latencies_ms: Iterable[float]) -> Dict[str, float]:
    v = sorted(float(x) for x in latencies_ms)
    if not v:
        raise ValueError("no latency samples")
    n = len(v)
    mean = sum(v) / n
    var = sum((x - mean) ** 2 for x in v) / n
    p = {q: percentile(v, q) for q in (10, 50, 90, 95, 99, 100)}
    return {
        "n": n,
        "mean_ms": mean,
        "std_ms": math.sqrt(var),
        "max_ms": p[100],
        "p10_ms": p[10],
        "p50_ms": p[50],
        "p90_ms": p[90],
        "p95_ms": p[95],
        "p99_ms": p[99],
        "tail_p100_p95_ms": p[100] - p[95],
        "flatness_p90_p10_ms": p[90] - p[10],
        "spread_p99_p50_ms": p[99] - p[50],
    }
