"""Comparison helpers shared by the parity tests (no method arithmetic here)."""
from __future__ import annotations

import numpy as np


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max over elements of |got - ref| / max(|ref|, rms(ref)).

    Plain relative error is unbounded where the reference crosses zero (normalised pixels,
    gates, logits); the denominator is floored by the tensor's rms.
    """
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    rms = float(np.sqrt(np.mean(ref * ref)))
    den = np.maximum(np.abs(ref), max(rms, 1e-30))
    return float(np.max(np.abs(got - ref) / den))


def rms_err(got: np.ndarray, ref: np.ndarray) -> float:
    """rms(got - ref) / rms(ref): insensitive to single rounding flips, sensitive to systematic error."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.sqrt(np.mean((got - ref) ** 2)) / max(np.sqrt(np.mean(ref * ref)), 1e-30))


def assert_close(got, ref, tol, what=""):
    e = rel_err(got, ref)
    assert e <= tol, f"{what}: relative error {e:.3e} > {tol:.1e} (max abs {np.max(np.abs(np.asarray(got, np.float64) - ref)):.3e})"
    return e


def check_masks(gpu_mask, ora_mask, ora_logits, zthr: float, band: float, what=""):
    """Masks must agree wherever the oracle logit is farther than `band` from the threshold."""
    outside = np.abs(ora_logits.astype(np.float64) - zthr) >= band
    bad = (gpu_mask != ora_mask) & outside
    assert not bad.any(), f"{what}: {int(bad.sum())} mask mismatches outside the +-{band} logit band"
    return float(1.0 - outside.mean())


def check_reductions_from_own_mask(result, gpu_mask):
    """count / centroid must be exactly the integer sums over the GPU's own mask."""
    T, hm, wm = gpu_mask.shape
    ys, xs = np.mgrid[0:hm, 0:wm]
    for t in range(T):
        m = gpu_mask[t].astype(bool)
        n = int(m.sum())
        assert int(result["count"][t]) == n, f"tool {t}: count {result['count'][t]} != {n}"
        if n == 0:
            assert result["cx"][t] == -1.0 and result["cy"][t] == -1.0
        else:
            assert result["cx"][t] == np.float32(xs[m].sum() / n), (t, result["cx"][t], xs[m].sum() / n)
            assert result["cy"][t] == np.float32(ys[m].sum() / n), (t, result["cy"][t], ys[m].sum() / n)
