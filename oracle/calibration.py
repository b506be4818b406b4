"""Threshold calibration for the detection rule -- TEST INFRASTRUCTURE (part of the oracle).

Sec. "Classification via Thresholding" flags a token iff its score lies below a
threshold tau, and tau is calibrated on benign traffic for a target false-positive
rate (appendix on score statistics: the threshold / FPR trade-off over about
250,000 benign tokens).  `threshold_at_fpr` is that calibration written out: the
largest tau that flags at most the target fraction of the benign scores.

`threshold_in_gap` is a device of the tests, not of the paper: a comparison of
decisions between two implementations whose scores agree to 2e-3 is only
well-posed when no score lies that close to tau, so the calibrated value is moved
to the centre of a nearby gap of the sorted scores that is wide enough, and the
half-width of that gap is reported as the guard band.
"""
from __future__ import annotations

import numpy as np


def threshold_at_fpr(benign_scores, fpr: float) -> float:
    """The largest tau such that #{benign score < tau} <= fpr * n (flag iff score < tau; NaN is always flagged
    and is not a calibration point)."""
    s = np.sort(np.asarray(benign_scores, dtype=np.float64))
    s = s[~np.isnan(s)]
    n = len(s)
    if n == 0:
        raise ValueError("no benign scores")
    if not (0.0 <= fpr < 1.0):
        raise ValueError("fpr must be in [0, 1)")
    k = int(np.floor(fpr * n))  # number of benign scores that may be flagged
    # tau = the (k+1)-th smallest score: exactly the k smaller ones (fewer with ties) lie strictly below it
    return float(s[k])


def threshold_in_gap(all_scores, tau: float, min_gap: float = 2e-2):
    """(tau', guard): the centre of a gap of width >= min_gap in the sorted scores and half that gap's width.
    Of the wide gaps the nearest one whose centre does not exceed tau is taken (so that no more benign scores
    are flagged than tau flags); if there is none, the nearest one above.  The ranges below the smallest and
    above the largest score count as gaps of twice the minimum width."""
    s = np.sort(np.asarray(all_scores, dtype=np.float64))
    s = s[np.isfinite(s)]
    if len(s) == 0:
        return float(tau), float("inf")
    left = np.concatenate([[s[0] - 2.0 * min_gap], s])
    right = np.concatenate([s, [s[-1] + 2.0 * min_gap]])
    width = right - left
    centre = 0.5 * (left + right)
    wide = width >= min_gap
    below = np.nonzero(wide & (centre <= tau))[0]
    pick = below if len(below) else np.nonzero(wide)[0]
    j = pick[np.argmin(np.abs(centre[pick] - tau))]
    return float(centre[j]), float(0.5 * width[j])
