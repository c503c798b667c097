"""CPU oracle for the threshold-tuning helpers (plain numpy / Python, written from the definitions).

TEST INFRASTRUCTURE.  Only tests may import this module; the product never does.

The paper tunes the threshold T on a small development set by running FSD at candidate
thresholds and looking at the resulting speed (Section "Selecting T", Table "T tuning"); it
gives no algorithm.  Because FSD's decision is deterministic given the divergences (Discussion,
"Potential further developments"), everything a sweep over T needs is already in the divergence
matrix D[B, gamma] that a verification call returns.  The reading used here:

  * accepted length of a row at threshold T: the number of leading positions whose divergence
    passes the test (D < T, or D <= T), i.e. the index of the first failing position -- the same
    rule as in verification (Section 3.2, step 3; Section 2 "first rejection").  A NaN
    divergence (non-finite input) never passes.
  * the speed proxy is the mean accepted length over the rows (each verification step emits the
    accepted tokens plus one);
  * sweep: that mean, and the accepted fraction of all positions, for each candidate T;
  * calibrate: the smallest float T >= 0 whose mean accepted length reaches a target, found here
    by brute force over every candidate value at which the mean can change;
  * labels: the per-position outcome D cmp T, ignoring the prefix rule (the token-level data set
    the Discussion proposes for a learned acceptance predictor).

Nothing here uses prefix maxima, sorting networks or histograms: the definitions are evaluated
as they stand, so that the GPU path (which does use them) is checked against something else.
"""

from __future__ import annotations

import numpy as np


def _passes(d: float, T: float, cmp: str) -> bool:
    if d != d:                      # NaN never passes
        return False
    return d < T if cmp == "lt" else d <= T


def accepted_lengths(D: np.ndarray, T: float, cmp: str = "lt") -> np.ndarray:
    """Index of the first failing position of every row (gamma if none fails)."""
    D = np.asarray(D, dtype=np.float32)
    T = float(np.float32(T))
    B, G = D.shape
    out = np.zeros(B, dtype=np.int64)
    for b in range(B):
        n = 0
        while n < G and _passes(float(D[b, n]), T, cmp):
            n += 1
        out[b] = n
    return out


def threshold_sweep(D: np.ndarray, thresholds, cmp: str = "lt"):
    """(mean accepted length, accepted fraction of all positions) for each candidate threshold."""
    D = np.asarray(D, dtype=np.float32)
    B, G = D.shape
    mean_len, frac = [], []
    for T in thresholds:
        n = accepted_lengths(D, T, cmp)
        total = int(n.sum())
        mean_len.append(np.float32(np.float64(total) / np.float64(B)))
        frac.append(np.float32(np.float64(total) / np.float64(B * G)))
    return np.array(mean_len, dtype=np.float32), np.array(frac, dtype=np.float32)


def calibrate_threshold(D: np.ndarray, target_mean_len: float, cmp: str = "lt"):
    """Smallest float32 T >= 0 with mean accepted length >= target, and the mean it achieves.

    The mean can only change at a divergence value (under <=) or just above one (under <), so
    those are the only candidates besides 0; +inf if no finite threshold reaches the target.
    The number of accepted positions needed is ceil(target * B), at least 0 and at most B * gamma.
    """
    D = np.asarray(D, dtype=np.float32)
    B, G = D.shape
    need = int(np.ceil(np.float64(np.float32(target_mean_len)) * B))
    need = min(max(need, 0), B * G)
    cands = {np.float32(0.0)}
    for v in D.ravel():
        if v == v and v >= 0 and np.isfinite(v):
            cands.add(np.float32(v))
            cands.add(np.nextafter(np.float32(v), np.float32(np.inf)))
    best = None
    for T in sorted(cands):
        if not np.isfinite(T):
            continue
        total = int(accepted_lengths(D, T, cmp).sum())
        if total >= need:
            best = (np.float32(T), total)
            break
    if best is None:
        total = int(accepted_lengths(D, np.float32(np.inf), cmp).sum())
        return np.float32(np.inf), np.float32(np.float64(total) / np.float64(B))
    return best[0], np.float32(np.float64(best[1]) / np.float64(B))


def accept_labels(D: np.ndarray, T: float, cmp: str = "lt") -> np.ndarray:
    """1 where the position's own divergence passes the test, else 0 (NaN: 0)."""
    D = np.asarray(D, dtype=np.float32)
    T = float(np.float32(T))
    out = np.zeros(D.shape, dtype=np.uint8)
    for idx in np.ndindex(*D.shape):
        out[idx] = 1 if _passes(float(D[idx]), T, cmp) else 0
    return out
