"""Plain CPU oracle for the data-parallel device ops: the elementwise steps of an AsyncSPARTA
averaging round and stage-wise gradient clipping.

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this file.  It shares no code with the CUDA library and never calls it.

Each function is the step of the paper written out in float64 with numpy (Sec. 4.2, Eq. sparta,
Eq. delta_rule, Algorithm 3 "Asynchronous sparse weight averaging, one worker's view"; Sec. 4.3 for
the clipping thresholds).  Reading taken where the text is silent: the paper prints the clipping
thresholds but not the clipping formula; the usual clip-by-norm coefficient min(1, c / (norm +
1e-6)) is used.

Pins (tests/test_oracle_pins.py): a whole round assembled from the steps equals the plain mean of
Eq. sparta; the delta rule keeps the local progress (theta_new - avg = theta - snap); a sender of
weight 0 adds nothing; the segments of one cycle tile the parameter range exactly once; the
thresholds the paper prints for S = 7 (0.3779 / 0.7558); the clipped norm equals min(norm, c); a
gradient inside the budget is returned unchanged.  No function here is left unpinned.
"""

from __future__ import annotations

import numpy as np


def sparta_segment(n_params: int, rounds_per_cycle: int, rnd: int):
    """Algorithm 3: the fraction s = 1/rounds_per_cycle of the parameters, rotated by round, the
    same on every peer: segment r = rnd mod R of R contiguous ones whose boundaries floor(n r / R)
    are rounded down to a multiple of 64 parameters (the last one ends at n)."""
    R = int(rounds_per_cycle)
    r = int(rnd) % R

    def boundary(i):
        return n_params if i == R else ((n_params * i) // R) // 64 * 64

    return boundary(r), boundary(r + 1)


def sparta_snapshot(buf: np.ndarray, lo: int, hi: int) -> np.ndarray:
    """Algorithm 3: snap <- copy(buf[P])."""
    return np.array(buf[lo:hi], dtype=np.float64, copy=True)


def sparta_accumulate(acc: np.ndarray, chunk: np.ndarray, w: float) -> np.ndarray:
    """Algorithm 3, reducer: acc += w_i c_i per arriving chunk."""
    return np.asarray(acc, dtype=np.float64) + float(w) * np.asarray(chunk, dtype=np.float64)


def sparta_deltas(acc: np.ndarray, sum_w: float, chunks):
    """Algorithm 3, reducer, all senders accounted: acc /= sum_i w_i; sender i gets acc - c_i.
    Returns (mean, [delta_i])."""
    mean = np.asarray(acc, dtype=np.float64) / float(sum_w)
    return mean, [mean - np.asarray(c, dtype=np.float64) for c in chunks]


def sparta_add_delta(buf: np.ndarray, lo: int, hi: int, delta: np.ndarray) -> np.ndarray:
    """Algorithm 3, sender: buf[P] += received deltas (buf[P] is then the group average)."""
    out = np.array(buf, dtype=np.float64, copy=True)
    out[lo:hi] += np.asarray(delta, dtype=np.float64)
    return out


def sparta_apply_round(theta: np.ndarray, lo: int, hi: int, avg: np.ndarray, snap: np.ndarray,
                       lam: float = 1.0) -> np.ndarray:
    """Eq. delta_rule: theta[I] <- theta[I] + lambda (avg[I] - snap[I]); the paper sets lambda = 1."""
    out = np.array(theta, dtype=np.float64, copy=True)
    out[lo:hi] += float(lam) * (np.asarray(avg, dtype=np.float64) - np.asarray(snap, dtype=np.float64))
    return out


def stage_clip_threshold(n_stages: int, is_tail: bool) -> float:
    """Sec. 4.3: 1 / sqrt(S) for the head and body stages, twice that for the tail."""
    t = 1.0 / np.sqrt(float(n_stages))
    return 2.0 * t if is_tail else t


def stage_clip(grads, threshold: float):
    """Clip-by-norm over all gradient tensors of one stage: norm = sqrt(sum_i ||g_i||^2),
    coef = min(1, threshold / (norm + 1e-6)).  Returns ([coef g_i], norm, coef)."""
    gs = [np.asarray(g, dtype=np.float64) for g in grads]
    norm = float(np.sqrt(sum(float(np.sum(g * g)) for g in gs)))
    coef = min(1.0, float(threshold) / (norm + 1e-6))
    return [g * coef for g in gs], norm, coef
