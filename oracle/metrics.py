"""Comparison metrics used by the parity tests (test infrastructure, no codec arithmetic).

Element-wise relative error is meaningless at the zero crossings of a signed tensor, so the
parity metric normalises every element's error by max(|expected|, rms(expected)).
"""

from __future__ import annotations

import numpy as np


def max_rel_err(got: np.ndarray, expected: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    expected = np.asarray(expected, dtype=np.float64)
    if got.shape != expected.shape:
        raise ValueError(f"shape mismatch {got.shape} vs {expected.shape}")
    if expected.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(expected * expected)))
    floor = rms if rms > 0.0 else 1.0
    return float(np.max(np.abs(got - expected) / np.maximum(np.abs(expected), floor)))


def fro_rel_err(got: np.ndarray, expected: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    expected = np.asarray(expected, dtype=np.float64)
    denom = float(np.linalg.norm(expected))
    return float(np.linalg.norm(got - expected)) / (denom if denom > 0.0 else 1.0)
