"""Helpers shared by the tests: the error metric and problem builders that hand the same seeded
inputs to the CUDA library and to the CPU oracle."""
import numpy as np


def rel_err(x, y):
    """max_i |x_i - y_i| / max(|y_i|, rms(y)) -- relative error that stays defined where the
    reference element is near zero (y is the oracle's value)."""
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    y = np.asarray(y, dtype=np.float64).reshape(-1)
    rms = float(np.sqrt(np.mean(y * y))) if y.size else 0.0
    den = np.maximum(np.abs(y), max(rms, 1e-30))
    return float((np.abs(x - y) / den).max()) if y.size else 0.0


def outlier_fraction(x, y, tol):
    """Fraction of elements whose error (same metric as rel_err) exceeds tol."""
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    y = np.asarray(y, dtype=np.float64).reshape(-1)
    rms = float(np.sqrt(np.mean(y * y)))
    den = np.maximum(np.abs(y), max(rms, 1e-30))
    return float(np.mean(np.abs(x - y) / den > tol))


def l2_rel(x, y):
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    y = np.asarray(y, dtype=np.float64).reshape(-1)
    return float(np.linalg.norm(x - y) / max(np.linalg.norm(y), 1e-30))
